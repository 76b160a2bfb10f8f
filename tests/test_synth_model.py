"""The synthetic activation model has the structure the paper describes in Section 3."""
import numpy as np

import oracle
from paper_2211_10438_b200 import synth


def test_outlier_channels_persist_and_starve_normal_channels():
    wl = synth.WORKLOADS[5]
    C = 2048  # narrow slice of the MT-NLG-shaped stream keeps the test quick
    ch, fac = wl.outliers(C)
    assert len(ch) == int(np.ceil(0.005 * C)) and np.all(fac == 100.0)
    a = synth.activations(5, 10, 256, C, "bf16", ch, fac)
    b = synth.activations(5, 11, 256, C, "bf16", ch, fac)
    assert not np.array_equal(a, b)
    assert np.array_equal(a, synth.activations(5, 10, 256, C, "bf16", ch, fac))  # seeded
    # outliers sit in the same channels in every batch (observation 3)
    for x in (a, b):
        top = np.argsort(np.abs(x).max(0))[-len(ch):]
        assert set(top) == set(ch)
    # observation 2: under per-tensor quantisation a non-outlier channel with maximum m_i
    # keeps about 2^8 m_i / m effective levels -- a handful when outliers are ~100x
    m = np.abs(a).max()
    normal = np.setdiff1d(np.arange(C), ch)
    levels = 256 * np.abs(a[:, normal]).max(0) / m
    assert 1.0 < np.median(levels) < 4.0
    # after smoothing at alpha = 0.5 with flat weights the figure rises by about sqrt(100)
    w = synth.weights(5, 20, 64, C, "bf16")
    s = oracle.smooth_scales(oracle.calib_absmax(a), oracle.calib_absmax(w), 0.5)
    ah = a / s
    levels_s = 256 * np.abs(ah[:, normal]).max(0) / np.abs(ah).max()
    assert np.median(levels_s) > 5 * np.median(levels)


def test_workload_table_matches_layer_shapes():
    w2 = synth.WORKLOADS[2]
    assert [(l.N, l.K) for l in w2.linears] == [(15360, 5120), (5120, 5120), (20480, 5120), (5120, 20480)]
    w4 = synth.WORKLOADS[4]
    assert [(l.N, l.K) for l in w4.linears] == [(36864, 12288), (49152, 12288), (12288, 49152)]
    assert synth.WORKLOADS[3].heads * synth.WORKLOADS[3].head_dim == 7168
    x = synth.activations(1, 2, 16, 512, "f16", *synth.WORKLOADS[1].outliers())
    assert x.shape == (16, 512) and np.array_equal(x, x.astype(np.float16).astype(np.float32))

"""B200-native SmoothQuant W8A8 hot path: CUDA kernels behind a C-ABI library.

`paper_2211_10438_b200.binding` loads the in-tree shared library and exposes the
`sq_*` entry points; `paper_2211_10438_b200.synth` draws the seeded synthetic
workloads.  Importing the package itself loads nothing.
"""
__all__ = ["binding", "synth"]

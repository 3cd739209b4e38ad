"""SGNS mini-batch training and DASGD message application on one B200, as hand-written CUDA.

`paper_2211_10280_b200.binding` wraps the C-ABI library `libtensair.so` (built by
`paper_2211_10280_b200.build`); `paper_2211_10280_b200.synth` generates the seeded synthetic
inputs.  Importing the package loads nothing: the CUDA library is opened on first use and its
absence is an error, there is no CPU fallback.
"""

__all__ = ["binding", "build", "synth"]

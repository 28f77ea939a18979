"""Local-update SGD (periodic averaging + AdaComm) on one B200.

Importing the package is cheap and loads no native code; the CUDA library is
loaded by `paper_1810_08313_b200.binding` on first use and its absence is an
error, never a fallback.
"""

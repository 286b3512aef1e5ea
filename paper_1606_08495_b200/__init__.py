"""SGNS minibatch step of arXiv 1606.08495 for one B200: a C-ABI CUDA library
(`csrc/`, built by `build.py`) and a thin ctypes binding (`binding.py`).

Importing the package is cheap and needs no GPU; the CUDA library is loaded the
first time `binding` is used and its absence is an error, never a fallback.
"""
__all__ = ["corpus", "binding", "build"]

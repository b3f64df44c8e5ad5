"""NetMax (arXiv 2009.05766) round simulator for one B200: Python binding of the C-ABI library.

The CUDA library is loaded on first use of :mod:`paper_2009_05766_b200.binding`;
importing the package (for example for :mod:`workloads`) loads nothing native.
"""
__all__ = ["binding", "workloads", "build"]

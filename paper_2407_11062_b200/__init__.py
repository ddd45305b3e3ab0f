"""B200 (sm_100a) library for the group-wise low-bit quantised linear layer of
EfficientQAT: C-ABI shared library (csrc/, include/eqat.h) plus a ctypes binding.

    from paper_2407_11062_b200 import binding as eqat

The binding loads the in-tree ``libeqat_b200.so`` and raises ImportError when it
has not been built (``python -m paper_2407_11062_b200.build``); there is no
other code path.
"""
__all__ = ["binding", "build"]

"""CPU oracle for the BFP KV cache with K-sort.

TEST INFRASTRUCTURE ONLY: a plain fp64 restatement of the paper's definitions,
compiled from ``kvbfp_oracle.c`` with gcc and called through ctypes.  It shares
no code with the CUDA library and must never be imported by it.
"""
from .binding import *  # noqa: F401,F403

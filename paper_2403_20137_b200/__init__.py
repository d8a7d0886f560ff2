"""B200-native Block-Floating-Point KV cache with K-sort (arXiv 2403.20137).

The product is the C-ABI CUDA library ``libkvbfp.so`` (sources under ``csrc/``,
declarations in ``include/kvbfp.h``); :mod:`.binding` marshals arguments to it
and :mod:`.workloads` draws seeded synthetic inputs.  There is no CPU fallback:
every call raises if the CUDA library cannot be loaded.
"""

__all__ = ["binding", "workloads", "build"]

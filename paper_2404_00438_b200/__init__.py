"""B200-native Distributed-Lion optimizer step (arXiv 2404.00438).

``dlion``   -- thin binding over the C-ABI CUDA library (loads it on import and
               raises if it is missing; there is no CPU fallback)
``inputs``  -- workload shapes and seeded synthetic gradients (no optimizer math)
``build``   -- compiles the CUDA library for sm_100a
"""
__all__ = ["dlion", "inputs", "build"]

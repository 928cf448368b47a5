"""B200-native Sparse Binary Compression (arXiv 1805.08768): encode / decode-aggregate.

The compute path is a C-ABI CUDA library (``csrc/``, declared in ``include/sbc.h``);
``binding`` marshals arguments to it and nothing else.  ``workloads`` holds the
seeded synthetic inputs.  The library is loaded on first use, and a missing or
unloadable library is an error: there is no CPU fallback.
"""
__version__ = "0.1.0"

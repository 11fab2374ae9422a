"""B200-native ChunkWise-LoRA hot path: token scoring, adaptive partition, adapted projection.

The compute lives in ``csrc/`` (CUDA for sm_100a behind a C ABI, ``libcwl.so``); ``binding``
marshals torch tensors into those calls.  Nothing here falls back to the CPU: using an entry
point without the built library raises.
"""
__version__ = "0.1.0"

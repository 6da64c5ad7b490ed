"""B200-native hot path of SkipKV sentence-level KV eviction (arxiv 2512.07993).

``workloads`` draws seeded synthetic inputs; ``binding`` is the thin ctypes layer over
the C-ABI CUDA library (``libskipkv.so``).  Nothing is loaded at import time; the
binding raises if the CUDA library is missing when a call is made.
"""
__all__ = ["workloads", "binding"]

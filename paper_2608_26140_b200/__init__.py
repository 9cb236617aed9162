"""B200-native affix-cache refresh path (anchor scoring, top-K selection,
selective recomputation, KV scatter) behind a C-ABI library.

``workloads`` (seeded synthetic inputs) imports without the CUDA library;
``binding`` loads the C-ABI shared library on first use and raises if it is
missing -- there is no CPU fallback.
"""
__all__ = ["workloads", "binding"]

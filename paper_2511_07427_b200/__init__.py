"""B200-native cluster-based KV-cache retrieval (DynaKV hot path): thin Python binding.

Every step of the path runs in the CUDA kernels of ``libdynakv.so``; this package only
marshals ``torch`` device tensors (memory and streams) into the C ABI declared in
``include/dynakv.h``.  There is no CPU fallback: importing the binding without the built
library raises.
"""
from .binding import (DynaKV, DynaKVConfig, DynaKVError, load_library, F32, BF16, FP8, INIT_KMEANSPP, INIT_RANDOM,
                      MODE_ADAPTIVE, MODE_STATIC, MODE_LOCAL, MODE_DELAYED,
                      ST_BUDGET_EXCEEDED, ST_MAX_CLUSTERS, ST_MAX_TOKENS, ST_PAGE_POOL, ST_INTERNAL, ST_TIER_CACHE, ST_BOUNDS, EXPORTED_SYMBOLS, attend_rows_noalloc)

__all__ = ["DynaKV", "DynaKVConfig", "DynaKVError", "load_library", "F32", "BF16", "FP8", "INIT_KMEANSPP", "INIT_RANDOM",
           "MODE_ADAPTIVE", "MODE_STATIC", "MODE_LOCAL", "MODE_DELAYED",
           "ST_BUDGET_EXCEEDED", "ST_MAX_CLUSTERS", "ST_MAX_TOKENS", "ST_PAGE_POOL", "ST_INTERNAL", "ST_TIER_CACHE", "ST_BOUNDS", "EXPORTED_SYMBOLS",
           "attend_rows_noalloc"]

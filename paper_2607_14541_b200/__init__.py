"""B200-native trace aggregation: production trace records -> per-problem importance weights
and roofline ceilings (the paper's Sec. 3.3-3.4, Eq. 1-3), as hand-written CUDA for sm_100a
behind a C ABI (``include/atrex_agg.h``).  This package is the thin Python binding.
"""
from .binding import *  # noqa: F401,F403
from .binding import (Aggregator, AtrexError, make_peaks, topk_entries_static, score_aggregate, OperatorWeights,
                      sort_entries_by_key, rank_entries,
                      lib, LIB_PATH,  # noqa: F401
                      EXPORTED_SYMBOLS)

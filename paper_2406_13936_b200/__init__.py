"""B200-native batch-size test and fused local-optimiser kernels (C ABI in include/abs.h)."""
from . import build  # noqa: F401
from .binding import (AbsError, Context, abs_test_stats_noalloc, load_library, make_adamw_cfg, make_round_opts, make_test_cfg,  # noqa: F401
                      stats_to_dicts, plan_stats)

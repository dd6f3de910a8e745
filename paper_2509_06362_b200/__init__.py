"""B200-native scoring of candidate model-instance placements by trace replay.

Thin Python binding over the C ABI in include/maaso.h (libmaaso.so, CUDA kernels for
sm_100a).  The binding only marshals arguments: every step of the computation runs in the
library's kernels.  Importing this package fails loudly if the library cannot be loaded.
"""
from .binding import (
    MaasoError, Context, Trace,
    maaso_create, maaso_destroy, maaso_load_profile, maaso_load_trace, maaso_free_trace,
    maaso_eval_placements, maaso_eval_placements_multi, maaso_eval_placements_host, maaso_topk, maaso_ins_deploy, maaso_partition, maaso_prune_configs, maaso_score, maaso_topk_scores, maaso_ttft_percentiles, maaso_topk_noalloc, NOALLOC_MAX_CAND, NOALLOC_MAX_K, maaso_launch_count, maaso_test_fail_allocs, maaso_set_timing, maaso_get_timing,
    maaso_strerror, maaso_last_error, lib_path,
    REQUEST_DTYPE, SLO_DTYPE, RESULT_DTYPE,
    FLAG_PRED_OPTIMISTIC, FLAG_ENGINE_FROZEN, FLAG_TBT_MAXGAP, FLAG_INSTANCE_QUEUES, FLAG_TEST_STALL, MAP_AUTO, MAP_BLOCK, MAP_GROUP, MAP_THREAD, CAND_STATUS,
)

__all__ = [
    "MaasoError", "Context", "Trace", "maaso_create", "maaso_destroy", "maaso_load_profile",
    "maaso_load_trace", "maaso_free_trace", "maaso_eval_placements", "maaso_eval_placements_multi", "maaso_eval_placements_host",
    "maaso_topk", "maaso_ins_deploy", "maaso_partition", "maaso_prune_configs", "maaso_score", "maaso_topk_scores", "maaso_ttft_percentiles", "maaso_topk_noalloc", "NOALLOC_MAX_CAND", "NOALLOC_MAX_K", "maaso_launch_count", "maaso_test_fail_allocs", "maaso_set_timing", "maaso_get_timing", "maaso_strerror", "maaso_last_error", "lib_path",
    "REQUEST_DTYPE", "SLO_DTYPE", "RESULT_DTYPE", "FLAG_PRED_OPTIMISTIC", "FLAG_ENGINE_FROZEN", "FLAG_TBT_MAXGAP", "FLAG_INSTANCE_QUEUES", "MAP_AUTO", "MAP_BLOCK",
    "MAP_GROUP", "MAP_THREAD", "CAND_STATUS",
]

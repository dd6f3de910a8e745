"""CPU oracle for placement scoring.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.
It compiles oracle/maaso_oracle.c with gcc on first use and calls it through ctypes;
it imports nothing from the CUDA package.
"""
from .binding import (build, eval_placements, eval_placements_parallel, topk, score, topk_scores, rejected_by_model, ins_deploy, partition, prune_configs, ttft_hist, ttft_percentiles,
                      FLAG_PRED_OPTIMISTIC, FLAG_ENGINE_FROZEN, FLAG_TBT_MAXGAP, FLAG_INSTANCE_QUEUES, STATUS)

__all__ = ["build", "eval_placements", "eval_placements_parallel", "topk", "score", "topk_scores", "rejected_by_model", "ins_deploy", "partition", "prune_configs", "ttft_hist", "ttft_percentiles",
           "FLAG_PRED_OPTIMISTIC", "FLAG_ENGINE_FROZEN", "FLAG_TBT_MAXGAP", "FLAG_INSTANCE_QUEUES", "STATUS"]

"""Synthetic latency tables (the profiler's output, as data).

A profile is a dict of int32 arrays:
  devices[S]              modeled devices one instance of strategy s occupies
  min_devices[M]          fewest devices an instance of model m needs (memory fit)
  prefill_base_us[M][S]   fixed prefill cost
  prefill_q16[M][S]       per-input-token prefill cost in Q16 microseconds
  step_us[M][S][WMAX]     one decode step at running count w (index w-1)
plus `strategies`, a list of (tp, pp) for humans.

The affine forms and the jitter recipe are those of the benchmark configurations;
tables are quantised once here with round-half-up and are integer ever after.
"""
import numpy as np
from .formats import WMAX

# (tp, pp) with tp*pp in {1, 2, 4, 8}
STRATEGIES_NODE = [(1, 1), (2, 1), (1, 2), (4, 1), (2, 2), (1, 4),
                   (8, 1), (4, 2), (2, 4), (1, 8)]


def _rhu(x):
    """round half up to integer"""
    return np.floor(np.asarray(x, dtype=np.float64) + 0.5).astype(np.int64)


def _build(strategies, model_scale, min_devices, rng, pp_bubble, jitter):
    S, M = len(strategies), len(model_scale)
    w = np.arange(1, WMAX + 1, dtype=np.float64)
    devices = np.array([tp * pp for tp, pp in strategies], dtype=np.int32)
    base = np.zeros((M, S), dtype=np.int32)
    q16 = np.zeros((M, S), dtype=np.int32)
    step = np.zeros((M, S, WMAX), dtype=np.int32)
    for m, scale in enumerate(model_scale):
        for s, (tp, pp) in enumerate(strategies):
            bubble = 1.0 + pp_bubble * (pp - 1)
            if rng is None:
                u_step = np.ones(WMAX)
                u_base = u_slope = 1.0
            else:
                u_step = rng.uniform(1.0 - jitter, 1.0 + jitter, size=WMAX)
                u_base = rng.uniform(1.0 - jitter, 1.0 + jitter)
                u_slope = rng.uniform(1.0 - jitter, 1.0 + jitter)
            step[m, s] = np.maximum(1, _rhu(scale * (9000.0 / tp + 150.0 * w) * bubble * u_step))
            base[m, s] = _rhu(scale * (2000.0 / tp) * bubble * u_base)
            q16[m, s] = _rhu(scale * (0.12 / tp) * bubble * u_slope * 65536.0)
    return {
        "n_models": M, "n_strategies": S, "wmax": WMAX,
        "devices": devices,
        "min_devices": np.asarray(min_devices, dtype=np.int32),
        "prefill_base_us": base, "prefill_q16": q16, "step_us": step,
        "strategies": list(strategies),
    }


def profile_decay(strategies=None, model_scale=(1.0, 1.9, 9.0), min_devices=(1, 1, 4)):
    """Tables generated from the throughput decay function of the paper's profiler (Eq. 1):
    F(M,P,B,W) = T0(M,P) * (1 - delta_P * ln(eps_P + min(B, W))) tokens/s per request, so one decode
    step at level w takes 1e6 / F microseconds.  T0 = tp / (9 ms * model scale), reduced by 15 % per
    extra pipeline stage; delta_P = 0.08 + 0.02 * log2(tp * pp) (higher-degree strategies decay faster,
    as the paper observes); eps_P = 1.  Prefill as in the other profiles, without jitter."""
    strategies = STRATEGIES_NODE if strategies is None else strategies
    prof = _build(strategies, list(model_scale), list(min_devices), None, 0.15, 0.0)
    w = np.arange(1, WMAX + 1, dtype=np.float64)
    for m, scale in enumerate(model_scale):
        for s, (tp, pp) in enumerate(strategies):
            t0 = tp / (0.009 * scale) / (1.0 + 0.15 * (pp - 1))
            delta = 0.08 + 0.02 * np.log2(tp * pp)
            f = t0 * (1.0 - delta * np.log(1.0 + w))
            prof["step_us"][m, s] = np.maximum(1, _rhu(1e6 / f))
    return prof


def profile_tiny():
    """One 7B-like model, tp in {1,2,4}; exact affine tables, no jitter."""
    return _build([(1, 1), (2, 1), (4, 1)], [1.0], [1], None, 0.0, 0.0)


def profile_node(seed=0):
    """One model, the ten (tp,pp) strategies, 15 % pipeline bubble per extra stage,
    +-5 % seeded jitter per table entry."""
    return _build(STRATEGIES_NODE, [1.0], [1], np.random.default_rng(seed), 0.15, 0.05)


def profile_multimodel(seed=0):
    """Three models with base costs 1x / 1.9x / 9x; the largest needs >= 4 devices."""
    return _build(STRATEGIES_NODE, [1.0, 1.9, 9.0], [1, 1, 4],
                  np.random.default_rng(seed), 0.15, 0.05)

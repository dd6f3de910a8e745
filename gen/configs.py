"""The five benchmark configurations as seeded synthetic inputs.

make_config(name, ...) returns a dict with keys
  profile, classes, traces (list of request arrays), offsets, inst, budget, name
`n_cand` / `n_req` shrink a configuration for tests (first n_cand candidates of the
seeded set, first n_req requests of each trace); None keeps the full size.
"""
import numpy as np
from .formats import make_classes
from .profiles import profile_tiny, profile_node, profile_multimodel, profile_decay
from .traces import make_trace
from .candidates import enumerate_tiny, enumerate_node, sample_candidates

CONFIG_NAMES = ("tiny", "node", "multimodel", "bursty", "scale")

# Table I of the paper: (decode-length range, SLO-factor range, share) groups of the six traces
TABLE1 = {
    1: [((300, 1000), (0.8, 1.5), 1.0)],
    2: [((300, 500), (0.8, 1.0), 0.5), ((300, 500), (1.2, 1.5), 0.5)],
    3: [((300, 500), (0.8, 1.2), 0.5), ((600, 1000), (0.8, 1.2), 0.5)],
    4: [((300, 500), (0.8, 1.0), 0.5), ((600, 1000), (1.2, 1.5), 0.5)],
    5: [((300, 500), (0.8, 1.0), 0.34), ((300, 500), (1.2, 1.5), 0.66)],
    6: [((300, 500), (0.8, 1.0), 0.66), ((300, 500), (1.2, 1.5), 0.34)],
}


def make_table1_config(trace_no, n_cand=2000, n_req=17_000, seed=0, cv=2.0, window_s=3600.0, budget=24):
    """Paper-shaped workload (Sec. V-A): gamma arrivals (CV 2) tuned to n_req arrivals per 3600 s
    window, three models in equal shares, decode length S_r and SLO factor theta_r drawn uniformly
    from the trace's groups of Table I; the normalised deadline tau_r = d_r * theta_r * theta becomes a
    per-token budget theta_r * theta, with theta_r quantised to 0.01 (one SLO class per value, 71
    classes) and theta = one decode step of the tp=1 instance of model 0 at level 1 (the paper's
    data-parallel instance with batch size 1).  Tables from Eq. 1 (profile_decay); candidates sampled for a 24-device cluster."""
    prof = profile_decay()
    theta = int(prof["step_us"][0, 0, 0])
    factors = np.round(np.arange(0.80, 1.5001, 0.01), 2)
    classes = make_classes([(None, int(np.floor(f * theta + 0.5)), None) for f in factors])
    tr = make_trace(n_req, n_req / window_s, seed, cv=cv, class_mix=(1.0,), model_mix=(1, 1, 1), doc_class=None)
    rng = np.random.default_rng(seed + 7919)
    groups = TABLE1[trace_no]
    g = rng.choice(len(groups), size=n_req, p=[x[2] for x in groups])
    lo = np.array([x[0][0] for x in groups])[g]
    hi = np.array([x[0][1] for x in groups])[g]
    tr["out_tokens"] = rng.integers(lo, hi + 1)
    flo = np.array([x[1][0] for x in groups])[g]
    fhi = np.array([x[1][1] for x in groups])[g]
    f = np.round(flo + (fhi - flo) * rng.random(n_req), 2)
    tr["cls"] = np.clip(np.rint((f - 0.80) / 0.01), 0, len(factors) - 1).astype(np.uint8)
    offsets, inst = sample_candidates(n_cand, seed + 1, budget, prof)
    return {"name": f"table1-{trace_no}", "profile": prof, "classes": classes, "traces": [tr],
            "offsets": offsets, "inst": inst, "budget": budget}

_INTERACTIVE = (500_000, 50_000, None)
_CHAT = (2_000_000, 150_000, None)
_DOCUMENT = (None, None, 180_000_000)
_BATCH = (30_000_000, None, 600_000_000)


def _head(offsets, inst, n_cand):
    if n_cand is None or n_cand >= len(offsets) - 1:
        return offsets, inst
    return offsets[: n_cand + 1].copy(), inst[: offsets[n_cand]].copy()


def make_config(name, n_cand=None, n_req=None):
    if name == "tiny":
        prof = profile_tiny()
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT])
        traces = [make_trace(500 if n_req is None else n_req, 8.0, 0)]
        offsets, inst = enumerate_tiny()
        budget = 4
    elif name == "node":
        prof = profile_node(0)
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT])
        traces = [make_trace(10_000 if n_req is None else n_req, 16.0, 0)]
        offsets, inst = enumerate_node(prof["devices"], 8)
        budget = 8
    elif name == "multimodel":
        prof = profile_multimodel(0)
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT])
        traces = [make_trace(100_000 if n_req is None else n_req, 64.0, 0,
                             model_mix=(0.6, 0.3, 0.1))]
        offsets, inst = sample_candidates(100_000 if n_cand is None else n_cand, 1, 32, prof)
        budget = 32
    elif name == "bursty":
        prof = profile_node(0)
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT])
        traces = [make_trace(10_000 if n_req is None else n_req, 64.0 ** (j / 15.0), 100 + j,
                             cv=4.0, class_mix=(0.7, 0.2, 0.1)) for j in range(16)]
        offsets, inst = enumerate_node(prof["devices"], 8)
        budget = 8
    elif name == "scale":
        prof = profile_multimodel(0)
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT, _BATCH])
        traces = [make_trace(1_000_000 if n_req is None else n_req, 256.0, 0,
                             class_mix=(0.45, 0.27, 0.18, 0.10), model_mix=(0.6, 0.3, 0.1),
                             in_dist=("pareto", 1.5, 32.0, 32, 32768),
                             out_dist=("lognormal", 5.0, 1.2, 1, 8192))]
        offsets, inst = sample_candidates(1_000_000 if n_cand is None else n_cand, 2, 128, prof)
        budget = 128
    elif name == "large":
        # Not one of the five benchmark configurations: placements of 33 to 128 instances on a modelled
        # cluster of 1,024 devices, the case the one-warp-per-placement kernel exists for.
        prof = profile_multimodel(0)
        classes = make_classes([_INTERACTIVE, _CHAT, _DOCUMENT, _BATCH])
        traces = [make_trace(10_000 if n_req is None else n_req, 400.0, 9,
                             class_mix=(0.45, 0.27, 0.18, 0.10), model_mix=(0.6, 0.3, 0.1))]
        want = 2_000 if n_cand is None else n_cand
        offsets, inst = sample_candidates(3 * want + 64, 3, 1024, prof, stop_p=0.015)
        keep = np.nonzero(np.diff(offsets.astype(np.int64)) > 32)[0][:want]
        parts = [inst[offsets[c]:offsets[c + 1]] for c in keep]
        offsets = np.concatenate([[0], np.cumsum([len(x) for x in parts])]).astype(np.uint32)
        inst = np.concatenate(parts).astype(np.uint32)
        budget = 1024
    elif name.startswith("table1-"):
        return make_table1_config(int(name.split("-")[1]), n_cand=2000 if n_cand is None else n_cand,
                                  n_req=17_000 if n_req is None else n_req)
    else:
        raise ValueError(f"unknown configuration {name!r}; choose from {CONFIG_NAMES} or table1-1..6")
    offsets, inst = _head(offsets, inst, n_cand)
    return {"name": name, "profile": prof, "classes": classes, "traces": traces,
            "offsets": offsets, "inst": inst, "budget": budget}

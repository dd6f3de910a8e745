"""The five benchmark configurations as seeded synthetic inputs.

make_config(name, ...) returns a dict with keys
  profile, classes, traces (list of request arrays), offsets, inst, budget, name
`n_cand` / `n_req` shrink a configuration for tests (first n_cand candidates of the
seeded set, first n_req requests of each trace); None keeps the full size.
"""
import numpy as np
from .formats import make_classes
from .profiles import profile_tiny, profile_node, profile_multimodel
from .traces import make_trace
from .candidates import enumerate_tiny, enumerate_node, sample_candidates

CONFIG_NAMES = ("tiny", "node", "multimodel", "bursty", "scale")

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
    else:
        raise ValueError(f"unknown configuration {name!r}; choose from {CONFIG_NAMES}")
    offsets, inst = _head(offsets, inst, n_cand)
    return {"name": name, "profile": prof, "classes": classes, "traces": traces,
            "offsets": offsets, "inst": inst, "budget": budget}

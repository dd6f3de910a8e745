"""Load the hand-worked timelines under tests/golden/ into the binary input layouts."""
import glob
import json
import os

import numpy as np

import gen

_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _custom_profile(spec):
    steps = list(spec["steps"])
    table = np.full((1, 1, gen.WMAX), steps[-1], dtype=np.int32)
    table[0, 0, : len(steps)] = steps
    return {"n_models": 1, "n_strategies": 1, "wmax": gen.WMAX,
            "devices": np.array([1], dtype=np.int32), "min_devices": np.array([1], dtype=np.int32),
            "prefill_base_us": np.array([[spec["prefill_base_us"]]], dtype=np.int32),
            "prefill_q16": np.array([[spec["prefill_q16"]]], dtype=np.int32),
            "step_us": table}


def load_case(path):
    with open(path) as f:
        raw = json.load(f)
    prof = gen.profile_tiny() if raw["profile"] == "tiny" else _custom_profile(raw["profile"])
    classes = gen.make_classes([tuple(row) for row in raw["classes"]])
    offsets, inst = gen.candidates_from_lists([[tuple(i) for i in raw["instances"]]])
    trace = np.zeros(len(raw["requests"]), dtype=gen.REQUEST_DTYPE)
    for k, (a, i, o, c, m) in enumerate(raw["requests"]):
        trace[k] = (a, i, o, c, m)
    runs = [(raw["flags"], raw["expect"])]
    if "expect_flags0" in raw:
        runs.append((0, raw["expect_flags0"]))
    if "expect_maxgap" in raw:                 # TBT term of the hit test on the largest token gap
        runs.append((4, raw["expect_maxgap"]))
    if "expect_frozen" in raw:                 # the engine that fixes the decode speed at admission
        runs.append((2, raw["expect_frozen"]))
    return {"name": os.path.basename(path), "profile": prof, "classes": classes,
            "offsets": offsets, "inst": inst, "trace": trace, "budget": 8, "runs": runs}


def all_cases():
    return [load_case(p) for p in sorted(glob.glob(os.path.join(_DIR, "*.json")))]


SCALAR_KEYS = ("n_counted", "n_served", "n_hit", "n_rejected", "n_cascade", "sum_ttft_us",
               "max_ttft_us", "sum_e2e_us", "max_e2e_us", "makespan_us", "tokens_out", "attempts")


def check_against_expect(result, dumps, expect):
    """result: one record; dumps: dict of per-request arrays for that candidate."""
    assert int(result["status"]) == 0
    for key in SCALAR_KEYS:
        assert int(result[key]) == expect[key], (key, int(result[key]), expect[key])
    assert list(map(int, result["hit_by_class"])) == expect["hit_by_class"], ("hit_by_class", result["hit_by_class"])
    assert list(map(int, dumps["finish_us"])) == expect["finish_us"]
    assert list(map(int, dumps["first_us"])) == expect["first_us"]
    assert list(map(int, dumps["inst"])) == expect["inst"]

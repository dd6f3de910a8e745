"""Are the oracle's pins sharp?  Each case plants one plausible mistake in a COPY of the oracle's
source (a dropped term, an off-by-one, a swapped comparison, a wrong table index), builds it on the
CPU, and requires that at least one pin fails for the mutant.  The unmodified copy must pass all of
them.  Nothing here touches the CUDA path."""
import importlib.util
import os
import shutil

import numpy as np
import pytest

import gen
import test_oracle_pins as pins
from golden_cases import all_cases

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MUTANTS = [
    ("prefill rounding term dropped", "* in_tokens + 32768u) >> 16", "* in_tokens + 0u) >> 16"),
    ("predicted finish counts one token too many", "fin = first + (S - 1) * sB;", "fin = first + S * sB;"),
    ("worst-case step taken at the current level", "int64_t sB = in->step[in->B - 1];",
     "int64_t sB = in->step[in->w > 0 ? in->w - 1 : 0];"),
    ("next free time one step early", "t0 = in->T + (min_fin(in) - in->K) *", "t0 = in->T + (min_fin(in) - in->K - 1) *"),
    ("clock jump overshoots when the gap is a whole number of steps", "int64_t need = (t - in->T + s - 1) / s;",
     "int64_t need = (t - in->T + s) / s;"),
    ("ties go to the higher index", "(tier == best_tier && first < best_first)", "(tier == best_tier && first <= best_first)"),
    ("free slot not preferred", "!have || tier < best_tier || (tier == best_tier && first < best_first)",
     "!have || first < best_first"),
    ("TBT budget counts one gap too many", "span <= (int64_t)(S - 1) * k->tbt_us", "span <= (int64_t)S * k->tbt_us"),
    ("idle instance does not start at once", "if (!drain && in->w == 0 && in->T < t) in->T = t;", ""),
    ("completion index one step late", "sl->fin_idx = in->K + S - 1;", "sl->fin_idx = in->K + S;"),
    ("decode step taken one level too low", "int64_t s = in->step[in->w - 1];", "int64_t s = in->step[in->w > 1 ? in->w - 2 : 0];"),
    ("wait overshoots by a microsecond", "now = best_t0;  ", "now = best_t0 + 1;"),
    ("class mask inverted", "if (has_mask && !((class_mask >> q->cls) & 1u)) continue;",
     "if (has_mask && ((class_mask >> q->cls) & 1u)) continue;"),
    ("ranking prefers higher mean latency", "if (l != r) return l < r;", "if (l != r) return l > r;"),
    ("ranking prefers fewer hits", "return x->n_hit > y->n_hit;", "return x->n_hit < y->n_hit;"),
    ("latency weight is beta instead of 1 - beta", "double c = (1.0 - p->beta) * phil;", "double c = p->beta * phil;"),
    ("histogram half-octave bit taken one position too low", "uint32_t h = (uint32_t)((t >> (e - 1)) & 1);",
     "uint32_t h = (uint32_t)((t >> (e - 2)) & 1);"),
    ("histogram counts rejected requests too", "if (first[q] >= 0) out[c * 64 + orc_ttft_bin(first[q] - reqs[q].arrival_us)]++;",
     "if (first[q] >= -1) out[c * 64 + orc_ttft_bin(first[q] - reqs[q].arrival_us)]++;"),
    ("percentile rank rounded down", "uint64_t target = ((uint64_t)permille * total + 999) / 1000;",
     "uint64_t target = ((uint64_t)permille * total) / 1000;"),
    ("percentile reports the lower bin edge", "return ((int64_t)1 << e) + (int64_t)(h + 1) * ((int64_t)1 << (e - 1)) - 1;",
     "return ((int64_t)1 << e) + (int64_t)h * ((int64_t)1 << (e - 1));"),
    ("frozen engine: slot freed one microsecond late", "if (f->busy[j] && f->until[j] <= clock) f->busy[j] = 0;",
     "if (f->busy[j] && f->until[j] < clock) f->busy[j] = 0;"),
    ("frozen engine: speed of one level too low", "int64_t speed = f->step[running];",
     "int64_t speed = f->step[running > 0 ? running - 1 : 0];"),
    ("frozen engine: wait overshoots", "int64_t start = tier_i == 0 ? clock : earliest;",
     "int64_t start = tier_i == 0 ? clock : earliest + 1;"),
    ("frozen engine: finish counts one token too many", "int64_t t_end = first_tok + (len - 1) * speed;",
     "int64_t t_end = first_tok + len * speed;"),
    ("frozen engine: optimistic estimate uses the current level", "tier_i == 0) s_pred = f->step[running];",
     "tier_i == 0) s_pred = f->step[running > 0 ? running - 1 : 0];"),
    ("largest gap forgets the stall before the step", "int64_t gap = in->T + s - sl->last_tok;", "int64_t gap = s;"),
    ("largest gap is not kept across jumps", "if (gap > sl->max_gap) sl->max_gap = gap;", "sl->max_gap = gap;"),
    ("largest gap of a new request starts at the boundary", "sl->last_tok = in->T; sl->max_gap = 0;",
     "sl->last_tok = in->T - prefill_us(in, q->in_tokens); sl->max_gap = 0;"),
    ("queued request takes the level of its arrival time", "if (x != j && f->until[x] > pick_start) still++;",
     "if (x != j && f->until[x] > clock) still++;"),
    ("queued request starts at its arrival", "int64_t q_first = pick_start + f->pre_base", "int64_t q_first = clock + f->pre_base"),
    ("queued request: finish counts one token too many", "int64_t q_end = q_first + (len - 1) * q_speed;",
     "int64_t q_end = q_first + len * q_speed;"),
    ("queued request takes the last slot to free", "if (j == f->B || f->until[x] < f->until[j]) j = x; /* the slot that frees first */",
     "if (j == f->B || f->until[x] > f->until[j]) j = x;"),
    ("hits booked under the class below", "r->hit_by_class[cls < 7 ? cls : 7]++;",
     "r->hit_by_class[cls == 0 ? 0 : (cls < 8 ? cls - 1 : 7)]++;"),
    ("last class bin starts one class early", "r->hit_by_class[cls < 7 ? cls : 7]++;", "r->hit_by_class[cls < 6 ? cls : 7]++;"),
    ("classes above 7 wrap around instead of sharing the last bin", "r->hit_by_class[cls < 7 ? cls : 7]++;",
     "r->hit_by_class[cls & 7]++;"),
    ("prefill does not stall the running batch", "in->T += prefill_us(in, q->in_tokens);\n                if (S == 1) {",
     "int64_t t_keep = in->T; in->T += prefill_us(in, q->in_tokens);\n                if (S == 1) {"),
]


def load_variant(tmp_path, tag, old=None, new=None):
    d = tmp_path / tag
    d.mkdir()
    for name in ("binding.py", "maaso_oracle.c"):
        shutil.copy(os.path.join(ROOT, "oracle", name), d / name)
    if old is not None:
        src = (d / "maaso_oracle.c").read_text()
        assert src.count(old) == 1, f"mutation target not unique or missing: {old!r}"
        (d / "maaso_oracle.c").write_text(src.replace(old, new))
    spec = importlib.util.spec_from_file_location(f"oracle_variant_{tag}", d / "binding.py")
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build(force=True)
    return mod


def run_pins(mod):
    """Run a compact selection of the pins against `mod`; returns the names of those that fail."""
    failed = []

    def attempt(name, fn, *args):
        try:
            fn(mod, *args)
        except AssertionError:
            failed.append(name)

    for case in all_cases():
        attempt("hand:" + case["name"], pins.test_hand_timelines, case)
    attempt("lindley", pins.test_single_server_closed_form)
    attempt("no contention", pins.test_no_contention_closed_form)
    for seed in (0, 3, 4, 7):
        attempt(f"token by token {seed}", pins.test_against_token_by_token, seed)
    attempt("invariants", pins.test_invariants_on_tiny_config)
    attempt("no cascade", pins.test_no_cascade_without_prefill, 0)
    attempt("mask algebra", pins.test_mask_algebra)
    attempt("ranking", pins.test_topk_brute_force)
    attempt("score", pins.test_score_worked_values)
    for seed in (0, 1, 2, 3):
        attempt(f"frozen token lists {seed}", pins.test_frozen_engine_against_token_lists, seed)
    attempt("frozen levels", pins.test_frozen_engine_levels_recomputed_from_the_dumps)
    attempt("frozen cap one", pins.test_frozen_engine_equals_default_engine_for_one_instance_with_cap_one)
    for seed in (0, 1, 2, 3):
        attempt(f"largest gap {seed}", pins.test_maxgap_against_token_timestamps, seed)
    attempt("largest gap vs mean", pins.test_maxgap_only_changes_the_hit_test)
    for seed in (0, 1, 2, 3):
        attempt(f"instance queues {seed}", pins.test_instance_queues_against_token_lists, seed)
    attempt("instance queues structure", pins.test_instance_queues_structure_from_the_dumps)
    attempt("instance queues, one server", pins.test_instance_queues_single_server_is_the_lindley_recursion)
    attempt("histogram edges", pins.test_ttft_histogram_bin_edges)
    attempt("histogram counts", pins.test_ttft_histogram_counts_served_requests_only)
    attempt("percentiles", pins.test_ttft_percentiles_by_hand)
    return failed


def test_unmodified_copy_passes_every_pin(tmp_path):
    assert run_pins(load_variant(tmp_path, "clean")) == []


@pytest.mark.parametrize("what,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, what, old, new):
    if what == "prefill does not stall the running batch":
        # second half of the mutation: the first token is still stamped, but the clock is put back
        mod = load_variant(tmp_path, "m", old, new)
        src = (tmp_path / "m" / "maaso_oracle.c").read_text()
        tgt = "sl->cls = q->cls;\n                    in->w++;"
        assert src.count(tgt) == 1
        (tmp_path / "m" / "maaso_oracle.c").write_text(src.replace(tgt, tgt + "\n                    if (in->w > 1) in->T = t_keep;"))
        mod.build(force=True)
        mod._lib = None
    else:
        mod = load_variant(tmp_path, "m", old, new)
    failed = run_pins(mod)
    assert failed, f"no pin noticed: {what}"

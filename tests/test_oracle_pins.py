"""Pins for the CPU oracle: things fixed by the paper's rules and by mathematics, none of
them produced by the oracle itself."""
import numpy as np
import pytest

import gen
from golden_cases import all_cases, check_against_expect, SCALAR_KEYS
from stepwise_sim import simulate, simulate_frozen

NONE3 = [(None, None, None)]


def one_instance_profile(step1=9150, steps=None, base=2000, q16=7864):
    table = np.full((1, 1, gen.WMAX), step1, dtype=np.int32)
    if steps is not None:
        table[0, 0, : len(steps)] = steps
        table[0, 0, len(steps):] = steps[-1]
    return {"n_models": 1, "n_strategies": 1, "wmax": gen.WMAX,
            "devices": np.array([1], dtype=np.int32), "min_devices": np.array([1], dtype=np.int32),
            "prefill_base_us": np.array([[base]], dtype=np.int32),
            "prefill_q16": np.array([[q16]], dtype=np.int32), "step_us": table}


def run_one(oracle, profile, trace, classes, instances, budget=128, mask=None, flags=0):
    offsets, inst = gen.candidates_from_lists([instances])
    cm = None if mask is None else np.array([mask], dtype=np.uint32)
    res, dumps = oracle.eval_placements(profile, trace, classes, offsets, inst, budget, cm, flags,
                                        dump_idx=[0])
    return res[0], {k: v[0] for k, v in dumps.items()}


# ---- P1: hand-worked timelines -------------------------------------------------------------
@pytest.mark.parametrize("case", all_cases(), ids=lambda c: c["name"])
def test_hand_timelines(oracle_mod, case):
    for flags, expect in case["runs"]:
        res, dumps = oracle_mod.eval_placements(case["profile"], case["trace"], case["classes"],
                                                case["offsets"], case["inst"], case["budget"],
                                                None, flags, dump_idx=[0])
        check_against_expect(res[0], {k: v[0] for k, v in dumps.items()}, expect)


# ---- P2: B = 1, one instance, no SLO limits = single-server FIFO (Lindley recursion) --------
def test_single_server_closed_form(oracle_mod):
    prof = gen.profile_tiny()
    trace = gen.make_trace(400, 3.0, 11)
    classes = gen.make_classes(NONE3 * 3)
    res, d = run_one(oracle_mod, prof, trace, classes, [(0, 1, 1)])
    base, q16, s1 = int(prof["prefill_base_us"][0, 1]), int(prof["prefill_q16"][0, 1]), int(prof["step_us"][0, 1, 0])
    prev = 0
    fin, first = [], []
    for q in trace:
        start = max(int(q["arrival_us"]), prev)
        f1 = start + base + ((q16 * int(q["in_tokens"]) + 32768) >> 16)
        prev = f1 + (int(q["out_tokens"]) - 1) * s1
        first.append(f1)
        fin.append(prev)
    assert d["finish_us"].tolist() == fin
    assert d["first_us"].tolist() == first
    assert int(res["n_served"]) == 400 and int(res["n_hit"]) == 400 and int(res["n_rejected"]) == 0
    arr = trace["arrival_us"].astype(np.int64)
    assert int(res["sum_e2e_us"]) == int((np.array(fin) - arr).sum())
    assert int(res["sum_ttft_us"]) == int((np.array(first) - arr).sum())
    assert int(res["max_ttft_us"]) == int((np.array(first) - arr).max())
    assert int(res["makespan_us"]) == fin[-1]
    assert int(res["tokens_out"]) == int(trace["out_tokens"].astype(np.int64).sum())


# ---- P3: no contention: every request alone in the system ---------------------------------
def test_no_contention_closed_form(oracle_mod):
    prof = gen.profile_tiny()
    trace = gen.make_trace(60, 1.0, 5)
    trace["arrival_us"] = np.arange(60, dtype=np.int64) * 400_000_000  # 400 s apart
    classes = gen.make_classes(NONE3 * 3)
    # instance 2 (tp4) has the smallest prefill; instances 0 and 1 are identical tp2 rows
    res, d = run_one(oracle_mod, prof, trace, classes, [(0, 1, 4), (0, 1, 8), (0, 2, 2), (0, 0, 16)])
    base, q16, s1 = int(prof["prefill_base_us"][0, 2]), int(prof["prefill_q16"][0, 2]), int(prof["step_us"][0, 2, 0])
    for k, q in enumerate(trace):
        f1 = int(q["arrival_us"]) + base + ((q16 * int(q["in_tokens"]) + 32768) >> 16)
        assert int(d["first_us"][k]) == f1
        assert int(d["finish_us"][k]) == f1 + (int(q["out_tokens"]) - 1) * s1
        assert int(d["inst"][k]) == 2
    # ties go to the lowest index
    res, d = run_one(oracle_mod, prof, trace, classes, [(0, 1, 4), (0, 1, 8)])
    assert set(d["inst"].tolist()) == {0}


# ---- P8: token-by-token re-formulation on tiny inputs -------------------------------------
@pytest.mark.parametrize("seed", range(12))
def test_against_token_by_token(oracle_mod, seed):
    rng = np.random.default_rng(1000 + seed)
    if seed % 3 == 2:
        prof = gen.profile_multimodel(seed)
        model_mix = (0.5, 0.3, 0.2)
    else:
        prof = gen.profile_node(seed)
        model_mix = (1.0,)
    M, S = prof["n_models"], prof["n_strategies"]
    trace = gen.make_trace(120, float(rng.choice([4.0, 20.0, 80.0])), seed, cv=float(rng.choice([1.0, 3.0])),
                           model_mix=model_mix, out_dist=("lognormal", 3.0, 1.0, 1, 300),
                           doc_out=(200, 400))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None),
                                (None, None, 8_000_000)])
    n_inst = int(rng.integers(1, 7))
    instances = []
    for _ in range(n_inst):
        m = int(rng.integers(M))
        ok = np.nonzero(prof["devices"] >= prof["min_devices"][m])[0]
        instances.append((m, int(rng.choice(ok)), int(rng.choice([1, 2, 3, 4, 8, 16, 64]))))
    mask = None if seed % 4 else 0b101
    flags = seed % 2
    res, d = run_one(oracle_mod, prof, trace, classes, instances, mask=mask, flags=flags)
    ref = simulate(prof, trace, classes, instances, class_mask=mask, optimistic=bool(flags))
    for key in SCALAR_KEYS:
        assert int(res[key]) == ref[key], key
    assert d["finish_us"].tolist() == ref["finish_us"]
    assert d["first_us"].tolist() == ref["first_us"]
    assert d["inst"].tolist() == ref["inst"]


# ---- the engine that fixes the decode speed at admission (flags = 2) -------------------------
FROZEN = 2


def _random_small_case(seed):
    rng = np.random.default_rng(2000 + seed)
    if seed % 3 == 2:
        prof, model_mix = gen.profile_multimodel(seed), (0.5, 0.3, 0.2)
    else:
        prof, model_mix = gen.profile_node(seed), (1.0,)
    trace = gen.make_trace(150, float(rng.choice([4.0, 20.0, 80.0])), seed, cv=float(rng.choice([1.0, 3.0])),
                           model_mix=model_mix, out_dist=("lognormal", 3.0, 1.0, 1, 300), doc_out=(200, 400))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 8_000_000)])
    instances = []
    for _ in range(int(rng.integers(1, 7))):
        m = int(rng.integers(prof["n_models"]))
        ok = np.nonzero(prof["devices"] >= prof["min_devices"][m])[0]
        instances.append((m, int(rng.choice(ok)), int(rng.choice([1, 2, 3, 4, 8, 16, 64]))))
    return prof, trace, classes, instances


@pytest.mark.parametrize("seed", range(10))
def test_frozen_engine_against_token_lists(oracle_mod, seed):
    prof, trace, classes, instances = _random_small_case(seed)
    mask = None if seed % 4 else 0b110
    opt = seed % 2
    res, d = run_one(oracle_mod, prof, trace, classes, instances, mask=mask, flags=FROZEN | opt)
    ref = simulate_frozen(prof, trace, classes, instances, class_mask=mask, optimistic=bool(opt))
    for key in SCALAR_KEYS:
        assert int(res[key]) == ref[key], key
    assert d["finish_us"].tolist() == ref["finish_us"]
    assert d["first_us"].tolist() == ref["first_us"]
    assert d["inst"].tolist() == ref["inst"]


def test_frozen_engine_equals_default_engine_for_one_instance_with_cap_one(oracle_mod):
    """One instance with B = 1: nobody runs beside anybody, so there is no slowdown and no stall
    and both engines must give every request the same times (single-server FIFO) and the same
    record.  Only the number of distributor rounds may differ: the default engine's clock sits
    on a decode-step boundary, so it can see the slot free one round earlier.  Requests of one
    token are left out: they hold a slot during their prefill in this engine, none in the other."""
    for seed in range(6):
        prof, trace, classes, instances = _random_small_case(seed)
        trace["out_tokens"] = np.maximum(trace["out_tokens"], 2)
        trace["model"] = instances[0][0]
        instances = [(instances[0][0], instances[0][1], 1)]
        for opt in (0, 1):
            a, da = run_one(oracle_mod, prof, trace, classes, instances, flags=opt)
            b, db = run_one(oracle_mod, prof, trace, classes, instances, flags=FROZEN | opt)
            a, b = a.copy(), b.copy()
            a["attempts"] = b["attempts"] = 0
            assert a.tobytes() == b.tobytes()
            for key in da:
                assert (da[key] == db[key]).all()


def test_frozen_engine_levels_recomputed_from_the_dumps(oracle_mod):
    """From the per-request times alone: a request holds its slot from (first token - prefill) to
    its finish; at its admission the instance must have had a free slot, and its tokens must be
    exactly one table step of the level (running + 1) apart.  No request may miss its SLO."""
    cfg = gen.make_config("tiny", n_req=300)
    prof, tr = cfg["profile"], cfg["traces"][0]
    off, inst = cfg["offsets"], cfg["inst"]
    pick = np.arange(0, len(off) - 1, 9)
    for opt in (0, 1):
        res, d = oracle_mod.eval_placements(prof, tr, cfg["classes"], off, inst, cfg["budget"], flags=FROZEN | opt,
                                            dump_idx=pick)
        for row, c in enumerate(pick):
            words = inst[off[c]:off[c + 1]]
            assert int(res[c]["n_cascade"]) == 0 and int(res[c]["n_served"]) == int(res[c]["n_hit"])
            for i, word in enumerate(words):
                m, s, B = int(word & 15), int((word >> 4) & 255), int((word >> 12) & 255)
                mine = np.nonzero(d["inst"][row] == i)[0]
                spans = []
                for r in mine:
                    pre = int(prof["prefill_base_us"][m, s]) + ((int(prof["prefill_q16"][m, s]) * int(tr["in_tokens"][r]) + 32768) >> 16)
                    spans.append((int(d["first_us"][row][r]) - pre, int(d["finish_us"][row][r]), r))
                for (t_adm, t_fin, r) in spans:
                    running = sum(1 for (a, f, o) in spans if o != r and a <= t_adm < f and (a, o) < (t_adm, r))
                    assert running < B
                    S = int(tr["out_tokens"][r])
                    if S > 1:
                        assert t_fin - int(d["first_us"][row][r]) == (S - 1) * int(prof["step_us"][m, s, running])


def test_largest_gap_with_stalls_that_shrink_from_one_admission_to_the_next(oracle_mod):
    """Forty admissions in a row, each stalling the running batch a little less than the one before, none
    of them finished yet: every request's largest gap is the stall right after its own admission, so
    the hit counts step through the classes' limits.  Token timestamps of the step-by-step simulator."""
    prof = gen.make_config("tiny")["profile"]
    trace = gen.shrinking_prompts_trace(n_classes=24)
    classes = gen.make_classes([(None, 18_600 + 150 * c, None) for c in range(24)])   # a limit every 150 us
    for opt in (0, 1):
        res, d = run_one(oracle_mod, prof, trace, classes, [(0, 0, 64)], flags=MAXGAP | opt)
        ref = simulate(prof, trace, classes, [(0, 0, 64)], optimistic=bool(opt), maxgap=True)
        for key in SCALAR_KEYS:
            assert int(res[key]) == ref[key], key
        assert d["finish_us"].tolist() == ref["finish_us"]
        assert int(res["n_served"]) == 41 and 5 < int(res["n_hit"]) < 36
        mean_form, _ = run_one(oracle_mod, prof, trace, classes, [(0, 0, 64)], flags=opt)
        assert int(mean_form["n_hit"]) == 41


# ---- requests queue at their instance, not at the dispatcher (flag 8) --------------------------
QUEUES = 8


@pytest.mark.parametrize("seed", range(10))
def test_instance_queues_against_token_lists(oracle_mod, seed):
    prof, trace, classes, instances = _random_small_case(seed)
    mask = None if seed % 4 else 0b011
    opt = seed % 2
    res, d = run_one(oracle_mod, prof, trace, classes, instances, mask=mask, flags=QUEUES | opt)
    ref = simulate_frozen(prof, trace, classes, instances, class_mask=mask, optimistic=bool(opt), queues=True)
    for key in SCALAR_KEYS:
        assert int(res[key]) == ref[key], key
    assert d["finish_us"].tolist() == ref["finish_us"]
    assert d["first_us"].tolist() == ref["first_us"]
    assert d["inst"].tolist() == ref["inst"]


def test_instance_queues_single_server_is_the_lindley_recursion(oracle_mod):
    """One instance with one slot, no limits: a first-come-first-served single-server queue, whose
    departure times obey D_k = max(A_k, D_{k-1}) + service_k (textbook recursion); the service time
    is prefill + (S - 1) steps at level 1."""
    for seed in range(4):
        prof, trace, _, instances = _random_small_case(seed)
        m, s, _ = instances[0]
        trace["model"] = m
        classes = gen.make_classes([(None, None, None)] * 3)
        res, d = run_one(oracle_mod, prof, trace, classes, [(m, s, 1)], flags=QUEUES)
        step1 = int(prof["step_us"][m][s][0])
        base, q16 = int(prof["prefill_base_us"][m][s]), int(prof["prefill_q16"][m][s]) & 0xFFFFFFFF
        depart = 0
        for k in range(len(trace)):
            start = max(int(trace["arrival_us"][k]), depart)
            first = start + base + ((q16 * int(trace["in_tokens"][k]) + 32768) >> 16)
            depart = first + (int(trace["out_tokens"][k]) - 1) * step1
            assert int(d["first_us"][k]) == first and int(d["finish_us"][k]) == depart, (seed, k)
        assert int(res["n_served"]) == len(trace) and int(res["attempts"]) == len(trace)


def test_instance_queues_structure_from_the_dumps(oracle_mod):
    """From the per-request times alone: one distributor round per request; on every instance the
    requests start in arrival order (first come first served), never more than B hold a slot at once,
    and a request never starts before its arrival."""
    cfg = gen.make_config("tiny", n_req=300)
    prof, tr = cfg["profile"], cfg["traces"][0]
    off, inst = cfg["offsets"], cfg["inst"]
    pick = np.arange(0, len(off) - 1, 7)
    res, d = oracle_mod.eval_placements(prof, tr, cfg["classes"], off, inst, cfg["budget"], flags=QUEUES, dump_idx=pick)
    waited = 0
    for row, c in enumerate(pick):
        assert int(res[c]["attempts"]) == int(res[c]["n_counted"])
        for i, word in enumerate(inst[off[c]:off[c + 1]]):
            m, s, B = int(word & 15), int((word >> 4) & 255), int((word >> 12) & 255)
            mine = np.nonzero(d["inst"][row] == i)[0]
            starts, spans = [], []
            for r in mine:
                pre = int(prof["prefill_base_us"][m, s]) + ((int(prof["prefill_q16"][m, s]) * int(tr["in_tokens"][r]) + 32768) >> 16)
                t_adm = int(d["first_us"][row][r]) - pre
                assert t_adm >= int(tr["arrival_us"][r])
                waited += t_adm > int(tr["arrival_us"][r])
                starts.append(t_adm)
                spans.append((t_adm, int(d["finish_us"][row][r])))
            assert starts == sorted(starts)
            for (a, f) in spans:
                assert sum(1 for (a2, f2) in spans if a2 <= a < f2) <= B
    assert waited > 0


# ---- TBT term of the hit test on the largest token gap (flag 4) -------------------------------
MAXGAP = 4


@pytest.mark.parametrize("seed", range(8))
def test_maxgap_against_token_timestamps(oracle_mod, seed):
    """The token-by-token simulator keeps every token's timestamp; the largest difference between
    neighbours decides the TBT term.  Tight limits so that stalls by prefills matter."""
    prof, trace, classes, instances = _random_small_case(seed)
    classes = gen.make_classes([(500_000, 14_000, None), (2_000_000, 30_000, None), (None, 60_000, 8_000_000)])
    opt = seed % 2
    res, d = run_one(oracle_mod, prof, trace, classes, instances, flags=MAXGAP | opt)
    ref = simulate(prof, trace, classes, instances, optimistic=bool(opt), maxgap=True)
    for key in SCALAR_KEYS:
        assert int(res[key]) == ref[key], key
    assert d["finish_us"].tolist() == ref["finish_us"]
    res2, _ = run_one(oracle_mod, prof, trace, classes, instances, flags=MAXGAP | FROZEN | opt)
    ref2 = simulate_frozen(prof, trace, classes, instances, optimistic=bool(opt), maxgap=True)
    for key in SCALAR_KEYS:
        assert int(res2[key]) == ref2[key], key


def test_maxgap_only_changes_the_hit_test(oracle_mod):
    """The largest gap is at least the mean gap: hits can only go down, nothing else moves."""
    cfg = gen.make_config("tiny", n_req=400)
    classes = gen.make_classes([(500_000, 12_000, None), (2_000_000, 20_000, None), (None, None, 180_000_000)])
    a = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], classes, cfg["offsets"], cfg["inst"], cfg["budget"], flags=1)
    b = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], classes, cfg["offsets"], cfg["inst"], cfg["budget"],
                                   flags=1 | MAXGAP)
    assert (b["n_hit"] <= a["n_hit"]).all() and int((a["n_hit"] - b["n_hit"]).sum()) > 0
    for key in ("n_counted", "n_served", "n_rejected", "sum_ttft_us", "sum_e2e_us", "makespan_us", "tokens_out",
                "checksum", "attempts"):
        assert (a[key] == b[key]).all(), key
    assert (b["n_cascade"] == b["n_served"] - b["n_hit"]).all()


# ---- P4: invariants -----------------------------------------------------------------------
def test_invariants_on_tiny_config(oracle_mod):
    cfg = gen.make_config("tiny")
    n = len(cfg["traces"][0])
    idx = np.arange(0, 143, 7, dtype=np.uint32)
    res, dumps = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"],
                                            cfg["offsets"], cfg["inst"], cfg["budget"], dump_idx=idx)
    assert (res["status"] == 0).all()          # includes the oracle's own invariant flag
    assert (res["n_counted"] == n).all()
    assert (res["n_served"] + res["n_rejected"] == n).all()      # conservation
    assert (res["n_cascade"] == res["n_served"] - res["n_hit"]).all()
    assert (res["hit_by_class"].sum(axis=1) == res["n_hit"]).all()
    arr = cfg["traces"][0]["arrival_us"].astype(np.int64)
    S = cfg["traces"][0]["out_tokens"].astype(np.int64)
    for row, c in enumerate(idx):
        fin, first, where = dumps["finish_us"][row], dumps["first_us"][row], dumps["inst"][row]
        served = fin >= 0
        assert served.sum() == res["n_served"][c]
        assert ((fin == -1) == (where == -1)).all()
        assert (first[served] >= arr[served]).all() and (fin[served] >= first[served]).all()
        assert int((first[served] - arr[served]).sum()) == int(res["sum_ttft_us"][c])
        assert int((fin[served] - arr[served]).sum()) == int(res["sum_e2e_us"][c])
        assert int(S[served].sum()) == int(res["tokens_out"][c])
        # batch cap: at any first-token instant, running requests on that instance <= B
        lo, hi = int(cfg["offsets"][c]), int(cfg["offsets"][c + 1])
        caps = ((cfg["inst"][lo:hi] >> 12) & 0xFF).astype(np.int64)
        for i, cap in enumerate(caps):
            on = served & (where == i) & (S > 1)
            f1, f2 = first[on], fin[on]
            for t in f1:
                assert ((f1 <= t) & (f2 > t)).sum() <= cap
        # first tokens on one instance are strictly ordered by request index (FIFO dispatcher)
        for i in range(hi - lo):
            on = served & (where == i)
            assert (np.diff(first[on]) > 0).all()


# ---- P6: worst-case prediction + zero prefill + monotone table => no cascaded misses --------
@pytest.mark.parametrize("seed", range(4))
def test_no_cascade_without_prefill(oracle_mod, seed):
    prof = gen.profile_node(seed)
    prof["prefill_base_us"][:] = 0
    prof["prefill_q16"][:] = 0
    prof["step_us"][:] = np.maximum.accumulate(prof["step_us"], axis=2)
    trace = gen.make_trace(1500, 40.0, seed, cv=2.0, out_dist=("lognormal", 4.0, 1.0, 1, 600),
                           doc_out=(500, 900))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None),
                                (None, None, 20_000_000)])
    offsets, inst = gen.enumerate_node(prof["devices"], 4, batches=(2, 16, 64))
    res = oracle_mod.eval_placements(prof, trace, classes, offsets, inst, 8)
    assert (res["status"] == 0).all()
    assert res["n_served"].sum() > 0 and res["n_rejected"].sum() > 0
    assert (res["n_cascade"] == 0).all()
    # the optimistic estimate must show cascades somewhere (what overflow protection prevents)
    res2 = oracle_mod.eval_placements(prof, trace, classes, offsets, inst, 8, flags=oracle_mod.FLAG_PRED_OPTIMISTIC)
    assert res2["n_cascade"].sum() > 0


# ---- P7: mask algebra ---------------------------------------------------------------------
def test_mask_algebra(oracle_mod):
    cfg = gen.make_config("tiny")
    tr = cfg["traces"][0]
    off, inst = cfg["offsets"], cfg["inst"]
    C = len(off) - 1
    a = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 4, np.full(C, 0b011, np.uint32))
    b = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 4, np.full(C, 0b100, np.uint32))
    full = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 4, np.full(C, 0b111, np.uint32))
    nomask = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 4)
    assert (a["n_counted"] + b["n_counted"] == len(tr)).all()
    assert (a["n_counted"] == (tr["cls"] < 2).sum()).all()
    assert full.tobytes() == nomask.tobytes()
    # a masked run equals a run on the filtered trace except for request numbering (checksum)
    sub = tr[tr["cls"] == 2]
    c = oracle_mod.eval_placements(cfg["profile"], sub, cfg["classes"], off, inst, 4)
    for key in SCALAR_KEYS:
        assert (b[key] == c[key]).all(), key


# ---- constraints (c), (d) and malformed instances -------------------------------------------
def test_candidate_validation(oracle_mod):
    prof = gen.profile_multimodel(0)
    tr = gen.make_trace(50, 8.0, 0, model_mix=(0.6, 0.3, 0.1))
    classes = gen.make_classes(NONE3 * 3)
    lists = [
        [(0, 6, 4), (0, 6, 4)],          # 16 devices > budget 8
        [(2, 0, 4)],                      # 70B-like on one device
        [(0, 0, 4)] * 129,                # too many
        [(3, 0, 4)],                      # unknown model
        [(0, 10, 4)],                     # unknown strategy
        [(0, 0, 0)],                      # batch cap 0
        [(0, 0, 65)],                     # batch cap too large
        [(0, 0, 4), (2, 3, 8)],           # fine
        [],                               # empty placement: everything is rejected
    ]
    off, inst = gen.candidates_from_lists(lists)
    inst = inst.copy()
    res = oracle_mod.eval_placements(prof, tr, classes, off, inst, 8)
    E = oracle_mod.STATUS
    assert res["status"].tolist() == [E["EBUDGET"], E["EMEMFIT"], E["ETOOMANY"], E["EBADINST"],
                                      E["EBADINST"], E["EBADINST"], E["EBADINST"], 0, 0]
    bad = res[res["status"] != 0]
    for key in SCALAR_KEYS:
        assert (bad[key] == 0).all()
    assert int(res["n_rejected"][8]) == 50 and int(res["n_served"][8]) == 0
    inst2 = inst.copy()
    inst2[off[7]] |= 1 << 20                  # reserved bit set
    res2 = oracle_mod.eval_placements(prof, tr, classes, off, inst2, 8)
    assert int(res2["status"][7]) == E["EBADINST"]


# ---- batch composition cannot matter ------------------------------------------------------
def test_alone_in_batch_duplicated(oracle_mod):
    cfg = gen.make_config("tiny")
    tr, off, inst = cfg["traces"][0], cfg["offsets"], cfg["inst"]
    full = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 4)
    for c in (0, 57, 142):
        words = inst[off[c]:off[c + 1]]
        o2 = np.array([0, len(words), 2 * len(words)], dtype=np.uint32)
        two = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], o2, np.concatenate([words, words]), 4)
        assert two[0].tobytes() == full[c].tobytes() and two[1].tobytes() == full[c].tobytes()
    par = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], off, inst, 4, workers=2)
    assert par.tobytes() == full.tobytes()


# ---- qualitative claims of the paper's batch-size study (Sec. III-B) ------------------------
def test_batch_cap_tradeoff(oracle_mod):
    prof = gen.profile_tiny()
    trace = gen.make_trace(300, 6.0, 3, out_dist=("lognormal", 4.0, 0.5, 2, 400), doc_class=None)
    classes = gen.make_classes(NONE3 * 3)
    r4, d4 = run_one(oracle_mod, prof, trace, classes, [(0, 0, 4)])
    r8, d8 = run_one(oracle_mod, prof, trace, classes, [(0, 0, 8)])
    assert int(r4["n_served"]) == int(r8["n_served"]) == 300
    # a larger cap relieves queuing ...
    assert int(r8["sum_ttft_us"]) < int(r4["sum_ttft_us"])
    # ... at the price of slower decoding per request
    span4 = (d4["finish_us"] - d4["first_us"]).sum()
    span8 = (d8["finish_us"] - d8["first_us"]).sum()
    assert span4 < span8


# ---- P5: ranking by brute force with exact rationals ----------------------------------------
def test_topk_brute_force(oracle_mod):
    from fractions import Fraction
    cfg = gen.make_config("tiny")
    res = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"],
                                     cfg["inst"], cfg["budget"])
    res = res.copy()
    res["status"][5] = 1           # invalid candidates go last
    res["n_served"][9] = 0         # nothing served ranks after anything served, same hits
    res["n_hit"][9] = res["n_hit"][10]
    res["n_hit"][20] = res["n_hit"][21]  # force a tie on hits, decided by mean TTFT

    def key(i):
        r = res[i]
        if r["status"] != 0:
            return (1, 0, 0, 0, i)
        served = int(r["n_served"])
        mean = Fraction(int(r["sum_ttft_us"]), served) if served else Fraction(0)
        return (0, -int(r["n_hit"]), 0 if served else 1, mean, i)

    want = sorted(range(len(res)), key=key)
    for k in (1, 7, 64, 143, 500):
        got = oracle_mod.topk(res, k).tolist()
        assert got == want[:k]


def test_topk_exact_fraction_compare(oracle_mod):
    """Means that differ by less than a double can resolve must still be ordered exactly."""
    res = np.zeros(3, dtype=gen.RESULT_DTYPE)
    big = (1 << 62) - 57
    res["n_hit"] = 5
    res["n_served"] = [1_000_003, 1_000_003, 1_000_002]
    res["sum_ttft_us"] = [big, big - 1, big - 1_000_000_000_000]
    # mean1 < mean0 by 1e-6/1e6; candidate 2: (big - 1e12)/1000002 vs big/1000003
    from fractions import Fraction
    want = sorted(range(3), key=lambda i: (Fraction(int(res["sum_ttft_us"][i]), int(res["n_served"][i])), i))
    assert oracle_mod.topk(res, 3).tolist() == want


# ---- generators -----------------------------------------------------------------------------
def test_generator_counts_and_layout():
    off, inst = gen.enumerate_tiny()
    assert len(off) - 1 == 143
    prof = gen.profile_node(0)
    off, inst = gen.enumerate_node(prof["devices"], 8)
    assert len(off) - 1 == 10864
    tr = gen.make_trace(1000, 16.0, 0)
    assert tr.dtype.itemsize == 16 and (np.diff(tr["arrival_us"]) >= 0).all()
    assert tr["out_tokens"].min() >= 1
    doc = tr["cls"] == 2
    assert tr["out_tokens"][doc].min() >= 2048 and tr["out_tokens"][~doc].max() <= 2048
    pm = gen.profile_multimodel(0)
    off, inst = gen.sample_candidates(2000, 1, 32, pm)
    m, s, b = gen.unpack_inst(inst)
    cand = np.repeat(np.arange(2000), np.diff(off.astype(np.int64)))
    used = np.bincount(cand, weights=pm["devices"][s], minlength=2000)
    assert used.max() <= 32 and (np.diff(off.astype(np.int64)) >= 1).all()
    assert (pm["devices"][s] >= pm["min_devices"][m]).all()
    a = gen.make_trace(100, 8.0, 7)
    b2 = gen.make_trace(100, 8.0, 7)
    assert a.tobytes() == b2.tobytes()


# ---- composite serving score (Sec. IV-D) ----------------------------------------------------
def _rec(**kw):
    r = np.zeros(1, dtype=gen.RESULT_DTYPE)
    for k, v in kw.items():
        r[k] = v
    return r


def test_score_worked_values(oracle_mod):
    # 50 of 100 requests hit; 1000 tokens in 1 s -> 1000 tok/s of gamma_T = 2000 -> 0.5;
    # mean TTFT 0.5 s of gamma_L = 2 s -> 0.75;  4*0.5 + 0.3*0.5 + 0.7*0.75 = 2.675
    r = _rec(n_counted=100, n_served=80, n_hit=50, tokens_out=1000, makespan_us=1_000_000,
             sum_ttft_us=80 * 500_000)
    assert oracle_mod.score(r, 4.0, 0.3, 2000.0, 2.0)[0] == pytest.approx(2.675, abs=1e-12)
    # throughput above the threshold is capped, latency beyond the threshold earns nothing
    r = _rec(n_counted=10, n_served=10, n_hit=10, tokens_out=10_000_000, makespan_us=1_000_000,
             sum_ttft_us=10 * 9_000_000)
    assert oracle_mod.score(r, 10.0, 0.25, 2000.0, 2.0)[0] == pytest.approx(10.0 + 0.25, abs=1e-12)
    # nothing served: only the (zero) SLO term; invalid: -1; nothing counted: 0
    assert oracle_mod.score(_rec(n_counted=7), 4.0, 0.3, 1.0, 1.0)[0] == 0.0
    assert oracle_mod.score(_rec(status=2), 4.0, 0.3, 1.0, 1.0)[0] == -1.0
    assert oracle_mod.score(_rec(), 4.0, 0.3, 1.0, 1.0)[0] == 0.0


def test_score_properties_and_ranking(oracle_mod):
    cfg = gen.make_config("tiny")
    res = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"],
                                     cfg["inst"], cfg["budget"])
    a4 = oracle_mod.score(res, 4.0, 0.3, 500.0, 5.0)
    a10 = oracle_mod.score(res, 10.0, 0.3, 500.0, 5.0)
    ratio = res["n_hit"] / res["n_counted"]
    # alpha only weighs the SLO term (MaaSO vs MaaSO*: alpha = 4 vs 10)
    assert np.allclose(a10 - a4, 6.0 * ratio, atol=1e-12)
    assert (a4 >= 4.0 * ratio - 1e-12).all() and (a4 <= 4.0 * ratio + 1.0 + 1e-12).all()
    # beta = 1: throughput only; beta = 0: latency only
    t_only = oracle_mod.score(res, 0.0, 1.0, 500.0, 5.0)
    thr = np.where(res["n_served"] > 0, res["tokens_out"] / (res["makespan_us"] * 1e-6), 0.0)
    assert np.allclose(t_only, np.minimum(thr, 500.0) / 500.0, atol=1e-12)
    l_only = oracle_mod.score(res, 0.0, 0.0, 500.0, 5.0)
    lat = np.where(res["n_served"] > 0, res["sum_ttft_us"] / np.maximum(res["n_served"], 1) * 1e-6, 5.0)
    assert np.allclose(l_only, np.maximum(5.0 - lat, 0.0) / 5.0, atol=1e-12)
    # ranking by score: brute force
    s = a4.copy()
    s[3] = s[77]                 # a tie decided by the index
    s[5] = np.nan                # NaN goes last
    want = sorted(range(len(s)), key=lambda i: (np.isnan(s[i]), -s[i] if not np.isnan(s[i]) else 0.0, i))
    assert oracle_mod.topk_scores(s, 143).tolist() == want
    assert oracle_mod.topk_scores(s, 10).tolist() == want[:10]


# ---- Alg. 1: simulator-based instance configuration -------------------------------------------
def test_ins_deploy_worked_example(oracle_mod):
    """Requests 400 s apart on a one-model profile: one instance serves everything, a second one
    changes nothing, so the score does not improve, the model saturates and the search stops.
    Phi*[k] / I*[k] are indexed by the devices the stored placement occupies (Sec. IV-E: "solutions
    for all possible GPU allocations k"): the one-instance placement sits in slot 1, slot 0 stays
    empty, and with a one-device cluster the last slot, Phi*[|G_x|], is the one that is filled."""
    prof = gen.profile_tiny()
    tr = gen.make_trace(40, 1.0, 5, doc_class=None)
    tr["arrival_us"] = np.arange(40, dtype=np.int64) * 400_000_000
    classes = gen.make_classes(NONE3 * 3)
    phi, I = oracle_mod.ins_deploy(prof, tr, classes, 3, [(0, 4)], 4.0, 0.3, 1000.0, 10.0)
    # closed form of the score: every request is a hit, first token = arrival + prefill
    base, q16, s1 = int(prof["prefill_base_us"][0, 0]), int(prof["prefill_q16"][0, 0]), int(prof["step_us"][0, 0, 0])
    pre = base + ((q16 * tr["in_tokens"].astype(np.int64) + 32768) >> 16)
    fin = tr["arrival_us"] + pre + (tr["out_tokens"].astype(np.int64) - 1) * s1
    thr = tr["out_tokens"].astype(np.int64).sum() / (fin.max() * 1e-6)
    lat = pre.sum() / 40 * 1e-6
    want = 4.0 * 1.0 + 0.3 * min(thr, 1000.0) / 1000.0 + 0.7 * max(10.0 - lat, 0.0) / 10.0
    assert phi[1] == pytest.approx(want, rel=1e-12)
    assert phi[0] == 0.0 and phi[2] == 0.0 and phi[3] == 0.0
    assert I[1].tolist() == [int(gen.pack_inst(0, 0, 4))]
    assert len(I[0]) == 0 and len(I[2]) == 0 and len(I[3]) == 0
    phi1, I1 = oracle_mod.ins_deploy(prof, tr, classes, 1, [(0, 4)], 4.0, 0.3, 1000.0, 10.0)
    assert phi1[1] == phi[1] and phi1[0] == 0.0 and I1[1].tolist() == I[1].tolist()
    # a two-device strategy on three devices: one instance fits (slot 2), a second one would not
    phi2, I2 = oracle_mod.ins_deploy(prof, tr, classes, 3, [(1, 4)], 4.0, 0.3, 1000.0, 10.0)
    assert phi2[2] > 0.0 and phi2[0] == phi2[1] == phi2[3] == 0.0 and len(I2[2]) == 1


def test_ins_deploy_properties(oracle_mod):
    prof = gen.profile_multimodel(0)
    tr = gen.make_trace(1200, 25.0, 3, model_mix=(0.2, 0.7, 0.1))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    configs = [(0, 8), (1, 16), (3, 8), (3, 64), (6, 16)]
    gpus = 12
    phi, I = oracle_mod.ins_deploy(prof, tr, classes, gpus, configs, 4.0, 0.3, 2000.0, 5.0)
    assert (phi >= 0).all() and phi.max() > 0
    for k in range(gpus + 1):
        if len(I[k]) == 0:
            assert phi[k] == 0.0
            continue
        m, s, b = gen.unpack_inst(I[k])
        assert len(set(zip(s.tolist(), b.tolist()))) == 1 and (int(s[0]), int(b[0])) in configs  # one (P, B) per solution
        assert prof["devices"][s].sum() == k          # slot k holds a placement of exactly k devices
        assert (prof["devices"][s] >= prof["min_devices"][m]).all()
        # the stored score is the score of the stored placement
        off = np.array([0, len(I[k])], dtype=np.uint32)
        rec = oracle_mod.eval_placements(prof, tr, classes, off, I[k], gpus)
        assert oracle_mod.score(rec, 4.0, 0.3, 2000.0, 5.0)[0] == phi[k]
    # the first instance of every chain serves the model with the most requests (model 1 here)
    assert len(I[0]) == 0
    first = next(k for k in range(gpus + 1) if len(I[k]))
    assert int(gen.unpack_inst(I[first])[0][0]) == 1
    # a strategy that needs more devices than the sub-cluster has can never be deployed
    phi2, I2 = oracle_mod.ins_deploy(prof, tr, classes, 4, [(6, 16)], 4.0, 0.3, 2000.0, 5.0)
    assert (phi2 == 0).all() and all(len(x) == 0 for x in I2)
    # the SLO weight only rescales: with alpha = 10 (MaaSO*) no slot scores less than with alpha = 4
    phi10, _ = oracle_mod.ins_deploy(prof, tr, classes, gpus, configs, 10.0, 0.3, 2000.0, 5.0)
    assert (phi10 >= phi - 1e-12).all()


def test_rejected_by_model_matches_dumps(oracle_mod):
    cfg = gen.make_config("multimodel", n_cand=40, n_req=1500)
    tr = cfg["traces"][0]
    rbm = oracle_mod.rejected_by_model(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32)
    res = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32)
    assert (rbm.sum(axis=1) == res["n_rejected"]).all()
    assert (rbm[:, 3:] == 0).all()
    assert (rbm <= np.bincount(tr["model"], minlength=16)[None, :]).all()


# ---- Alg. 2: dynamic resource partition -----------------------------------------------------
def test_partition_scan(oracle_mod):
    prof = gen.profile_multimodel(0)
    tr = gen.make_trace(1500, 20.0, 3, model_mix=(0.6, 0.3, 0.1))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    configs = [(0, 8), (1, 16), (3, 8), (3, 64)]
    gpus, mt, ml = 12, 0b001, 0b110
    args = (4.0, 0.3, 2000.0, 5.0)
    got = oracle_mod.partition(prof, tr, classes, mt, ml, gpus, configs, *args)
    n_l = int(((ml >> tr["cls"]) & 1).sum())
    gl_max = n_l * gpus // len(tr)
    phi_l, I_l = oracle_mod.ins_deploy(prof, tr, classes, gl_max, configs, *args, class_mask=ml)
    phi_t, I_t = oracle_mod.ins_deploy(prof, tr, classes, gpus, configs, *args, class_mask=mt)
    best, arg = 0.0, (0, 0)
    for gl in range(1, gl_max + 1):            # brute-force scan, first strictly better wins
        if phi_t[gpus - gl] + phi_l[gl] > best:
            best, arg = phi_t[gpus - gl] + phi_l[gl], (gpus - gl, gl)
    assert (got["g_t"], got["g_l"]) == arg and got["phi"] == best
    assert got["g_t"] + got["g_l"] == gpus
    # constraint (c) of Sec. IV-C: each sub-cluster's placement fits its share of the devices
    for side, g in (("inst_t", got["g_t"]), ("inst_l", got["g_l"])):
        if len(got[side]):
            assert prof["devices"][gen.unpack_inst(got[side])[1]].sum() <= g
    assert got["inst_t"].tolist() == I_t[arg[0]].tolist() and got["inst_l"].tolist() == I_l[arg[1]].tolist()
    # homogeneous fallback: an unbeatable baseline leaves the cluster unpartitioned
    phi_h, _ = oracle_mod.ins_deploy(prof, tr, classes, gpus, configs, *args, class_mask=mt | ml)
    with_base = oracle_mod.partition(prof, tr, classes, mt, ml, gpus, configs, *args, baseline=True)
    assert with_base["phi"] == max(best, phi_h.max())
    # no latency-tolerant requests -> G'_l = 0 -> nothing to scan
    none = oracle_mod.partition(prof, tr, classes, 0b111, 0, gpus, configs, *args)
    assert (none["g_t"], none["g_l"], none["phi"]) == (0, 0, 0.0) and len(none["inst_t"]) == 0


# ---- paper-shaped workload (Table I) and Eq.-1 tables ----------------------------------------
def test_table1_generator_shapes():
    cfg = gen.make_config("table1-4", n_cand=50, n_req=4000)
    tr = cfg["traces"][0]
    assert len(cfg["classes"]) == 71 and (cfg["classes"]["ttft_us"] < 0).all()
    theta = int(cfg["profile"]["step_us"][0, 0, 0])
    f = 0.80 + 0.01 * tr["cls"]
    short = tr["out_tokens"] <= 500
    assert ((tr["out_tokens"] >= 300) & (tr["out_tokens"] <= 1000)).all()
    assert (f[short] <= 1.0 + 1e-9).all() and (f[~short] >= 1.2 - 1e-9).all()      # trace 4 pairs them
    assert abs(short.mean() - 0.5) < 0.05
    assert (cfg["classes"]["tbt_us"] == np.floor((0.80 + 0.01 * np.arange(71)) * theta + 0.5)).all()
    # Eq. 1: per-request decode rate decays with the level and is truncated at the batch cap by use
    step = cfg["profile"]["step_us"]
    assert (np.diff(step, axis=2) >= 0).all()
    rate = 1e6 / step[0, 0]
    t0 = rate[0] / (1.0 - 0.08 * np.log(2.0))
    assert np.allclose(rate, t0 * (1.0 - 0.08 * np.log(1.0 + np.arange(1, 65))), rtol=2e-4)
    # gamma arrivals with CV 2: squared CV of the gaps near 4
    gaps = np.diff(tr["arrival_us"].astype(np.float64))
    assert 2.5 < gaps.var() / gaps.mean() ** 2 < 6.0


# ---- configuration tree and pruning (Sec. III-C, IV-D) ---------------------------------------
def test_prune_configs_strategy_rule_and_order(oracle_mod):
    """Hand-made tables: strategy 1 is slower than 0 on more devices (dropped), 2 is faster on more
    devices (kept), 3 copies 2 (the copy is dropped), 4 is faster than 0 at low levels but slower at
    high ones (kept: no dominance), 5 fits no model (dropped)."""
    W = gen.WMAX
    w = np.arange(1, W + 1)
    step = np.stack([9000 + 100 * w, 9500 + 100 * w, 5000 + 100 * w, 5000 + 100 * w,
                     6000 + 400 * w, 3000 + 50 * w])[None].astype(np.int32)
    prof = {"n_models": 1, "n_strategies": 6, "wmax": W,
            "devices": np.array([1, 2, 2, 2, 1, 1], dtype=np.int32), "min_devices": np.array([1], dtype=np.int32),
            "prefill_base_us": np.array([[2000, 2000, 1000, 1000, 2000, 500]], dtype=np.int32),
            "prefill_q16": np.array([[7000, 7000, 3500, 3500, 7000, 100]], dtype=np.int32), "step_us": step}
    prof["min_devices"] = np.array([1], dtype=np.int32)
    tr = gen.make_trace(300, 10.0, 1, doc_class=None)
    classes = gen.make_classes(NONE3 * 3)
    got = oracle_mod.prune_configs(prof, tr, classes, [4])
    # strategy 5 needs one device and is faster than every other row everywhere: it alone survives
    assert [s for s, _ in got] == [5]
    prof["min_devices"] = np.array([2], dtype=np.int32)      # now nothing fits on one device
    got = oracle_mod.prune_configs(prof, tr, classes, [4])
    assert [s for s, _ in got] == [2]                         # a strategy that hosts nothing dominates nothing
    prof["min_devices"] = np.array([1], dtype=np.int32)
    prof["step_us"] = step.copy()
    prof["step_us"][0, 5] = 20000                             # strategy 5 no longer dominates anybody
    got = oracle_mod.prune_configs(prof, tr, classes, [4])
    # order: increasing level-1 step: 2 (5100), 4 (6400), 0 (9100), 5 (20000); 1 and 3 dropped
    assert [s for s, _ in got] == [2, 4, 0, 5]


def test_prune_configs_batch_pareto(oracle_mod):
    from fractions import Fraction
    prof = gen.profile_multimodel(0)
    tr = gen.make_trace(1500, 25.0, 3, model_mix=(0.6, 0.3, 0.1))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    batches = [1, 2, 4, 8, 16, 32, 64]
    for mask in (None, 0b011):
        got = oracle_mod.prune_configs(prof, tr, classes, batches, class_mask=mask)
        strategies = []
        for s, _ in got:
            if s not in strategies:
                strategies.append(s)
        assert all(gen.STRATEGIES_NODE[s][1] == 1 for s in strategies)      # pipeline strategies lose to tp / dp
        lvl1 = [int(prof["step_us"][0, s, 0]) for s in strategies]
        assert lvl1 == sorted(lvl1)
        want = []
        for s in strategies:                                                 # brute-force Pareto front
            outcome = []
            for b in batches:
                lst = [(m, s, b) for m in range(3) if prof["devices"][s] >= prof["min_devices"][m]]
                off, inst = gen.candidates_from_lists([lst])
                cm = None if mask is None else np.array([mask], dtype=np.uint32)
                r = oracle_mod.eval_placements(prof, tr, classes, off, inst, 10 ** 9, cm)[0]
                lat = Fraction(int(r["sum_ttft_us"]), int(r["n_served"])) if r["n_served"] else None
                outcome.append((int(r["n_hit"]), lat))
            def le(x, y):
                return y is None or (x is not None and x <= y)
            for i, b in enumerate(batches):
                dom = False
                for j in range(len(batches)):
                    if i == j:
                        continue
                    hit_ge, hit_gt = outcome[j][0] >= outcome[i][0], outcome[j][0] > outcome[i][0]
                    lat_le = le(outcome[j][1], outcome[i][1])
                    lat_lt = lat_le and outcome[j][1] != outcome[i][1]
                    if hit_ge and lat_le and (hit_gt or lat_lt or batches[j] < b):
                        dom = True
                if not dom:
                    want.append((s, b))
        assert got == want


# ---- time-to-first-token histogram and percentiles (Sec. V-A "response latency") -----------
def _prefill_only_profile(bases):
    """One model; strategy s = an instance whose prefill takes exactly bases[s] us (no per-token part)."""
    n = len(bases)
    return {"n_models": 1, "n_strategies": n, "wmax": gen.WMAX,
            "devices": np.ones(n, dtype=np.int32), "min_devices": np.array([1], dtype=np.int32),
            "prefill_base_us": np.array([bases], dtype=np.int32),
            "prefill_q16": np.zeros((1, n), dtype=np.int32),
            "step_us": np.full((1, n, gen.WMAX), 5000, dtype=np.int32)}


# time to first token -> bin, worked out by hand from the definition in include/maaso.h:
# below 1024 -> 0; 1024..1535 -> 1; 1536..2047 -> 2; 2048..3071 -> 3; 3072..4095 -> 4; 2^20 -> 21;
# 1.5 * 2^20 -> 22; 2^30 -> 41; 2^30 + 2^29 -> 42
TTFT_BIN_EDGES = [(0, 0), (1, 0), (1023, 0), (1024, 1), (1535, 1), (1536, 2), (2047, 2), (2048, 3), (3071, 3),
                  (3072, 4), (4095, 4), (4096, 5), (1 << 20, 21), ((1 << 20) + (1 << 19), 22),
                  ((1 << 21) - 1, 22), (1 << 30, 41), ((1 << 30) + (1 << 29), 42), ((1 << 31) - 1, 42)]


def test_ttft_histogram_bin_edges(oracle_mod):
    """One idle instance, one request: the time to first token is exactly the prefill time."""
    bases = [b for b, _ in TTFT_BIN_EDGES]
    prof = _prefill_only_profile(bases)
    trace = np.zeros(1, dtype=gen.REQUEST_DTYPE)
    trace["arrival_us"] = 5
    trace["in_tokens"] = 100
    trace["out_tokens"] = 2
    classes = gen.make_classes(NONE3)
    offsets, inst = gen.candidates_from_lists([[(0, s, 1)] for s in range(len(bases))])
    hist = oracle_mod.ttft_hist(prof, trace, classes, offsets, inst, 4)
    for c, (_, want_bin) in enumerate(TTFT_BIN_EDGES):
        row = np.zeros(64, dtype=np.uint32)
        row[want_bin] = 1
        assert hist[c].tolist() == row.tolist(), (c, TTFT_BIN_EDGES[c], np.nonzero(hist[c])[0])


def test_ttft_histogram_counts_served_requests_only(oracle_mod):
    cfg = gen.make_config("tiny")
    tr = cfg["traces"][0]
    res, dumps = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"],
                                            cfg["budget"], dump_idx=np.arange(len(cfg["offsets"]) - 1))
    hist = oracle_mod.ttft_hist(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], cfg["budget"])
    assert (hist.sum(axis=1) == res["n_served"]).all()
    assert int(res["n_rejected"].sum()) > 0
    # every percentile bound brackets the exact order statistic of the dumped first-token times
    arr = tr["arrival_us"].astype(np.int64)
    pct = oracle_mod.ttft_percentiles(hist, [500, 900, 990, 1000])
    for c in range(0, len(hist), 7):
        first = dumps["first_us"][c]
        t = np.sort((first - arr)[first >= 0])
        if len(t) == 0:
            assert (pct[c] == -1).all()
            continue
        for j, pm in enumerate([500, 900, 990, 1000]):
            exact = int(t[(pm * len(t) + 999) // 1000 - 1])      # the ceil(pm * n / 1000)-th smallest
            upper = int(pct[c, j])
            assert exact <= upper, (c, pm, exact, upper)
            assert upper < max(1024, exact + exact // 2 + 1), (c, pm, exact, upper)   # two bins per octave


def test_ttft_percentiles_by_hand(oracle_mod):
    h = np.zeros((4, 64), dtype=np.uint32)
    h[0, 0], h[0, 3] = 10, 10        # ten below 1024 us, ten in 2048..3071
    h[1, 63] = 5                     # open last bin
    h[2, 21] = 1                     # a single value in [2^20, 1.5 * 2^20)
    pct = oracle_mod.ttft_percentiles(h, [1, 500, 501, 1000])
    assert pct[0].tolist() == [1023, 1023, 3071, 3071]    # ranks 1, 10, 11, 20 of 20
    assert pct[1].tolist() == [np.iinfo(np.int64).max] * 4
    assert pct[2].tolist() == [(1 << 20) + (1 << 19) - 1] * 4
    assert pct[3].tolist() == [-1] * 4                    # nothing served

"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact records,
per-request times and ranking."""
import numpy as np
import pytest

import gen
from golden_cases import all_cases, check_against_expect
from gpu_common import gpu_eval, assert_records_equal

pytestmark = pytest.mark.gpu

MAPPINGS = [3, 2, 1]  # thread per placement, lane groups, block layout


@pytest.fixture(scope="module")
def ctx():
    import paper_2509_06362_b200 as m
    c = m.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("case", all_cases(), ids=lambda c: c["name"])
def test_hand_timelines_on_gpu(ctx, case, mapping):
    for flags, expect in case["runs"]:
        if (flags & 14) and mapping != 2:
            continue      # the fixed-speed engine and the largest-gap test exist in the lane-group mapping only
        res, dumps = gpu_eval(ctx, case["profile"], case["trace"], case["classes"], case["offsets"],
                              case["inst"], case["budget"], None, flags, mapping, dump_idx=[0])
        check_against_expect(res[0], {k: v[0] for k, v in dumps.items()}, expect)


@pytest.mark.parametrize("mapping", MAPPINGS)
@pytest.mark.parametrize("flags", [0, 1])
def test_tiny_config_full(ctx, oracle_mod, mapping, flags):
    cfg = gen.make_config("tiny")
    tr = cfg["traces"][0]
    idx = np.arange(0, 143, 5, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"],
                                          cfg["budget"], None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], cfg["budget"],
                       None, flags, mapping, dump_idx=idx)
    assert_records_equal(got, want, "tiny")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_node_config_subset(ctx, oracle_mod, mapping):
    # ragged sizes: 1777 requests = 6 tiles of 256 + a tail; candidates span every group width
    cfg = gen.make_config("node", n_req=1777)
    sel = np.arange(0, 10864, 23)
    lists = []
    for c in sel:
        w = cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]]
        m, s, b = gen.unpack_inst(w)
        lists.append(list(zip(m.tolist(), s.tolist(), b.tolist())))
    off, inst = gen.candidates_from_lists(lists)
    tr = cfg["traces"][0]
    idx = np.arange(0, len(sel), 37, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 8, mapping=mapping, dump_idx=idx)
    assert_records_equal(got, want, "node subset")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_multimodel_subset_with_masks(ctx, oracle_mod, mapping):
    cfg = gen.make_config("multimodel", n_cand=600, n_req=3000)
    tr = cfg["traces"][0]
    rng = np.random.default_rng(5)
    mask = rng.integers(1, 8, size=600).astype(np.uint32)
    want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32, mask)
    got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32, mask,
                      mapping=mapping)
    assert_records_equal(got, want, "multimodel masks")


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_bursty_optimistic_shows_cascades(ctx, oracle_mod, mapping):
    cfg = gen.make_config("bursty", n_req=1500)
    sel = slice(0, 10864, 61)
    off_full, inst_full = cfg["offsets"], cfg["inst"]
    lists = []
    for c in range(0, 10864, 61):
        m, s, b = gen.unpack_inst(inst_full[off_full[c]:off_full[c + 1]])
        lists.append(list(zip(m.tolist(), s.tolist(), b.tolist())))
    off, inst = gen.candidates_from_lists(lists)
    total_cascade = 0
    for j in (3, 9, 15):
        tr = cfg["traces"][j]
        for flags in (0, 1):
            want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags)
            got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags, mapping)
            assert_records_equal(got, want, f"bursty trace {j} flags {flags}")
            total_cascade += int(got["n_cascade"].sum())
    assert total_cascade > 0


def _large_placements():
    prof = gen.profile_multimodel(0)
    rng = np.random.default_rng(3)
    lists = []
    for n_i in (33, 40, 64, 97, 128, 128, 5, 32, 1):
        lst = []
        for _ in range(n_i):
            m = int(rng.integers(3))
            s = 3 if m == 2 else 0
            lst.append((m, s, int(rng.choice([1, 2, 4, 8, 16, 32, 64]))))
        lists.append(lst)
    off, inst = gen.candidates_from_lists(lists)
    tr = gen.make_trace(4000, 400.0, 9, model_mix=(0.6, 0.3, 0.1), class_mix=(0.45, 0.27, 0.18, 0.10))
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None),
                                (None, None, 180_000_000), (30_000_000, None, 600_000_000)])
    return prof, off, inst, tr, classes


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_large_placements_over_32_instances(ctx, oracle_mod, mapping):
    """Candidates with up to 128 instances (budget 128): the thread kernel, the block path."""
    prof, off, inst, tr, classes = _large_placements()
    idx = np.array([1, 4, 6], dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(prof, tr, classes, off, inst, 1024, dump_idx=idx)
    got, gd = gpu_eval(ctx, prof, tr, classes, off, inst, 1024, mapping=mapping, dump_idx=idx)
    assert (want["status"] == 0).all()
    assert_records_equal(got, want, "large placements")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


@pytest.mark.parametrize("flags", [0, 1, 2, 3, 4, 5, 6, 8, 9, 12])
def test_large_placements_over_32_instances_every_engine(ctx, oracle_mod, flags):
    """No engine stops at 32 instances: the optimistic estimate, the fixed-speed engine, the largest-gap
    test and per-instance queues (and combinations) on placements of 33 to 128 instances, records and
    per-request times against the oracle; no ETOOMANY below 129 instances."""
    prof, off, inst, tr, classes = _large_placements()
    idx = np.array([0, 4, 6], dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(prof, tr, classes, off, inst, 1024, None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, prof, tr, classes, off, inst, 1024, None, flags, 0, dump_idx=idx)
    assert (want["status"] == 0).all()
    assert_records_equal(got, want, f"large placements, flags {flags}")
    for k in wd:
        assert (gd[k] == wd[k]).all(), (k, flags)


@pytest.mark.parametrize("flags,mapping", [(0, 0), (0, 3), (1, 0), (2, 0), (8, 0), (4, 0)])
def test_large_configuration_sample(ctx, oracle_mod, flags, mapping):
    """The configuration of placements with 33 to 128 instances (2,000 of them in full): every 25th
    against the whole trace, one warp per placement (and the thread kernel, forced)."""
    cfg = gen.make_config("large")
    sel = np.arange(0, len(cfg["offsets"]) - 1, 25)
    parts = [cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]] for c in sel]
    off = np.concatenate([[0], np.cumsum([len(x) for x in parts])]).astype(np.uint32)
    inst = np.concatenate(parts).astype(np.uint32)
    tr = cfg["traces"][0]
    idx = np.array([0, 40, 79], dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, cfg["budget"], None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, cfg["budget"], None, flags, mapping, dump_idx=idx)
    assert (want["status"] == 0).all()
    assert_records_equal(got, want, f"large configuration, flags {flags}, mapping {mapping}")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


@pytest.mark.parametrize("flags", [0, 1])
def test_thread_kernel_classes_no_instance_can_serve(ctx, oracle_mod, flags):
    """The thread kernel turns a request away while scanning when no instance of its model can meet the
    class's TBT limit (the prediction step of every instance is above it).  The cases around that rule:
    such a request of ONE output token has no TBT term and must still be served; classes 32 and up are
    never filtered there; a class without a TBT limit; the optimistic estimate, where the step of a lower
    level may meet the limit although the step at the batch cap does not.  Records, per-request times and
    per-model rejection counts against the oracle."""
    import torch
    prof = gen.profile_multimodel(0)
    # model 1 / strategy 9 / cap 64: 71 ms per step at the cap, 35 ms at level 1; model 2 is slower still
    lists = [[(1, 9, 64), (1, 9, 64)], [(1, 9, 64), (2, 5, 8), (0, 6, 4)], [(2, 9, 64)], [(1, 9, 2), (1, 5, 32)],
             [(0, 0, 64), (1, 3, 64), (2, 6, 1)], [(2, 3, 1), (2, 4, 2), (1, 8, 64)]]
    off, inst = gen.candidates_from_lists(lists)
    rows = [(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000), (None, 40_000, None)]
    rows += [(3_000_000, 60_000 + 5_000 * k, None) for k in range(36)]          # classes 4..39, some beyond bit 31
    classes = gen.make_classes(rows)
    tr = gen.make_trace(6000, 80.0, 17, model_mix=(0.3, 0.4, 0.3), class_mix=(0.25, 0.2, 0.1, 0.15) + (0.3 / 36,) * 36)
    tr["out_tokens"][::5] = 1                                                   # no TBT term for these
    tr["out_tokens"][1::9] = 2
    idx = np.arange(len(lists), dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(prof, tr, classes, off, inst, 1024, None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, prof, tr, classes, off, inst, 1024, None, flags, 3, dump_idx=idx)
    assert (want["status"] == 0).all()
    assert_records_equal(got, want, f"classes no instance can serve, flags {flags}")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k
    served_single = (wd["finish_us"][0] >= 0) & (tr["out_tokens"] == 1) & (tr["cls"] == 0) & (tr["model"] == 1)
    assert served_single.any()        # the case exists: class 0 on the 71 ms instances, served because of one token
    ctx.load_profile(prof)
    t = ctx.load_trace(tr, classes)
    rbm = torch.full((len(lists), 16), 77, dtype=torch.int32, device="cuda")
    ctx.eval_placements(t, ctx.to_device(off), ctx.to_device(inst), 1024, None, flags, 3, rejected_by_model=rbm)
    torch.cuda.synchronize()
    assert (rbm.cpu().numpy().view(np.uint32) == oracle_mod.rejected_by_model(prof, tr, classes, off, inst, 1024, flags=flags)).all()
    ctx.free_trace(t)


@pytest.mark.parametrize("flags,mapping", [(0, 2), (2, 0), (8, 0), (4, 0)])
def test_large_placements_several_traces_in_one_pass(ctx, oracle_mod, flags, mapping):
    """The same placements against three traces in one call, where the thread kernel is not used (lane
    groups forced, or one of the other engines): one warp per placement with the lane-group code."""
    import torch
    prof, off, inst, tr, classes = _large_placements()
    traces_np = [tr[:1500], tr[1000:3100].copy(), tr[:700]]
    traces_np[1]["arrival_us"] -= traces_np[1]["arrival_us"][0]
    ctx.load_profile(prof)
    handles = [ctx.load_trace(t, classes) for t in traces_np]
    out = ctx.eval_placements_multi(handles, ctx.to_device(off), ctx.to_device(inst), 1024, None, flags, mapping=mapping)
    torch.cuda.synchronize()
    got = ctx.results_to_numpy(out).reshape(3, -1)
    for t, trn in enumerate(traces_np):
        want = oracle_mod.eval_placements(prof, trn, classes, off, inst, 1024, None, flags)
        assert (want["status"] == 0).all()
        assert_records_equal(got[t], want, f"trace {t}, flags {flags}")
    for h in handles:
        ctx.free_trace(h)


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_edge_cases(ctx, oracle_mod, mapping):
    prof = gen.profile_multimodel(0)
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    lists = [
        [(0, 6, 4), (0, 6, 4)], [(2, 0, 4)], [(0, 0, 4)] * 129, [(3, 0, 4)], [(0, 10, 4)], [(0, 0, 0)],
        [(0, 0, 65)], [(0, 0, 4), (2, 3, 8)], [], [(1, 1, 64)],
    ]
    off, inst = gen.candidates_from_lists(lists)
    tr = gen.make_trace(700, 30.0, 4, model_mix=(0.6, 0.3, 0.1))
    tr["out_tokens"][::7] = 1          # single-token requests never occupy a slot
    tr["arrival_us"][100:140] = tr["arrival_us"][100]   # simultaneous arrivals
    want = oracle_mod.eval_placements(prof, tr, classes, off, inst, 8)
    got, _ = gpu_eval(ctx, prof, tr, classes, off, inst, 8, mapping=mapping)
    assert_records_equal(got, want, "edge cases")
    # empty trace: every valid candidate gets an all-zero record
    empty = tr[:0]
    want = oracle_mod.eval_placements(prof, empty, classes, off, inst, 8)
    got, _ = gpu_eval(ctx, prof, empty, classes, off, inst, 8, mapping=mapping)
    assert_records_equal(got, want, "empty trace")
    # one request, one candidate
    want = oracle_mod.eval_placements(prof, tr[:1], classes, off[7:9] - off[7], inst[off[7]:off[8]], 8)
    got, _ = gpu_eval(ctx, prof, tr[:1], classes, off[7:9] - off[7], inst[off[7]:off[8]], 8, mapping=mapping)
    assert_records_equal(got, want, "single")


def _subset(cfg, sel):
    lists = []
    for c in sel:
        m, s, b = gen.unpack_inst(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        lists.append(list(zip(m.tolist(), s.tolist(), b.tolist())))
    return gen.candidates_from_lists(lists)


def test_node_config_full_size_as_benchmarked(ctx, oracle_mod):
    """The benchmark's workload and launch configuration: all 10,864 placements x 10,000 requests."""
    cfg = gen.make_config("node")
    tr = cfg["traces"][0]
    want = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8)
    assert (want["status"] == 0).all() and (want["n_counted"] == 10000).all()
    for mapping in (0, 2, 3, 1):
        got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=mapping)
        assert_records_equal(got, want, f"node full, mapping {mapping}")


@pytest.mark.parametrize("flags", [1, 2, 4, 8, 9])
def test_node_config_full_size_variants_sampled(ctx, oracle_mod, flags):
    """The other readings on the benchmark's workload, full size on the GPU (so that every placement sits
    in the launch bucket, warp and lane it gets there); every 50th record checked against the oracle."""
    cfg = gen.make_config("node")
    tr = cfg["traces"][0]
    got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, None, flags, 0)
    sel = list(range(0, 10864, 50)) + [10863]
    off, inst = _subset(cfg, sel)
    want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags)
    assert_records_equal(got[sel], want, f"node full, flags {flags}, sampled")


def test_multimodel_full_trace_sampled_candidates(ctx, oracle_mod):
    cfg = gen.make_config("multimodel")
    tr = cfg["traces"][0]
    n_i = np.diff(cfg["offsets"].astype(np.int64))
    sel = sorted(set(np.arange(0, 100_000, 400).tolist() + np.argsort(n_i)[-6:].tolist()))
    off, inst = _subset(cfg, sel)
    idx = np.array([0, len(sel) - 1], dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 32, dump_idx=idx)
    for mapping in (2, 3):
        got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 32, mapping=mapping, dump_idx=idx)
        assert_records_equal(got, want, f"multimodel full trace, mapping {mapping}")
        for k in wd:
            assert (gd[k] == wd[k]).all(), (k, mapping)


def test_scale_full_trace_sampled_candidates(ctx, oracle_mod):
    """10^6-request trace, four SLO classes, 272 placements of the 10^6-placement set: an even sample,
    the ones with the most instances (over 32) and some of every lane-group width (1, 2, 3-4, 5-8,
    9-16, 17-32 instances); per-request times compared for six of them."""
    cfg = gen.make_config("scale")
    tr = cfg["traces"][0]
    n_i = np.diff(cfg["offsets"].astype(np.int64))
    pick = set(np.arange(0, 1_000_000, 5_000).tolist() + np.argsort(n_i)[-8:].tolist())
    for lo_n, hi_n in ((1, 1), (2, 2), (3, 4), (5, 8), (9, 16), (17, 32), (33, 128)):
        pick.update(np.nonzero((n_i >= lo_n) & (n_i <= hi_n))[0][:10].tolist())
    sel = sorted(pick)
    assert len(sel) >= 256 and (n_i[sel] > 32).sum() >= 4
    off, inst = _subset(cfg, sel)
    big = [k for k, c in enumerate(sel) if n_i[c] > 32][:2]
    idx = np.array(sorted(set([0, len(sel) // 3, len(sel) // 2, len(sel) - 1] + big)), dtype=np.uint32)
    want = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], off, inst, 128, workers=8)
    _, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], *_subset(cfg, [sel[k] for k in idx]), 128,
                                       dump_idx=np.arange(len(idx), dtype=np.uint32))
    assert (want["status"] == 0).all() and n_i.max() > 32
    for mapping in (2, 3):
        got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 128, mapping=mapping, dump_idx=idx)
        assert_records_equal(got, want, f"scale full trace, mapping {mapping}")
        for k in wd:
            assert (gd[k] == wd[k]).all(), (k, mapping)


def test_multimodel_all_candidates_trace_prefix(ctx, oracle_mod):
    """Every one of the 100,000 placements of the multi-model sweep in ONE call (the batch size the
    benchmark launches: many waves of work items, cost-sorted buckets), against the first 200 requests."""
    cfg = gen.make_config("multimodel", n_req=200)
    tr = cfg["traces"][0]
    want = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32,
                                               workers=8)
    assert len(want) == 100_000 and (want["status"] == 0).all()
    for mapping in (2, 3):
        got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 32, mapping=mapping)
        assert_records_equal(got, want, f"multimodel, all placements, mapping {mapping}")


def test_scale_all_candidates_trace_prefix_and_topk(ctx, oracle_mod):
    """All 10^6 placements of the scale-stress sweep in ONE call (placements of more than 32 instances
    mixed in), against the first 100 requests; records byte for byte, and the top-64 of that run
    against the CPU ranking."""
    import torch
    cfg = gen.make_config("scale", n_req=100)
    tr = cfg["traces"][0]
    want = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 128,
                                               workers=8)
    assert len(want) == 1_000_000 and (want["status"] == 0).all()
    top = oracle_mod.topk(want, 64)
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    d_off, d_inst = ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"])
    for mapping in (2, 3):
        out = ctx.eval_placements(t, d_off, d_inst, 128, mapping=mapping)
        idx, rec = ctx.topk(out, 64)
        torch.cuda.synchronize()
        assert_records_equal(ctx.results_to_numpy(out), want, f"scale, all placements, mapping {mapping}")
        assert idx.cpu().numpy().view(np.uint32).tolist() == top.tolist()
        assert rec.cpu().numpy().tobytes() == want[top].tobytes()
    ctx.free_trace(t)


def test_bursty_all_traces_full_length(ctx, oracle_mod):
    cfg = gen.make_config("bursty")
    off, inst = _subset(cfg, range(0, 10864, 97))
    for j, tr in enumerate(cfg["traces"]):
        flags = j % 2
        want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags)
        got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags)
        assert_records_equal(got, want, f"bursty trace {j}")


def test_determinism_and_mapping_independence(ctx):
    cfg = gen.make_config("node", n_cand=700, n_req=2000)
    tr = cfg["traces"][0]
    a, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=0)
    b, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=0)
    c, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=1)
    d, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=2)
    e, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 8, mapping=3)
    assert a.tobytes() == b.tobytes() == c.tobytes() == d.tobytes() == e.tobytes()


def test_host_entry_point_matches_device_entry_point(ctx, oracle_mod):
    cfg = gen.make_config("tiny")
    tr = cfg["traces"][0]
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    host = ctx.eval_placements_host(t, cfg["offsets"], cfg["inst"], 4)
    ctx.free_trace(t)
    want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 4)
    assert_records_equal(host, want, "host entry")


def test_topk_matches_oracle_ranking(ctx, oracle_mod):
    import torch
    cfg = gen.make_config("node", n_cand=9000, n_req=600)
    tr = cfg["traces"][0]
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    res = ctx.eval_placements(t, ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"]), 8)
    torch.cuda.synchronize()
    rec = ctx.results_to_numpy(res)
    want_rec = oracle_mod.eval_placements_parallel(cfg["profile"], tr, cfg["classes"], cfg["offsets"],
                                                   cfg["inst"], 8)
    assert_records_equal(rec, want_rec, "topk input")
    for k in (1, 64, 1000):
        idx, out = ctx.topk(res, k)
        torch.cuda.synchronize()
        want = oracle_mod.topk(want_rec, k)
        got = idx.cpu().numpy().view(np.uint32)
        assert got.tolist() == want.tolist(), k
        assert ctx.results_to_numpy(out).tobytes() == want_rec[want].tobytes()
    # doctored records: invalid ones last, exact mean comparison, padding when k > n
    doctored = want_rec[:100].copy()
    doctored["status"][3] = 8
    doctored["n_hit"][:] = 7
    doctored["n_served"][:] = 1_000_003
    doctored["sum_ttft_us"][:] = (1 << 62) - np.arange(100, dtype=np.int64) % 5
    doctored["n_served"][10] = 0
    d = torch.from_numpy(doctored.view(np.uint8).reshape(100, 128)).cuda()
    idx, _ = ctx.topk(d, 128)
    torch.cuda.synchronize()
    got = idx.cpu().numpy().view(np.uint32)
    want = oracle_mod.topk(doctored, 128)
    assert got[:100].tolist() == want.tolist()
    assert (got[100:] == 0xFFFFFFFF).all()
    ctx.free_trace(t)


def test_topk_million_records_three_passes(ctx, oracle_mod):
    """Selection at the scale configuration's size: 10^6 records, k = 64 (three passes of the
    grid-level reduction), many ties on the hit count so that the exact mean comparison and
    the index tie-break decide."""
    import torch
    n = 1_000_000
    rng = np.random.default_rng(11)
    rec = np.zeros(n, dtype=gen.RESULT_DTYPE)
    rec["status"] = (rng.random(n) < 0.01) * 2
    rec["n_hit"] = rng.integers(900, 1000, n)
    rec["n_served"] = rng.integers(1, 1200, n)
    rec["sum_ttft_us"] = rng.integers(1, 1 << 44, n)
    dup = rng.integers(0, n, 2000)                      # exact duplicates: index decides
    rec[dup[:1000]] = rec[dup[1000:]]
    dev = torch.from_numpy(rec.view(np.uint8).reshape(n, 128)).cuda()
    for k in (64, 1024):
        idx, out = ctx.topk(dev, k)
        torch.cuda.synchronize()
        want = oracle_mod.topk(rec, k)
        assert idx.cpu().numpy().view(np.uint32).tolist() == want.tolist()
        assert ctx.results_to_numpy(out).tobytes() == rec[want].tobytes()


def test_score_and_ranking_by_score(ctx, oracle_mod):
    """Composite serving score (Sec. IV-D) in double precision: the kernel uses explicitly rounded
    operations in the oracle's order, so values are expected to be identical; the test allows
    4 ulp.  Ranking by score takes its decisions on the same doubles on both sides."""
    import torch
    cfg = gen.make_config("node", n_cand=6000, n_req=800)
    tr = cfg["traces"][0]
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    res = ctx.eval_placements(t, ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"]), 8)
    torch.cuda.synchronize()
    rec = ctx.results_to_numpy(res).copy()
    rec["status"][17] = 4
    rec["n_served"][23] = 0
    rec["n_counted"][29] = 0
    dev = torch.from_numpy(rec.view(np.uint8).reshape(-1, 128)).cuda()
    for (alpha, beta, gt, gl) in [(4.0, 0.3, 800.0, 10.0), (10.0, 0.3, 800.0, 10.0), (2.5, 0.0, 50.0, 0.5),
                                  (1.0, 1.0, 1e9, 1e-9)]:
        got = ctx.score(dev, alpha, beta, gt, gl).cpu().numpy()
        want = oracle_mod.score(rec, alpha, beta, gt, gl)
        ulp = np.spacing(np.maximum(np.abs(want), 1e-300))
        assert (np.abs(got - want) <= 4 * ulp).all(), np.abs(got - want).max()
        for k in (1, 64, 1000):
            idx, out = ctx.topk_scores(dev, torch.from_numpy(want).cuda(), k)
            torch.cuda.synchronize()
            w = oracle_mod.topk_scores(want, k)
            assert idx.cpu().numpy().view(np.uint32).tolist() == w.tolist()
            assert ctx.results_to_numpy(out).tobytes() == rec[w].tobytes()
    s = oracle_mod.score(rec, 4.0, 0.3, 800.0, 10.0)
    s[5] = np.nan
    s[100] = s[200] = s.max() + 1.0
    idx, _ = ctx.topk_scores(dev, torch.from_numpy(s).cuda(), 1024)
    torch.cuda.synchronize()
    assert idx.cpu().numpy().view(np.uint32).tolist() == oracle_mod.topk_scores(s, 1024).tolist()
    # NaN ranks last: a tiny set where k covers everything
    small = torch.from_numpy(rec[:8].view(np.uint8).reshape(8, 128)).cuda()
    idx, _ = ctx.topk_scores(small, torch.from_numpy(s[:8]).cuda(), 8)
    torch.cuda.synchronize()
    assert idx.cpu().numpy().view(np.uint32).tolist() == oracle_mod.topk_scores(s[:8], 8).tolist()
    ctx.free_trace(t)


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_rejected_by_model(ctx, oracle_mod, mapping):
    import torch
    cfg = gen.make_config("multimodel", n_cand=300, n_req=2500)
    tr = cfg["traces"][0]
    lists = [[(2, 0, 4)], []]                       # an invalid candidate and the empty placement
    off2, inst2 = gen.candidates_from_lists(lists)
    off = np.concatenate([cfg["offsets"], cfg["offsets"][-1] + off2[1:]]).astype(np.uint32)
    inst = np.concatenate([cfg["inst"], inst2]).astype(np.uint32)
    mask = np.random.default_rng(2).integers(1, 8, size=len(off) - 1).astype(np.uint32)
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    rbm = torch.full((len(off) - 1, 16), 77, dtype=torch.int32, device="cuda")
    ctx.eval_placements(t, ctx.to_device(off), ctx.to_device(inst), 32, ctx.to_device(mask), mapping=mapping,
                        rejected_by_model=rbm)
    torch.cuda.synchronize()
    want = oracle_mod.rejected_by_model(cfg["profile"], tr, cfg["classes"], off, inst, 32, mask)
    assert (rbm.cpu().numpy().view(np.uint32) == want).all()
    ctx.free_trace(t)


def test_ins_deploy_matches_oracle(ctx, oracle_mod):
    """Alg. 1 driven on the GPU (one batch of tentative placements per greedy step) against the
    sequential oracle: identical scores (same doubles) and identical placements per device count."""
    prof = gen.profile_multimodel(0)
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    ctx.load_profile(prof)
    cases = [
        (gen.make_trace(3000, 30.0, 3, model_mix=(0.2, 0.7, 0.1)), 16, [(0, 8), (1, 16), (3, 8), (3, 64), (6, 16), (0, 1)], None),
        (gen.make_trace(2000, 60.0, 4, cv=2.0, model_mix=(0.6, 0.3, 0.1)), 24,
         [(s, b) for s in (0, 1, 3, 6) for b in (4, 16, 64)], 0b011),
        (gen.make_trace(500, 5.0, 5, model_mix=(1.0, 0.0, 0.0)), 3, [(6, 16), (0, 2)], None),
    ]
    for tr, gpus, configs, mask in cases:
        t = ctx.load_trace(tr, classes)
        for alpha in (4.0, 10.0):
            phi, I = ctx.ins_deploy(t, gpus, configs, alpha, 0.3, 3000.0, 5.0, class_mask=mask)
            wphi, wI = oracle_mod.ins_deploy(prof, tr, classes, gpus, configs, alpha, 0.3, 3000.0, 5.0, class_mask=mask)
            assert phi.tolist() == wphi.tolist()
            assert [x.tolist() for x in I] == [x.tolist() for x in wI]
        ctx.free_trace(t)


def test_partition_matches_oracle(ctx, oracle_mod):
    prof = gen.profile_multimodel(0)
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    ctx.load_profile(prof)
    tr = gen.make_trace(2500, 30.0, 6, cv=2.0, model_mix=(0.6, 0.3, 0.1))
    t = ctx.load_trace(tr, classes)
    configs = [(s, b) for s in (0, 1, 3) for b in (4, 16, 64)]
    for (mt, ml, base) in [(0b001, 0b110, False), (0b011, 0b100, True), (0b111, 0, False)]:
        got = ctx.partition(t, mt, ml, 16, configs, 4.0, 0.3, 3000.0, 5.0, baseline=base)
        want = oracle_mod.partition(prof, tr, classes, mt, ml, 16, configs, 4.0, 0.3, 3000.0, 5.0, baseline=base)
        assert (got["g_t"], got["g_l"], got["phi"]) == (want["g_t"], want["g_l"], want["phi"])
        assert got["inst_t"].tolist() == want["inst_t"].tolist()
        assert got["inst_l"].tolist() == want["inst_l"].tolist()
        # constraint (c) of Sec. IV-C: each sub-cluster's placement fits its share of the devices
        for side, g in (("inst_t", got["g_t"]), ("inst_l", got["g_l"])):
            if len(got[side]):
                assert prof["devices"][gen.unpack_inst(got[side])[1]].sum() <= g
    ctx.free_trace(t)


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_bounded_waits_give_up_cleanly(ctx, mapping):
    """Failure path without a fault: with the stall hook the trace copies are never issued, so every
    device-side wait runs into its bound.  The call must return, every valid candidate must carry
    ETIMEOUT (and nothing else), invalid ones keep their own status, and the context must score the
    same batch correctly right afterwards."""
    import torch
    import paper_2509_06362_b200 as m
    cfg = gen.make_config("node", n_cand=3000, n_req=700)
    lists = [[(0, 12, 4)]]
    off2, inst2 = gen.candidates_from_lists(lists)
    off = np.concatenate([cfg["offsets"], cfg["offsets"][-1] + off2[1:]]).astype(np.uint32)
    inst = np.concatenate([cfg["inst"], inst2]).astype(np.uint32)
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(cfg["traces"][0], cfg["classes"])
    d_off, d_inst = ctx.to_device(off), ctx.to_device(inst)
    res = ctx.eval_placements(t, d_off, d_inst, 8, flags=m.FLAG_TEST_STALL, mapping=mapping)
    torch.cuda.synchronize()
    rec = ctx.results_to_numpy(res)
    assert (rec["status"][:-1] == m.CAND_STATUS["ETIMEOUT"]).all()
    assert rec["status"][-1] == m.CAND_STATUS["EBADINST"]
    for name in ("n_counted", "n_served", "n_hit", "n_rejected", "checksum", "attempts"):
        assert (rec[name] == 0).all()
    good = ctx.eval_placements(t, d_off, d_inst, 8, mapping=mapping)
    torch.cuda.synchronize()
    g = ctx.results_to_numpy(good)
    assert (g["status"][:-1] == 0).all() and (g["n_counted"][:-1] == 700).all()
    ctx.free_trace(t)


@pytest.mark.parametrize("trace_no", [1, 4])
def test_table1_workload(ctx, oracle_mod, trace_no):
    """Paper-shaped workload: 17,000 arrivals per hour with CV 2, 71 SLO classes (more than 32, so
    class masks are ignored and classes >= 7 share the last per-class bin), Eq.-1 tables, 24 devices."""
    cfg = gen.make_config(f"table1-{trace_no}", n_cand=800)
    tr = cfg["traces"][0]
    mask = np.full(800, 0b1, dtype=np.uint32)          # must be ignored: 71 classes
    idx = np.array([3, 500], dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 24,
                                          mask, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], 24, mask, dump_idx=idx)
    assert (want["n_counted"] == 17000).all() and want["n_hit"].sum() > 0
    assert_records_equal(got, want, f"table1-{trace_no}")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


def test_prune_configs_matches_oracle(ctx, oracle_mod):
    classes = gen.make_classes([(500_000, 50_000, None), (2_000_000, 150_000, None), (None, None, 180_000_000)])
    batches = [1, 2, 4, 8, 16, 32, 64]
    for prof, mix in ((gen.profile_multimodel(0), (0.6, 0.3, 0.1)), (gen.profile_decay(), (1, 1, 1)),
                      (gen.profile_node(3), (1.0,))):
        ctx.load_profile(prof)
        for rate, mask in ((8.0, None), (40.0, 0b011), (150.0, 0b100)):
            tr = gen.make_trace(2500, rate, 7, cv=2.0, model_mix=mix)
            t = ctx.load_trace(tr, classes)
            got = ctx.prune_configs(t, prof["n_strategies"], batches, class_mask=mask)
            want = oracle_mod.prune_configs(prof, tr, classes, batches, class_mask=mask)
            assert got == want and len(got) > 0
            ctx.free_trace(t)


def test_placer_end_to_end(ctx, oracle_mod):
    """The placer as the paper runs it: getPrunedConfigs, then Alg. 2 over Alg. 1, on a Table-I
    shaped hour of traffic; library and oracle must name the same partition and placements."""
    cfg = gen.make_config("table1-4", n_cand=1, n_req=6000)
    prof, tr, classes = cfg["profile"], cfg["traces"][0], cfg["classes"][:32].copy()
    tr = tr.copy()
    tr["cls"] = np.minimum(tr["cls"] // 3, 31)           # 24 classes so that the class masks apply
    strict = sum(1 << k for k in range(0, 8))             # SLO factors up to about 1.0
    relaxed = sum(1 << k for k in range(8, 32))
    ctx.load_profile(prof)
    t = ctx.load_trace(tr, classes)
    batches = [1, 4, 16, 64]
    configs = ctx.prune_configs(t, prof["n_strategies"], batches)
    assert configs == oracle_mod.prune_configs(prof, tr, classes, batches) and len(configs) >= 2
    got = ctx.partition(t, strict, relaxed, 24, configs, 4.0, 0.3, 20000.0, 10.0, baseline=True)
    want = oracle_mod.partition(prof, tr, classes, strict, relaxed, 24, configs, 4.0, 0.3, 20000.0, 10.0, baseline=True)
    assert (got["g_t"], got["g_l"], got["phi"]) == (want["g_t"], want["g_l"], want["phi"])
    assert got["inst_t"].tolist() == want["inst_t"].tolist() and got["inst_l"].tolist() == want["inst_l"].tolist()
    ctx.free_trace(t)


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_extreme_values(ctx, oracle_mod, mapping):
    """Corners of the integer ranges: 65535-token outputs (16-bit completion keys at their limit and
    wrapping many times), decode steps of 2^30 us, 4-billion-token inputs, arrivals near 2^50 us with
    gaps far above 2^32 us (the wide division path), single-token requests, full 64-slot instances."""
    W = gen.WMAX
    rng = np.random.default_rng(17)
    step = np.zeros((2, 3, W), dtype=np.int32)
    step[:, 0] = 1 + np.arange(W)                      # microsecond steps
    step[:, 1] = (1 << 30) - np.arange(W)              # the largest allowed steps, decreasing with the level
    step[:, 2] = rng.integers(1, 1 << 20, size=(2, W))
    prof = {"n_models": 2, "n_strategies": 3, "wmax": W,
            "devices": np.array([1, 1, 2], dtype=np.int32), "min_devices": np.array([1, 1], dtype=np.int32),
            "prefill_base_us": np.array([[0, 1 << 30, 7], [3, 0, 1 << 20]], dtype=np.int32),
            "prefill_q16": np.array([[0, (1 << 31) - 1, 65536], [1, 0, 123456]], dtype=np.int32), "step_us": step}
    n = 1200
    tr = np.zeros(n, dtype=gen.REQUEST_DTYPE)
    gaps = rng.choice([0, 1, 1000, 10 ** 7, 5 * 10 ** 9, 3 * 10 ** 11], size=n, p=[0.2, 0.2, 0.3, 0.2, 0.07, 0.03])
    tr["arrival_us"] = np.minimum(np.cumsum(gaps), (1 << 50) - 1)
    tr["in_tokens"] = rng.choice([0, 1, 4096, 2 ** 32 - 1], size=n)
    tr["out_tokens"] = rng.choice([1, 2, 300, 40000, 65535], size=n)
    tr["cls"] = rng.integers(0, 3, size=n)
    tr["model"] = rng.integers(0, 2, size=n)
    classes = gen.make_classes([(None, None, None), (1 << 40, 1 << 40, 1 << 40), (10 ** 9, 10 ** 6, None)])
    lists = [[(0, 0, 64), (1, 0, 64)], [(0, 1, 1), (1, 1, 2)], [(0, 2, 64), (1, 2, 3), (0, 0, 1), (1, 1, 64)],
             [(m, s, b) for m in (0, 1) for s in (0, 1, 2) for b in (1, 7, 64)],
             [(0, 0, 1)], [(1, 2, 64)] * 40]
    off, inst = gen.candidates_from_lists(lists)
    idx = np.arange(len(lists), dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(prof, tr, classes, off, inst, 10 ** 6, dump_idx=idx)
    got, gd = gpu_eval(ctx, prof, tr, classes, off, inst, 10 ** 6, mapping=mapping, dump_idx=idx)
    assert (want["status"] == 0).all() and want["n_served"].sum() > 0
    assert_records_equal(got, want, "extreme values")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k


def test_step_counter_wraps_32_bits(ctx, oracle_mod):
    """70,000 requests of 65535 tokens through one single-slot instance: the instance's step counter
    passes 2^32 (the kernels keep it modulo 2^32 and compare only 16-bit distances; the oracle counts
    in 64 bits).  No limits, so everything is served in order (single-server queue)."""
    prof = gen.profile_tiny()
    prof["step_us"][:] = 3
    n = 70_000
    tr = np.zeros(n, dtype=gen.REQUEST_DTYPE)
    tr["arrival_us"] = np.arange(n, dtype=np.int64) * 150_000
    tr["in_tokens"] = 16
    tr["out_tokens"] = 65535
    classes = gen.make_classes([(None, None, None)])
    off, inst = gen.candidates_from_lists([[(0, 0, 1)], [(0, 1, 2)]])
    want = oracle_mod.eval_placements(prof, tr, classes, off, inst, 4)
    got, _ = gpu_eval(ctx, prof, tr, classes, off, inst, 4)
    assert int(want["n_served"][0]) == n and int(want["tokens_out"][0]) == n * 65535 > 2 ** 32
    assert_records_equal(got, want, "counter wrap")


def test_api_errors(ctx):
    import paper_2509_06362_b200 as m
    cfg = gen.make_config("tiny")
    ctx.load_profile(cfg["profile"])
    bad = cfg["traces"][0].copy()
    bad["arrival_us"][5] = bad["arrival_us"][4] - 1
    with pytest.raises(m.MaasoError):
        ctx.load_trace(bad, cfg["classes"])
    bad = cfg["traces"][0].copy()
    bad["model"][0] = 3
    with pytest.raises(m.MaasoError):
        ctx.load_trace(bad, cfg["classes"])
    bad = cfg["traces"][0].copy()
    bad["cls"][0] = 9
    with pytest.raises(m.MaasoError):
        ctx.load_trace(bad, cfg["classes"])
    bad = cfg["traces"][0].copy()
    bad["out_tokens"][0] = 0
    with pytest.raises(m.MaasoError):
        ctx.load_trace(bad, cfg["classes"])
    p = dict(cfg["profile"])
    p["step_us"] = cfg["profile"]["step_us"].copy()
    p["step_us"][0, 0, 3] = 0
    with pytest.raises(m.MaasoError):
        ctx.load_profile(p)
    fresh = m.Context(0)
    with pytest.raises(m.MaasoError):
        fresh.load_trace(cfg["traces"][0], cfg["classes"])    # no profile yet
    fresh.close()
    # a device-resident trace loads as well
    import torch
    ctx.load_profile(cfg["profile"])
    dev = torch.from_numpy(cfg["traces"][0].view(np.uint8)).cuda()
    t = ctx.load_trace(dev, cfg["classes"])
    assert t.n == 500
    ctx.free_trace(t)


@pytest.mark.parametrize("mapping", MAPPINGS)
def test_ttft_histogram_and_percentiles(ctx, oracle_mod, mapping):
    import torch
    cfg = gen.make_config("multimodel", n_cand=400, n_req=3000)
    tr = cfg["traces"][0]
    lists = [[(2, 0, 4)], []]                       # an invalid candidate and the empty placement
    off2, inst2 = gen.candidates_from_lists(lists)
    off = np.concatenate([cfg["offsets"], cfg["offsets"][-1] + off2[1:]]).astype(np.uint32)
    inst = np.concatenate([cfg["inst"], inst2]).astype(np.uint32)
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(tr, cfg["classes"])
    n_cand = len(off) - 1
    hist = torch.full((n_cand, 64), 77, dtype=torch.int32, device="cuda")
    out = ctx.eval_placements(t, ctx.to_device(off), ctx.to_device(inst), 32, mapping=mapping, ttft_hist=hist)
    pct = ctx.ttft_percentiles(hist, [500, 950, 990, 1000])
    torch.cuda.synchronize()
    want = oracle_mod.ttft_hist(cfg["profile"], tr, cfg["classes"], off, inst, 32)
    got = hist.cpu().numpy().view(np.uint32)
    assert (got == want).all(), np.nonzero((got != want).any(axis=1))[0][:5]
    rec = ctx.results_to_numpy(out)
    assert (got.sum(axis=1) == rec["n_served"]).all()
    assert (pct.cpu().numpy() == oracle_mod.ttft_percentiles(want, [500, 950, 990, 1000])).all()
    ctx.free_trace(t)


def test_ttft_histogram_bin_edges_on_gpu(ctx, oracle_mod):
    """The hand-worked bin edges of the oracle's pin, through the CUDA path."""
    import torch
    from test_oracle_pins import TTFT_BIN_EDGES, _prefill_only_profile, NONE3
    prof = _prefill_only_profile([b for b, _ in TTFT_BIN_EDGES])
    trace = np.zeros(1, dtype=gen.REQUEST_DTYPE)
    trace["arrival_us"], trace["in_tokens"], trace["out_tokens"] = 5, 100, 2
    offsets, inst = gen.candidates_from_lists([[(0, s, 1)] for s in range(len(TTFT_BIN_EDGES))])
    for mapping in MAPPINGS:
        ctx.load_profile(prof)
        t = ctx.load_trace(trace, gen.make_classes(NONE3))
        hist = torch.zeros((len(TTFT_BIN_EDGES), 64), dtype=torch.int32, device="cuda")
        ctx.eval_placements(t, ctx.to_device(offsets), ctx.to_device(inst), 4, mapping=mapping, ttft_hist=hist)
        torch.cuda.synchronize()
        got = hist.cpu().numpy()
        for c, (_, want_bin) in enumerate(TTFT_BIN_EDGES):
            assert np.nonzero(got[c])[0].tolist() == [want_bin] and got[c, want_bin] == 1, (mapping, c)
        ctx.free_trace(t)


# ---- the engine that fixes the decode speed at admission (flag 2) ----------------------------
@pytest.mark.parametrize("flags", [2, 3, 8, 9, 10])
def test_frozen_engine_tiny_config_full(ctx, oracle_mod, flags):
    cfg = gen.make_config("tiny")
    tr = cfg["traces"][0]
    idx = np.arange(0, 143, 5, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"],
                                          cfg["budget"], None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"], cfg["budget"],
                       None, flags, 0, dump_idx=idx)
    assert_records_equal(got, want, "tiny, fixed-speed engine")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k
    assert int(want["n_served"].sum()) > 0 and int(want["n_rejected"].sum()) > 0
    if flags & 8:       # queues at the instances: one distributor round per request, and some requests did wait
        assert (want["attempts"] == want["n_counted"]).all()
        plain = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], cfg["offsets"], cfg["inst"],
                                           cfg["budget"], None, (flags & 1) | 2)
        assert int((plain["attempts"] > plain["n_counted"]).sum()) > 0


@pytest.mark.parametrize("flags", [2, 3, 8, 9])
def test_frozen_engine_node_and_multimodel_subsets(ctx, oracle_mod, flags):
    # ragged trace length (tiles of 64 + a tail), every group width up to 32 lanes, class masks, dumps
    cfg = gen.make_config("node", n_req=1777)
    sel = np.arange(0, 10864, 29)
    off = np.zeros(len(sel) + 1, dtype=np.uint32)
    parts = []
    for k, c in enumerate(sel):
        parts.append(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        off[k + 1] = off[k] + len(parts[-1])
    inst = np.concatenate(parts).astype(np.uint32)
    tr = cfg["traces"][0]
    idx = np.arange(0, len(sel), 41, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 8, None, flags, 0, dump_idx=idx)
    assert_records_equal(got, want, "node subset, fixed-speed engine")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k

    cfg = gen.make_config("multimodel", n_cand=500, n_req=3000)
    n_i = np.diff(cfg["offsets"])
    keep = np.nonzero(n_i <= 32)[0]
    off = np.zeros(len(keep) + 1, dtype=np.uint32)
    parts = []
    for k, c in enumerate(keep):
        parts.append(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        off[k + 1] = off[k] + len(parts[-1])
    inst = np.concatenate(parts).astype(np.uint32)
    mask = np.random.default_rng(5).integers(1, 8, size=len(keep)).astype(np.uint32)
    tr = cfg["traces"][0]
    want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 32, mask, flags)
    got, _ = gpu_eval(ctx, cfg["profile"], tr, cfg["classes"], off, inst, 32, mask, flags, 0)
    assert_records_equal(got, want, "multimodel subset, fixed-speed engine")


def test_frozen_engine_limits(ctx):
    """No block mapping for this engine; more than 128 instances are refused, placement by placement."""
    import paper_2509_06362_b200 as m
    cfg = gen.make_config("tiny", n_req=50)
    ctx.load_profile(cfg["profile"])
    t = ctx.load_trace(cfg["traces"][0], cfg["classes"])
    d_off, d_inst = ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"])
    with pytest.raises(m.MaasoError):
        ctx.eval_placements(t, d_off, d_inst, 4, flags=2, mapping=1)
    with pytest.raises(m.MaasoError):
        ctx.eval_placements(t, d_off, d_inst, 4, flags=8, mapping=1)
    off, inst = gen.candidates_from_lists([[(0, 0, 1)] * 129, [(0, 0, 1)] * 33, [(0, 0, 1)] * 32])
    import torch
    out = ctx.eval_placements(t, ctx.to_device(off), ctx.to_device(inst), 256, flags=2)
    torch.cuda.synchronize()
    rec = ctx.results_to_numpy(out)
    assert int(rec["status"][0]) == m.CAND_STATUS["ETOOMANY"]          # the limit is 128 instances, for every engine
    assert int(rec["status"][1]) == 0 and int(rec["status"][2]) == 0
    ctx.free_trace(t)


@pytest.mark.parametrize("flags", [2, 8])
def test_fixed_speed_engine_time_limit_flags_one_placement_only(ctx, oracle_mod, flags):
    """Finish times of the fixed-speed engine must stay below 2^57 us.  A placement that passes the
    limit (two one-slot instances, no SLO limits, a long run of requests of the largest cost the
    tables allow, each starting when a slot frees) comes back with ELOOP and a zeroed record; the
    flag is raised by one lane of its group in the middle of the trace, and the placements that share
    its warp must be scored as if nothing had happened."""
    import paper_2509_06362_b200 as m
    prof = gen.profile_tiny()
    prof["prefill_base_us"] = prof["prefill_base_us"].copy()
    prof["prefill_q16"] = prof["prefill_q16"].copy()
    prof["step_us"] = prof["step_us"].copy()
    prof["prefill_base_us"][0, 2] = 2 ** 31 - 1      # strategy 2 is as slow as the tables allow
    prof["prefill_q16"][0, 2] = 2 ** 31 - 1
    prof["step_us"][0, 2, :] = 2 ** 30
    classes = gen.make_classes([(None, None, None)])
    n = 3000
    tr = np.zeros(n, dtype=gen.REQUEST_DTYPE)
    tr["arrival_us"] = np.arange(n)
    tr["in_tokens"] = 2 ** 32 - 1
    tr["out_tokens"] = 65535
    lists = [[(0, 2, 1), (0, 2, 1)], [(0, 0, 4), (0, 1, 2)], [(0, 0, 1)], [(0, 1, 8), (0, 1, 8)], [(0, 2, 1), (0, 0, 2)]]
    off, inst = gen.candidates_from_lists(lists)
    got, _ = gpu_eval(ctx, prof, tr, classes, off, inst, 64, None, flags, 2)
    want = oracle_mod.eval_placements(prof, tr, classes, off, inst, 64, None, flags)
    assert int(got["status"][0]) == m.CAND_STATUS["ELOOP"]
    assert got[0].tobytes()[4:] == bytes(124)                  # nothing but the status
    assert (want["status"] == 0).all()                        # the oracle has no such limit
    assert_records_equal(got[1:], want[1:], "placements beside the flagged one")


@pytest.mark.parametrize("flags", [0, 1, 2, 3, 4, 5, 8, 13])
def test_slot_keys_in_global_scratch_when_the_pool_is_too_small(oracle_mod, flags):
    """A context created with MAASO_GROUP_BLOCKS=8 leaves no shared memory for the key pool, so
    every lane keeps its slot keys in global scratch: same results."""
    import os
    import paper_2509_06362_b200 as m
    old = os.environ.get("MAASO_GROUP_BLOCKS")
    os.environ["MAASO_GROUP_BLOCKS"] = "8"
    try:
        c = m.Context(0)
    finally:
        if old is None:
            del os.environ["MAASO_GROUP_BLOCKS"]
        else:
            os.environ["MAASO_GROUP_BLOCKS"] = old
    try:
        cfg = gen.make_config("multimodel", n_cand=300, n_req=2000)
        keep = np.nonzero(np.diff(cfg["offsets"]) <= 32)[0]
        off = np.zeros(len(keep) + 1, dtype=np.uint32)
        parts = []
        for k, cand in enumerate(keep):
            parts.append(cfg["inst"][cfg["offsets"][cand]:cfg["offsets"][cand + 1]])
            off[k + 1] = off[k] + len(parts[-1])
        inst = np.concatenate(parts).astype(np.uint32)
        tr = cfg["traces"][0]
        want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 32, None, flags)
        got, _ = gpu_eval(c, cfg["profile"], tr, cfg["classes"], off, inst, 32, None, flags, 0)
        assert_records_equal(got, want, "keys in global scratch")
    finally:
        c.close()


# ---- TBT term of the hit test on the largest token gap (flag 4) -------------------------------
@pytest.mark.parametrize("flags", [4, 5, 6, 7, 12])
def test_largest_gap_hit_test(ctx, oracle_mod, flags):
    """Default and fixed-speed engine, with and without the optimistic estimate; limits tight
    enough for prefill stalls to matter; every group width; ragged trace; dumps."""
    tight = gen.make_classes([(500_000, 14_000, None), (2_000_000, 30_000, None), (None, 60_000, 180_000_000)])
    cfg = gen.make_config("node", n_req=1777)
    sel = np.arange(0, 10864, 31)
    off = np.zeros(len(sel) + 1, dtype=np.uint32)
    parts = []
    for k, c in enumerate(sel):
        parts.append(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        off[k + 1] = off[k] + len(parts[-1])
    inst = np.concatenate(parts).astype(np.uint32)
    tr = cfg["traces"][0]
    idx = np.arange(0, len(sel), 43, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(cfg["profile"], tr, tight, off, inst, 8, None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, cfg["profile"], tr, tight, off, inst, 8, None, flags, 0, dump_idx=idx)
    assert_records_equal(got, want, "node subset, largest-gap test")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k
    mean_form = oracle_mod.eval_placements(cfg["profile"], tr, tight, off, inst, 8, None, flags & ~4)
    if not flags & 10:
        assert int((mean_form["n_hit"] - want["n_hit"]).sum()) > 0     # the option changes something here

    cfg = gen.make_config("multimodel", n_cand=400, n_req=2500)
    keep = np.nonzero(np.diff(cfg["offsets"]) <= 32)[0]
    off = np.zeros(len(keep) + 1, dtype=np.uint32)
    parts = []
    for k, c in enumerate(keep):
        parts.append(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        off[k + 1] = off[k] + len(parts[-1])
    inst = np.concatenate(parts).astype(np.uint32)
    mask = np.random.default_rng(6).integers(1, 8, size=len(keep)).astype(np.uint32)
    tight3 = gen.make_classes([(500_000, 60_000, None), (2_000_000, 150_000, None), (None, 300_000, 180_000_000)])
    tr = cfg["traces"][0]
    want = oracle_mod.eval_placements(cfg["profile"], tr, tight3, off, inst, 32, mask, flags)
    got, _ = gpu_eval(ctx, cfg["profile"], tr, tight3, off, inst, 32, mask, flags, 0)
    assert_records_equal(got, want, "multimodel subset, largest-gap test")


@pytest.mark.parametrize("flags", [4, 5])
def test_largest_gap_when_the_list_of_stretch_gaps_overflows(ctx, oracle_mod, flags):
    """Forty admissions whose stalls shrink one after the other while everybody keeps running: the lane's
    list of stretch gaps (16 entries, decreasing) fills up and its oldest entries must be folded into
    the slots.  Limits chosen so that the hit counts depend on each request's exact largest gap.  Also
    with other placements in the same warp and with a second, smaller instance."""
    prof = gen.make_config("tiny")["profile"]
    trace = gen.shrinking_prompts_trace(n_classes=24)
    classes = gen.make_classes([(None, 18_600 + 150 * c, None) for c in range(24)])   # a limit every 150 us
    off, inst = gen.candidates_from_lists([[(0, 0, 64)], [(0, 0, 64), (0, 0, 8)], [(0, 0, 48)], [(0, 0, 40), (0, 0, 24)]])
    idx = np.arange(4, dtype=np.uint32)
    want, wd = oracle_mod.eval_placements(prof, trace, classes, off, inst, 4, None, flags, dump_idx=idx)
    got, gd = gpu_eval(ctx, prof, trace, classes, off, inst, 4, None, flags, 0, dump_idx=idx)
    assert_records_equal(got, want, "shrinking stalls")
    for k in wd:
        assert (gd[k] == wd[k]).all(), k
    assert int(want["n_served"][0]) == 41 and 5 < int(want["n_hit"][0]) < 36


# ---- several traces in one pass ----------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, 1, 2, 4, 8])
def test_several_traces_in_one_pass(ctx, oracle_mod, flags):
    """The bursty load sweep, cut down: the candidate set against 5 traces of different rates and
    lengths in one call; every block of records must equal the oracle's for that trace, and so must
    the per-model rejection counts and the histograms."""
    import torch
    cfg = gen.make_config("bursty", n_req=1500)
    sel = np.arange(0, 10864, 37)
    off = np.zeros(len(sel) + 1, dtype=np.uint32)
    parts = []
    for k, c in enumerate(sel):
        parts.append(cfg["inst"][cfg["offsets"][c]:cfg["offsets"][c + 1]])
        off[k + 1] = off[k] + len(parts[-1])
    inst = np.concatenate(parts).astype(np.uint32)
    traces_np = [cfg["traces"][j][: 1500 - 211 * i] for i, j in enumerate((0, 5, 9, 13, 15))]   # ragged lengths
    ctx.load_profile(cfg["profile"])
    handles = [ctx.load_trace(t, cfg["classes"]) for t in traces_np]
    n_cand, n_tr = len(sel), len(handles)
    mask = np.random.default_rng(9).integers(1, 8, size=n_cand).astype(np.uint32)
    rbm = torch.full((n_tr * n_cand, 16), 77, dtype=torch.int32, device="cuda")
    hist = torch.full((n_tr * n_cand, 64), 77, dtype=torch.int32, device="cuda")
    out = ctx.eval_placements_multi(handles, ctx.to_device(off), ctx.to_device(inst), 8, ctx.to_device(mask), flags,
                                    rejected_by_model=rbm, ttft_hist=hist)
    torch.cuda.synchronize()
    got = ctx.results_to_numpy(out).reshape(n_tr, n_cand)
    rbm_h = rbm.cpu().numpy().view(np.uint32).reshape(n_tr, n_cand, 16)
    hist_h = hist.cpu().numpy().view(np.uint32).reshape(n_tr, n_cand, 64)
    for t, tr in enumerate(traces_np):
        want = oracle_mod.eval_placements(cfg["profile"], tr, cfg["classes"], off, inst, 8, mask, flags)
        assert_records_equal(got[t], want, f"trace {t} of the joint pass")
        if flags == 0:
            assert (rbm_h[t] == oracle_mod.rejected_by_model(cfg["profile"], tr, cfg["classes"], off, inst, 8, mask)).all()
            assert (hist_h[t] == oracle_mod.ttft_hist(cfg["profile"], tr, cfg["classes"], off, inst, 8, mask)).all()
    for h in handles:
        ctx.free_trace(h)


@pytest.mark.parametrize("flags", [0, 1])
def test_several_traces_in_one_pass_on_the_thread_kernel(oracle_mod, monkeypatch, flags):
    """Several traces in one pass under both routings of the default mapping: with the routing threshold
    at zero the loaded batch goes to the thread kernel, placements of more than 32 instances included;
    with a threshold out of reach the lane groups take it and one warp per placement replays the large
    ones (no ETOOMANY below 129 instances either way); records, per-model rejection counts and histograms
    must equal the oracle's for every trace."""
    import torch
    import paper_2509_06362_b200 as m
    prof = gen.profile_multimodel(0)
    rng = np.random.default_rng(21)
    lists = []
    for n_i in (33, 40, 128, 5, 1, 64, 9, 2):
        lists.append([(int(rng.integers(2)), 0, int(rng.choice([1, 2, 4, 8, 16, 32, 64]))) for _ in range(n_i)])
    cfg = gen.make_config("multimodel", n_cand=300, n_req=10)
    off, inst = gen.candidates_from_lists(lists)
    off = np.concatenate([off, off[-1] + cfg["offsets"][1:]]).astype(np.uint32)
    inst = np.concatenate([inst, cfg["inst"]]).astype(np.uint32)
    classes = cfg["classes"]
    traces_np = [gen.make_trace(900 - 150 * i, 40.0 * (i + 1), 30 + i, model_mix=(0.6, 0.3, 0.1)) for i in range(3)]
    n_cand, n_tr = len(off) - 1, len(traces_np)
    for min_cand in ("0", "1000000"):        # the whole batch on the thread kernel / only the large placements
        monkeypatch.setenv("MAASO_THREAD_MIN_CAND", min_cand)
        c = m.Context(0)
        c.load_profile(prof)
        handles = [c.load_trace(t, classes) for t in traces_np]
        rbm = torch.full((n_tr * n_cand, 16), 77, dtype=torch.int32, device="cuda")
        hist = torch.full((n_tr * n_cand, 64), 77, dtype=torch.int32, device="cuda")
        c.set_timing(True)
        out = c.eval_placements_multi(handles, c.to_device(off), c.to_device(inst), 1024, None, flags,
                                      rejected_by_model=rbm, ttft_hist=hist)
        torch.cuda.synchronize()
        tm = c.get_timing()
        got = c.results_to_numpy(out).reshape(n_tr, n_cand)
        rbm_h = rbm.cpu().numpy().view(np.uint32).reshape(n_tr, n_cand, 16)
        hist_h = hist.cpu().numpy().view(np.uint32).reshape(n_tr, n_cand, 64)
        for t, tr in enumerate(traces_np):
            want = oracle_mod.eval_placements(prof, tr, classes, off, inst, 1024, None, flags)
            assert (want["status"] == 0).all()
            assert_records_equal(got[t], want, f"trace {t}, routing threshold {min_cand}")
            if flags == 0:
                assert (rbm_h[t] == oracle_mod.rejected_by_model(prof, tr, classes, off, inst, 1024)).all()
                assert (hist_h[t] == oracle_mod.ttft_hist(prof, tr, classes, off, inst, 1024)).all()
        if min_cand == "0":
            assert tm["thread_ms"] > 0.5 and tm["block_ms"] < 0.5      # everything on the thread kernel
        else:
            assert tm["thread_ms"] < 0.5 and tm["block_ms"] > 0.5      # lane groups + one warp per large placement
        c.close()


def test_several_traces_limits(ctx):
    import paper_2509_06362_b200 as m
    cfg = gen.make_config("tiny", n_req=60)
    ctx.load_profile(cfg["profile"])
    a = ctx.load_trace(cfg["traces"][0], cfg["classes"])
    other = gen.make_classes([(1_000_000, None, None)] * 3)
    b = ctx.load_trace(cfg["traces"][0], other)
    d_off, d_inst = ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"])
    with pytest.raises(m.MaasoError):          # different SLO class tables
        ctx.eval_placements_multi([a, b], d_off, d_inst, 4)
    with pytest.raises(m.MaasoError):          # more than 16 traces
        ctx.eval_placements_multi([a] * 17, d_off, d_inst, 4)
    ctx.free_trace(a)
    ctx.free_trace(b)


def test_refused_scratch_allocation_is_reported_and_survived(oracle_mod):
    """Host-side failure path: the context's scratch growth is refused (test hook, as if the device
    were out of memory).  The call returns MAASO_ENOMEM and enqueues nothing; the same context then
    scores the same batch correctly, a larger one too, and holds no more device memory than a context
    that never saw a failure."""
    import torch
    import paper_2509_06362_b200 as m
    cfg = gen.make_config("node", n_cand=2000, n_req=600)
    want = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"], cfg["inst"], 8)

    def used_by(fail_first):
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        c = m.Context(0)
        c.load_profile(cfg["profile"])
        t = c.load_trace(cfg["traces"][0], cfg["classes"])
        d_off, d_inst = c.to_device(cfg["offsets"][:501]), c.to_device(cfg["inst"][:int(cfg["offsets"][500])])
        out = torch.full((500, 128), 0xAB, dtype=torch.uint8, device="cuda")
        if fail_first:
            c.test_fail_allocs(1)
            with pytest.raises(m.MaasoError) as err:
                c.eval_placements(t, d_off, d_inst, 8, out=out)
            assert err.value.code == -3
            torch.cuda.synchronize()
            assert bool((out == 0xAB).all())                      # nothing was enqueued
            idx = torch.empty(8, dtype=torch.int32, device="cuda")
            c.test_fail_allocs(1)
            with pytest.raises(m.MaasoError) as err:
                c.topk(out, 8)                                    # the ranking's scratch is refused as well
            assert err.value.code == -3
        got = c.eval_placements(t, d_off, d_inst, 8, out=out)
        torch.cuda.synchronize()
        assert c.results_to_numpy(got).tobytes() == want[:500].tobytes()
        big = c.eval_placements(t, c.to_device(cfg["offsets"]), c.to_device(cfg["inst"]), 8)   # grows the scratch
        c.topk(big, 8)
        torch.cuda.synchronize()
        assert c.results_to_numpy(big).tobytes() == want.tobytes()
        used = free0 - torch.cuda.mem_get_info()[0]
        c.close()
        return used

    clean = used_by(False)
    assert used_by(True) <= clean

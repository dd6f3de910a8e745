"""Randomised differential test: small seeded workloads of every shape the entry point takes (placement
sizes from 1 to 128 instances, class tables with and without limits, request subsets, single-token
requests, every engine flag, every mapping the flag allows) through the C ABI and through the oracle,
records and per-request times compared bit for bit.  The fixed cases elsewhere pin known corners; this
one looks for the corners nobody thought of."""
import numpy as np
import pytest

import gen
from gpu_common import gpu_eval, assert_records_equal

pytestmark = pytest.mark.gpu

FLAGS = [0, 1, 2, 3, 4, 5, 6, 8, 9, 12]


@pytest.fixture(scope="module")
def ctx():
    import paper_2509_06362_b200 as m
    c = m.Context(0)
    yield c
    c.close()


def _case(seed):
    rng = np.random.default_rng(1000 + seed)
    prof = gen.profile_multimodel(int(rng.integers(3)))
    n_models, n_strat = prof["n_models"], prof["n_strategies"]
    dev, min_dev = np.asarray(prof["devices"]), np.asarray(prof["min_devices"])
    sizes = [1, 2, 3, 5, 8, 9, 16, 17, 31, 32, 33, 40, 64, 100, 128]
    lists = []
    for _ in range(int(rng.integers(20, 60))):
        n_i = int(rng.choice(sizes, p=np.array([6, 6, 6, 6, 5, 5, 4, 4, 3, 3, 2, 2, 1, 1, 1]) / 55))
        lst = []
        for _ in range(n_i):
            m = int(rng.integers(n_models))
            ok = np.nonzero(dev >= min_dev[m])[0]
            s = int(rng.choice(ok))
            lst.append((m, s, int(rng.choice([1, 2, 3, 4, 7, 8, 9, 16, 31, 32, 33, 64]))))
        lists.append(lst)
    off, inst = gen.candidates_from_lists(lists)
    n_cls = int(rng.choice([1, 3, 4, 9, 40]))
    rows = []
    for _ in range(n_cls):
        kind = int(rng.integers(4))
        ttft = None if kind == 2 else int(rng.choice([200_000, 500_000, 2_000_000, 30_000_000]))
        tbt = None if kind >= 2 else int(rng.choice([15_000, 40_000, 60_000, 150_000]))
        e2e = None if kind == 0 else int(rng.choice([20_000_000, 180_000_000, 600_000_000]))
        rows.append((ttft, tbt, e2e))
    classes = gen.make_classes(rows)
    mm = rng.dirichlet(np.ones(n_models))
    cm = rng.dirichlet(np.ones(n_cls))
    tr = gen.make_trace(int(rng.integers(300, 1800)), float(rng.choice([5.0, 40.0, 300.0])), 77 + seed,
                        model_mix=tuple(mm), class_mix=tuple(cm), cv=float(rng.choice([1.0, 3.0])),
                        doc_class=None if n_cls < 3 else 2)
    tr["out_tokens"][rng.random(len(tr)) < 0.08] = 1
    mask = None
    if n_cls <= 32 and rng.random() < 0.5:
        mask = rng.integers(1, 1 << n_cls, size=len(lists), dtype=np.uint64).astype(np.uint32)
    return prof, off, inst, classes, tr, mask


@pytest.mark.parametrize("seed", range(24))
def test_random_case_every_engine_and_mapping(ctx, oracle_mod, seed):
    prof, off, inst, classes, tr, mask = _case(seed)
    n_cand = len(off) - 1
    idx = np.array(sorted({0, n_cand // 2, n_cand - 1}), dtype=np.uint32)
    rng = np.random.default_rng(seed)
    for flags in [0, 1] + list(rng.choice(FLAGS[2:], size=3, replace=False)):
        flags = int(flags)
        want, wd = oracle_mod.eval_placements(prof, tr, classes, off, inst, 1024, mask, flags, dump_idx=idx)
        mappings = [0, 2, 3, 1] if flags < 2 else [0, 2]
        for mapping in mappings:
            got, gd = gpu_eval(ctx, prof, tr, classes, off, inst, 1024, mask, flags, mapping, dump_idx=idx)
            assert_records_equal(got, want, f"seed {seed}, flags {flags}, mapping {mapping}")
            for k in wd:
                assert (gd[k] == wd[k]).all(), (seed, flags, mapping, k)


@pytest.mark.parametrize("seed", range(6))
def test_random_case_several_traces_in_one_pass(oracle_mod, seed, monkeypatch):
    """The same kind of workload against three traces in one call, under both routings of the default
    mapping (the thread kernel takes the loaded part of the batch / only what the lane groups cannot)."""
    import torch
    import paper_2509_06362_b200 as m
    prof, off, inst, classes, tr, mask = _case(100 + seed)
    n = len(tr)
    traces_np = [tr[: n // 2].copy(), tr[n // 3:].copy(), tr.copy()]
    for t in traces_np:
        t["arrival_us"] -= t["arrival_us"][0]
    rng = np.random.default_rng(seed)
    for min_cand in ("0", "1000000"):
        monkeypatch.setenv("MAASO_THREAD_MIN_CAND", min_cand)
        c = m.Context(0)
        c.load_profile(prof)
        handles = [c.load_trace(t, classes) for t in traces_np]
        d_mask = None if mask is None else c.to_device(mask)
        for flags in (0, int(rng.choice([1, 2, 4, 8]))):
            mappings = [0, 2, 3] if flags < 2 else [0, 2]
            want = [oracle_mod.eval_placements(prof, t, classes, off, inst, 1024, mask, flags) for t in traces_np]
            for mapping in mappings:
                out = c.eval_placements_multi(handles, c.to_device(off), c.to_device(inst), 1024, d_mask, flags,
                                              mapping=mapping)
                torch.cuda.synchronize()
                got = c.results_to_numpy(out).reshape(len(traces_np), -1)
                for k in range(len(traces_np)):
                    assert_records_equal(got[k], want[k], f"seed {seed}, trace {k}, flags {flags}, mapping {mapping}, "
                                                          f"routing threshold {min_cand}")
        c.close()

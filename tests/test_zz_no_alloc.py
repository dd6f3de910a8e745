"""maaso_topk_noalloc: the top-k variant for callers that cannot allocate device memory
(code running under a memory pool that owns the device, or a serving loop that must not
synchronise on an allocation).  Its scratch is a fixed array inside the library, so this
test checks, through the C ABI, that it returns exactly what maaso_topk and the CPU oracle's
ranking return, twice in a row on different inputs (the second call reuses whatever the first
left in the array), at the full capacity it was sized for, without changing the amount of free
device memory, and that sizes beyond the fixed capacity are refused.  Collected last on purpose."""
import numpy as np
import pytest

import gen

pytestmark = pytest.mark.gpu


def _records(seed, n):
    rng = np.random.default_rng(seed)
    rec = np.zeros(n, dtype=gen.RESULT_DTYPE)
    rec["status"] = (rng.random(n) < 0.02) * 8
    rec["n_hit"] = rng.integers(0, 40, n)            # many ties on hits
    rec["n_served"] = rng.integers(0, 50, n)
    rec["sum_ttft_us"] = rng.integers(0, 1 << 40, n) * (rec["n_served"] > 0)
    rec["n_counted"] = 50
    return rec


def test_no_alloc_topk_matches_topk_twice(oracle_mod):
    import torch
    import paper_2509_06362_b200 as m
    ctx = m.Context(0)
    for call, (seed, n, k) in enumerate([(1, 70_000, 64), (2, 9_001, 17)]):
        rec = _records(seed, n)
        dev = torch.from_numpy(rec.view(np.uint8).reshape(n, 128)).cuda()
        want_idx, want_rec = ctx.topk(dev, k)
        got_idx = torch.full((k,), -7, dtype=torch.int32, device="cuda")
        got_rec = torch.empty((k, 128), dtype=torch.uint8, device="cuda")
        rc = m.maaso_topk_noalloc(dev, n, k, got_idx, got_rec)
        torch.cuda.synchronize()
        assert rc == 0, f"call {call}: {m.maaso_strerror(rc)}"
        assert torch.equal(got_idx, want_idx), f"call {call}: indices differ"
        assert torch.equal(got_rec, want_rec), f"call {call}: records differ"
        want = oracle_mod.topk(rec, k)
        assert got_idx.cpu().numpy().view(np.uint32).tolist() == want.tolist(), f"call {call}: oracle ranking differs"
    ctx.close()


def test_no_alloc_topk_at_full_capacity_leaves_free_memory_alone(oracle_mod):
    """The largest input the fixed array was sized for (three selection passes, both halves of the
    array in use); the amount of free device memory is the same before and after the calls."""
    import torch
    import paper_2509_06362_b200 as m
    n, k = m.NOALLOC_MAX_CAND, m.NOALLOC_MAX_K
    rec = _records(3, n)
    dev = torch.from_numpy(rec.view(np.uint8).reshape(n, 128)).cuda()
    got_idx = torch.full((k,), -7, dtype=torch.int32, device="cuda")
    got_rec = torch.empty((k, 128), dtype=torch.uint8, device="cuda")
    assert m.maaso_topk_noalloc(dev, n, k, got_idx, got_rec) == 0    # first call: the device code is loaded by now
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    assert m.maaso_topk_noalloc(dev, n, k, got_idx, got_rec) == 0
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    want = oracle_mod.topk(rec, k)
    assert got_idx.cpu().numpy().view(np.uint32).tolist() == want.tolist()
    assert got_rec.cpu().numpy().tobytes() == rec[want].tobytes()


def test_no_alloc_topk_refuses_sizes_beyond_its_capacity():
    import torch
    import paper_2509_06362_b200 as m
    dev = torch.zeros((16, 128), dtype=torch.uint8, device="cuda")
    idx = torch.full((128,), -7, dtype=torch.int32, device="cuda")
    assert m.maaso_topk_noalloc(dev, 16, m.NOALLOC_MAX_K + 1, idx) == -5
    assert m.maaso_topk_noalloc(dev, m.NOALLOC_MAX_CAND + 1, 8, idx) == -5
    torch.cuda.synchronize()
    assert (idx == -7).all()            # a refused call writes nothing
    assert "capacity" in m.maaso_strerror(-5)

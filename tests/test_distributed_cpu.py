"""World-size-2 and -3 gloo tests (CPU) of the sharding and gather/merge logic of the multi-GPU path.
The ranking functions are injected: here the oracle's, on the GPU machine maaso_topk."""
import os
import socket
import sys

import numpy as np
import pytest

import gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, k, out_dir):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2509_06362_b200.distributed import sharded_topk
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = gen.make_config("tiny")
    mask = _masks()

    def score_shard(off, inst, m):          # the scoring is injected: here the oracle's
        local = oracle.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], off, inst, cfg["budget"], m)
        if rank == 1:
            local["status"][3] = 8          # an invalid candidate in one shard
        return torch.from_numpy(local.view(np.uint8).reshape(-1, 128).copy())

    def topk_cpu(rec_t, kk):
        rec = rec_t.numpy().reshape(-1).view(gen.RESULT_DTYPE)
        idx = oracle.topk(rec, kk).astype(np.int64)
        pad = np.full(kk, -1, dtype=np.int64)
        pad[:len(idx)] = idx
        out = np.zeros(kk, dtype=gen.RESULT_DTYPE)
        out[:len(idx)] = rec[idx]
        return torch.from_numpy(pad.astype(np.int32)), torch.from_numpy(out.view(np.uint8).reshape(kk, 128).copy())

    order, rec, (lo, hi), _ = sharded_topk(score_shard, topk_cpu, topk_cpu, cfg["offsets"], cfg["inst"], k, mask)
    if rank == 0:
        np.save(os.path.join(out_dir, "order.npy"), np.asarray(order, dtype=np.int64))
        np.save(os.path.join(out_dir, "rec.npy"), rec.numpy())
    np.save(os.path.join(out_dir, f"shard{rank}.npy"), np.asarray([lo, hi]))
    dist.barrier()
    dist.destroy_process_group()


def _masks():
    return np.random.default_rng(11).integers(1, 8, size=143).astype(np.uint32)


@pytest.mark.parametrize("world,k", [(2, 8), (2, 100), (3, 64), (3, 1024)])
def test_sharded_topk_equals_single_rank(tmp_path, oracle_mod, world, k):
    """One sweep sharded over 2 and 3 ranks (143 candidates: uneven shards), class masks sharded with
    it, k up to the library's maximum (world * k beyond what one ranking call returns)."""
    import torch.multiprocessing as mp
    mp.spawn(_worker, args=(world, _free_port(), k, str(tmp_path)), nprocs=world, join=True)
    cfg = gen.make_config("tiny")
    full = oracle_mod.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"],
                                      cfg["inst"], cfg["budget"], _masks())
    from paper_2509_06362_b200.distributed import shard_range
    lo1, _ = shard_range(143, 1, world)
    full["status"][lo1 + 3] = 8
    want = oracle_mod.topk(full, k).tolist()
    got = np.load(tmp_path / "order.npy").tolist()
    assert got == want[:len(got)] and len(got) == min(k, 143)
    rec = np.load(tmp_path / "rec.npy").reshape(-1).view(gen.RESULT_DTYPE)
    assert rec.tobytes() == full[want[:len(got)]].tobytes()
    cuts = [np.load(tmp_path / f"shard{r}.npy").tolist() for r in range(world)]
    assert cuts == [list(shard_range(143, r, world)) for r in range(world)]
    sizes = [h - l for l, h in cuts]
    assert sum(sizes) == 143 and (world == 2 or len(set(sizes)) == 2)     # 143 = 48 + 48 + 47


def test_shard_ranges_partition():
    from paper_2509_06362_b200.distributed import shard_range, shard_csr
    for n in (0, 1, 7, 143, 10864):
        for world in (1, 2, 3, 8):
            cuts = [shard_range(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            assert max(h - l for l, h in cuts) - min(h - l for l, h in cuts) <= 1
    off, inst = gen.enumerate_tiny()
    o2, i2 = shard_csr(off, inst, 10, 20)
    assert o2[0] == 0 and len(o2) == 11 and (i2 == inst[off[10]:off[20]]).all()

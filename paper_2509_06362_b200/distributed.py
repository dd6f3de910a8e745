"""Multi-GPU use of the scoring path: candidates are independent, so they are sharded over
ranks in contiguous index ranges, every rank scores its shard on its own GPU (trace and
latency tables are replicated by plain copies into each GPU's own memory), selects a local
top-k, and one all-gather of k (index, record) pairs per rank followed by the same exact
ranking over the gathered records gives the global top-k.  Contiguous shards and rank-major
gather order keep ties in global-index order, so the answer equals the single-GPU answer.

Only host logic and torch.distributed plumbing live here; ranking runs in maaso_topk.
"""
import numpy as np

PAD = 0xFFFFFFFF
MAX_MERGE = 1024   # MAASO_MAX_TOPK


def shard_range(n, rank, world):
    """[lo, hi) of the contiguous shard of `n` candidates owned by `rank`."""
    base, rem = divmod(int(n), int(world))
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_csr(offsets, inst, lo, hi):
    """CSR arrays (numpy uint32) of candidates [lo, hi), offsets rebased to 0."""
    off = np.asarray(offsets[lo:hi + 1], dtype=np.int64)
    return (off - off[0]).astype(np.uint32), np.asarray(inst[off[0]:off[-1]], dtype=np.uint32)


def global_topk(local_topk, merge_topk, results, base, k, group=None):
    """Global top-k of a sharded sweep.

    results: this rank's record tensor [n_local, 128] (uint8), on the device the backend needs.
    base: global index of this rank's first candidate.
    local_topk(results, k) -> (idx int32 tensor [k] with PAD (as -1) padding, rec uint8 [k,128]);
    merge_topk(records [m,128], m) -> (positions int32 [m], rec) ranking the gathered records.
    Returns (global indices as a python list, best first; record tensor [len, 128])."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    idx, rec = local_topk(results, k)
    gidx = idx.to(torch.int64)
    gidx = torch.where(gidx < 0, gidx, gidx + int(base))          # PAD stays negative
    if world > 1:
        if world * k > MAX_MERGE:
            raise ValueError(f"world*k = {world * k} exceeds the merge capacity {MAX_MERGE}")
        all_idx = [torch.empty_like(gidx) for _ in range(world)]
        all_rec = [torch.empty_like(rec) for _ in range(world)]
        dist.all_gather(all_idx, gidx, group=group)
        dist.all_gather(all_rec, rec, group=group)
        gidx, rec = torch.cat(all_idx), torch.cat(all_rec)
    # padding must rank behind every real candidate, scored or not
    status = rec.view(torch.int32)[:, 0]
    status[gidx < 0] = -1
    m = int(gidx.shape[0])
    pos, mrec = merge_topk(rec, m)
    pos = pos.to(torch.int64)
    order = gidx[pos]
    keep = order >= 0
    return order[keep][:k].tolist(), mrec[keep][:k]

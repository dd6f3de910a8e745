"""Multi-GPU use of the scoring path: candidates are independent, so ONE sweep is sharded over
ranks in contiguous index ranges, every rank scores its shard on its own GPU (trace and
latency tables are replicated by plain copies into each GPU's own memory), selects a local
top-k, and one all-gather of k (index, record) pairs per rank followed by the same exact
ranking over the gathered records gives the global top-k.  Contiguous shards and rank-major
gather order keep ties in global-index order, so the answer equals the single-GPU answer.
No peer-memory access and no collective on the data path: the only exchange is the gather of
k records per rank.

Only host logic and torch.distributed plumbing live here; scoring and ranking run in the
library's kernels (injected as callables, so the plumbing can be tested on CPU ranks).
"""
import numpy as np

PAD = 0xFFFFFFFF


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
    """Global top-k of a sharded sweep, two levels: a top-k per rank, then one ranking of the
    world * k gathered records (any world size: the second level asks for k records only).

    results: this rank's record tensor [n_local, 128] (uint8), on the device the backend needs.
    base: global index of this rank's first candidate.
    local_topk(results, k) -> (idx int32 tensor [k] with PAD (as -1) padding, rec uint8 [k,128]);
    merge_topk(records [m,128], kk) -> (positions int32 [kk], rec) ranking the gathered records.
    Returns (global indices as a python list, best first; record tensor [len, 128])."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    idx, rec = local_topk(results, k)
    gidx = idx.to(torch.int64)
    gidx = torch.where(gidx < 0, gidx, gidx + int(base))          # PAD stays negative
    if world > 1:
        all_idx = [torch.empty_like(gidx) for _ in range(world)]
        all_rec = [torch.empty_like(rec) for _ in range(world)]
        dist.all_gather(all_idx, gidx, group=group)
        dist.all_gather(all_rec, rec, group=group)
        gidx, rec = torch.cat(all_idx), torch.cat(all_rec)
    # Padding (ranks with fewer than k candidates) goes behind every real candidate, scored or not:
    # real entries keep their rank-major order (ties in the ranking fall to the lower position, which
    # is the lower global index), padding entries follow and carry a status that marks them unscored.
    pad = gidx < 0
    order = torch.argsort(pad.to(torch.int8), stable=True)
    gidx, rec = gidx[order], rec[order].contiguous()
    rec.view(torch.int32)[:, 0][gidx < 0] = -1
    m = int(gidx.shape[0])
    pos, mrec = merge_topk(rec, min(int(k), m))
    pos = pos.to(torch.int64)
    ok = pos >= 0
    chosen = gidx[pos[ok]]
    keep = chosen >= 0
    return chosen[keep][:k].tolist(), mrec[ok][keep][:k]


def sharded_topk(score_shard, local_topk, merge_topk, offsets, inst, k, class_mask=None, group=None):
    """Score ONE sweep on all ranks and return its global top-k (the same on every rank).

    offsets / inst / class_mask: the FULL candidate batch as numpy arrays, identical on every
    rank.  This rank takes the contiguous shard shard_range(n_cand, rank, world), scores it with
    score_shard(offsets_shard, inst_shard, class_mask_shard or None) -> record tensor
    [n_shard, 128], and the shards' best records are merged by global_topk.
    Returns (global indices, best first; record tensor; (lo, hi) of this rank's shard; its records)."""
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    n = len(offsets) - 1
    lo, hi = shard_range(n, rank, world)
    off, ins = shard_csr(offsets, inst, lo, hi)
    mask = None if class_mask is None else np.ascontiguousarray(class_mask[lo:hi], dtype=np.uint32)
    results = score_shard(off, ins, mask)
    order, rec = global_topk(local_topk, merge_topk, results, lo, k, group=group)
    return order, rec, (lo, hi), results


def sharded_topk_on_gpu(ctx, trace, offsets, inst, budget, k, class_mask=None, flags=0, mapping=0,
                        group=None, stream=None):
    """sharded_topk with the library's kernels: this rank's shard is copied to its GPU, scored by
    maaso_eval_placements and ranked by maaso_topk; `ctx` / `trace` are this rank's context and its
    copy of the trace."""
    def score_shard(off, ins, mask):
        d_off = ctx.to_device(off)
        d_inst = ctx.to_device(ins if len(ins) else np.zeros(1, np.uint32))
        if len(ins) == 0:
            d_inst = d_inst[:0]
        d_mask = None if mask is None else ctx.to_device(mask)
        return ctx.eval_placements(trace, d_off, d_inst, budget, d_mask, flags, mapping, stream=stream)

    def rank_topk(rec, kk):
        return ctx.topk(rec, kk, stream=stream)

    return sharded_topk(score_shard, rank_topk, rank_topk, offsets, inst, k, class_mask, group)

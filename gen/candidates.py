"""Candidate placements: ordered instance lists in CSR form.

offsets[C+1] (uint32) and inst[] (uint32 packed words, see formats.pack_inst).
"""
import itertools
import numpy as np
from .formats import pack_inst


def candidates_from_lists(lists):
    """lists: one list of (model, strategy, batch) tuples per candidate."""
    offsets = np.zeros(len(lists) + 1, dtype=np.uint32)
    words = []
    for c, lst in enumerate(lists):
        for (m, s, b) in lst:
            words.append(int(pack_inst(m, s, b)))
        offsets[c + 1] = len(words)
    return offsets, np.asarray(words, dtype=np.uint32)


def enumerate_tiny():
    """Every non-empty multiset of (tp in {1,2,4}) x (batch in {1,4,8,16}) that fits in
    4 devices: 143 candidates.  Strategy index s has tp = 2**s."""
    types = [(s, b) for s in range(3) for b in (1, 4, 8, 16)]
    cost = {s: 1 << s for s in range(3)}
    out = []
    for size in range(1, 5):
        for combo in itertools.combinations_with_replacement(types, size):
            if sum(cost[s] for s, _ in combo) <= 4:
                out.append([(0, s, b) for s, b in combo])
    return candidates_from_lists(out)


def enumerate_node(devices, budget=8, batches=(1, 2, 4, 8, 16, 32, 64)):
    """Every non-empty multiset of strategies that fits the budget, where instances of
    the same strategy share one batch cap drawn from `batches`."""
    S = len(devices)
    out = []

    def rec(s, left, counts):
        if s == S:
            used = [(k, n) for k, n in enumerate(counts) if n]
            if not used:
                return
            for bs in itertools.product(batches, repeat=len(used)):
                lst = []
                for (k, n), b in zip(used, bs):
                    lst.extend([(0, k, b)] * n)
                out.append(lst)
            return
        n = 0
        while n * int(devices[s]) <= left:
            rec(s + 1, left - n * int(devices[s]), counts + [n])
            n += 1

    rec(0, budget, [])
    return candidates_from_lists(out)


def sample_candidates(n, seed, budget, profile, batches=(1, 2, 4, 8, 16, 32, 64),
                      stop_p=0.125, max_instances=128):
    """Sequential sampler: repeatedly draw uniformly among the (model, strategy, batch)
    types that still fit the remaining budget (and the model's minimum devices), add it,
    and stop with probability stop_p or when nothing fits.  Instances are then sorted by
    (model, strategy, batch); duplicates are allowed."""
    rng = np.random.default_rng(seed)
    dev = np.asarray(profile["devices"], dtype=np.int64)
    mind = np.asarray(profile["min_devices"], dtype=np.int64)
    types = [(m, s, b) for m in range(len(mind)) for s in range(len(dev)) if dev[s] >= mind[m]
             for b in batches]
    types.sort(key=lambda t: (dev[t[1]], t))
    tcost = np.array([dev[t[1]] for t in types], dtype=np.int64)
    tword = np.array([int(pack_inst(*t)) for t in types], dtype=np.uint32)
    tkey = np.array([(t[0] << 16) | (t[1] << 8) | t[2] for t in types], dtype=np.int64)
    fit_count = np.searchsorted(tcost, np.arange(budget + 1), side="right")

    left = np.full(n, budget, dtype=np.int64)
    active = np.ones(n, dtype=bool)
    count = np.zeros(n, dtype=np.int64)
    picks = []            # (candidate ids, type ids) per round
    while active.any():
        ids = np.nonzero(active)[0]
        nfit = fit_count[left[ids]]
        can = (nfit > 0) & (count[ids] < max_instances)
        active[ids[~can]] = False
        ids, nfit = ids[can], nfit[can]
        if ids.size == 0:
            break
        t = (rng.random(ids.size) * nfit).astype(np.int64)
        t = np.minimum(t, nfit - 1)
        picks.append((ids, t))
        left[ids] -= tcost[t]
        count[ids] += 1
        stop = rng.random(ids.size) < stop_p
        active[ids[stop]] = False
    cand = np.concatenate([p[0] for p in picks])
    typ = np.concatenate([p[1] for p in picks])
    order = np.lexsort((tkey[typ], cand))
    cand, typ = cand[order], typ[order]
    offsets = np.zeros(n + 1, dtype=np.uint32)
    offsets[1:] = np.cumsum(np.bincount(cand, minlength=n))
    return offsets, tword[typ]

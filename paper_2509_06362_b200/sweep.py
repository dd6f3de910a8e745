"""Long sweeps in resumable chunks.

A sweep of many placements is scored in contiguous candidate ranges; each range's records are
written to `<out_dir>/chunk_<lo>_<hi>.npy` (atomically: a temporary file renamed when complete),
so a run that was interrupted picks up where it stopped: ranges whose file is present and of the
right size are loaded instead of scored.  The records of a range do not depend on the other
ranges, so the assembled result equals the one-call result byte for byte.

Scoring is a callable (on a GPU machine: Context.eval_placements on the range's CSR arrays); this
module holds only the bookkeeping.
"""
import os

import numpy as np

from .binding import RESULT_DTYPE
from .distributed import shard_csr


def chunk_ranges(n_cand, chunk):
    chunk = max(1, int(chunk))
    return [(lo, min(lo + chunk, int(n_cand))) for lo in range(0, int(n_cand), chunk)]


def _chunk_path(out_dir, lo, hi):
    return os.path.join(out_dir, f"chunk_{lo:09d}_{hi:09d}.npy")


def _load_finished(path, n):
    """Records of a finished range, or None if the file is missing, truncated or of another shape."""
    try:
        rec = np.load(path)
    except Exception:
        return None
    if rec.dtype != RESULT_DTYPE or rec.shape != (n,):
        return None
    return rec


def chunked_sweep(score_chunk, offsets, inst, chunk, out_dir, class_mask=None, on_chunk=None):
    """Score candidates [0, n_cand) in ranges of `chunk`, resuming from the files in out_dir.

    score_chunk(offsets_range, inst_range, class_mask_range or None) -> numpy records [hi - lo].
    on_chunk(lo, hi, resumed) is called after every range (progress reporting).
    Returns (records [n_cand], number of ranges scored now, number of ranges resumed)."""
    os.makedirs(out_dir, exist_ok=True)
    n = len(offsets) - 1
    out = np.zeros(n, dtype=RESULT_DTYPE)
    scored = resumed = 0
    for lo, hi in chunk_ranges(n, chunk):
        path = _chunk_path(out_dir, lo, hi)
        rec = _load_finished(path, hi - lo)
        if rec is None:
            off, ins = shard_csr(offsets, inst, lo, hi)
            mask = None if class_mask is None else np.ascontiguousarray(class_mask[lo:hi], dtype=np.uint32)
            rec = np.ascontiguousarray(score_chunk(off, ins, mask)).reshape(-1).view(RESULT_DTYPE)
            if rec.shape != (hi - lo,):
                raise ValueError(f"range [{lo}, {hi}): scoring returned {rec.shape[0]} records")
            tmp = path + f".{os.getpid()}.tmp"
            with open(tmp, "wb") as f:
                np.save(f, rec)
                f.flush()
                os.fsync(f.fileno())
            os.replace(tmp, path)
            scored += 1
            was_resumed = False
        else:
            resumed += 1
            was_resumed = True
        out[lo:hi] = rec
        if on_chunk is not None:
            on_chunk(lo, hi, was_resumed)
    return out, scored, resumed

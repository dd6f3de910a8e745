"""Helpers for the GPU parity tests: run a workload through the C ABI and through the oracle."""
import numpy as np

import gen


def gpu_eval(ctx, cfg_profile, trace, classes, offsets, inst, budget, class_mask=None, flags=0, mapping=0,
             dump_idx=None):
    """Returns (records as numpy RESULT_DTYPE, dumps dict of numpy arrays or None)."""
    import torch
    ctx.load_profile(cfg_profile)
    tr = ctx.load_trace(trace, classes)
    d_off, d_inst = ctx.to_device(offsets), ctx.to_device(inst if len(inst) else np.zeros(1, np.uint32))
    if len(inst) == 0:
        d_inst = d_inst[:0]
    d_mask = None if class_mask is None else ctx.to_device(class_mask)
    out = ctx.eval_placements(tr, d_off, d_inst, budget, d_mask, flags, mapping, dump_idx)
    torch.cuda.synchronize()
    dumps = None
    if dump_idx is not None:
        out, dumps = out
        dumps = {k: v.cpu().numpy() for k, v in dumps.items()}
    res = ctx.results_to_numpy(out)
    ctx.free_trace(tr)
    return res, dumps


def assert_records_equal(got, want, what=""):
    if got.tobytes() == want.tobytes():
        return
    for name in want.dtype.names:
        bad = np.nonzero(got[name] != want[name])[0] if got[name].ndim == 1 else \
            np.nonzero((got[name] != want[name]).any(axis=1))[0]
        if len(bad):
            c = int(bad[0])
            raise AssertionError(f"{what}: field {name} differs for {len(bad)} candidates; first {c}: "
                                 f"gpu {got[name][c]} oracle {want[name][c]}\n gpu {got[c]}\n cpu {want[c]}")
    raise AssertionError(f"{what}: records differ in padding bytes")

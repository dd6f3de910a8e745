"""ctypes wrapper around the C oracle (test infrastructure, not a product path)."""
import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "maaso_oracle.c")
_SO = os.path.join(_HERE, "libmaaso_oracle.so")

FLAG_PRED_OPTIMISTIC = 1
FLAG_INSTANCE_QUEUES = 8  # requests wait at their instance, not at the dispatcher (implies the fixed-speed engine)
FLAG_TBT_MAXGAP = 4      # hit test on the largest token gap instead of the mean gap
FLAG_ENGINE_FROZEN = 2   # decode speed fixed at admission (see frozen_replay in maaso_oracle.c)
STATUS = {"EBUDGET": 1, "EMEMFIT": 2, "ETOOMANY": 4, "EBADINST": 8, "ETIMEOUT": 16, "ELOOP": 32,
          "EINVARIANT": 0x80000000}

# local copies of the layouts: the oracle shares no code with the CUDA package
_REQ = np.dtype([("arrival_us", "<i8"), ("in_tokens", "<u4"), ("out_tokens", "<u2"),
                 ("cls", "u1"), ("model", "u1")])
_SLO = np.dtype([("ttft_us", "<i8"), ("tbt_us", "<i8"), ("e2e_us", "<i8")])
_RES = np.dtype([("status", "<u4"), ("n_counted", "<u4"), ("n_served", "<u4"), ("n_hit", "<u4"),
                 ("n_rejected", "<u4"), ("n_cascade", "<u4"), ("hit_by_class", "<u4", (8,)),
                 ("sum_ttft_us", "<i8"), ("max_ttft_us", "<i8"), ("sum_e2e_us", "<i8"),
                 ("max_e2e_us", "<i8"), ("makespan_us", "<i8"), ("tokens_out", "<u8"),
                 ("checksum", "<u8"), ("attempts", "<u8"), ("reserved", "<u8")])


class _Profile(C.Structure):
    _fields_ = [("n_models", C.c_uint32), ("n_strategies", C.c_uint32), ("wmax", C.c_uint32),
                ("devices", C.c_void_p), ("min_devices", C.c_void_p),
                ("prefill_base_us", C.c_void_p), ("prefill_q16", C.c_void_p),
                ("step_us", C.c_void_p)]


_lib = None


def build(force=False):
    """Compile the oracle with gcc -O2 (plain C, single thread)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
                               "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_eval_batch.restype = C.c_int
        _lib.orc_topk.restype = C.c_int
        _lib.orc_score.restype = C.c_int
        _lib.orc_topk_scores.restype = C.c_int
        _lib.orc_rejected_by_model.restype = C.c_int
        _lib.orc_ins_deploy.restype = C.c_int
        _lib.orc_partition.restype = C.c_int
        _lib.orc_prune_configs.restype = C.c_int
        _lib.orc_ttft_hist.restype = C.c_int
        _lib.orc_ttft_percentile.restype = C.c_int64
    return _lib


def _ptr(a):
    return C.c_void_p(a.ctypes.data) if a is not None else C.c_void_p(0)


def _profile_struct(profile):
    keep = {k: np.ascontiguousarray(profile[k], dtype=np.int32)
            for k in ("devices", "min_devices", "prefill_base_us", "prefill_q16", "step_us")}
    p = _Profile(int(profile["n_models"]), int(profile["n_strategies"]), int(profile["wmax"]),
                 keep["devices"].ctypes.data, keep["min_devices"].ctypes.data,
                 keep["prefill_base_us"].ctypes.data, keep["prefill_q16"].ctypes.data,
                 keep["step_us"].ctypes.data)
    return p, keep


def eval_placements(profile, trace, classes, offsets, inst, budget, class_mask=None, flags=0,
                    dump_idx=None):
    """Score every candidate; returns the result records (and the dumps if asked).

    dump_idx: candidate indices whose per-request (finish, first token, instance) arrays
    are also returned as a dict of [len(dump_idx)][n] arrays."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint32)
    inst = np.ascontiguousarray(inst, dtype=np.uint32)
    if inst.size == 0:
        inst = np.zeros(1, dtype=np.uint32)
    n_cand = len(offsets) - 1
    mask = None if class_mask is None else np.ascontiguousarray(class_mask, dtype=np.uint32)
    out = np.zeros(n_cand, dtype=_RES)
    n = len(trace)
    dumps = None
    didx = None
    if dump_idx is not None:
        didx = np.ascontiguousarray(dump_idx, dtype=np.uint32)
        dumps = {"finish_us": np.zeros((len(didx), n), dtype=np.int64),
                 "first_us": np.zeros((len(didx), n), dtype=np.int64),
                 "inst": np.zeros((len(didx), n), dtype=np.int32)}
    rc = lib.orc_eval_batch(C.byref(p), _ptr(trace), C.c_uint64(n), _ptr(classes),
                            C.c_uint32(len(classes)), _ptr(offsets), _ptr(inst), _ptr(mask),
                            C.c_uint64(n_cand), C.c_uint32(budget), C.c_uint32(flags), _ptr(out),
                            _ptr(didx), C.c_uint32(0 if didx is None else len(didx)),
                            _ptr(dumps["finish_us"]) if dumps else C.c_void_p(0),
                            _ptr(dumps["first_us"]) if dumps else C.c_void_p(0),
                            _ptr(dumps["inst"]) if dumps else C.c_void_p(0))
    if rc != 0:
        raise RuntimeError(f"oracle failed with code {rc}")
    del keep
    return (out, dumps) if dump_idx is not None else out


def _chunk(args):
    profile, trace, classes, offsets, inst, budget, mask, flags = args
    return eval_placements(profile, trace, classes, offsets, inst, budget, mask, flags)


def eval_placements_parallel(profile, trace, classes, offsets, inst, budget, class_mask=None,
                             flags=0, workers=None, pool=None):
    """Same results as eval_placements, candidates spread over `workers` processes
    (a `spawn` pool, so it is safe to create after CUDA has been initialised)."""
    import multiprocessing as mp
    offsets = np.asarray(offsets, dtype=np.uint32)
    inst = np.asarray(inst, dtype=np.uint32)
    n_cand = len(offsets) - 1
    workers = workers or min(os.cpu_count() or 1, 32)
    import sys
    main = sys.modules.get("__main__")
    if pool is None and not hasattr(main, "__file__"):
        workers = 1   # a spawn pool cannot re-import a __main__ that came from stdin
    if n_cand < 2 * workers or workers <= 1:
        return eval_placements(profile, trace, classes, offsets, inst, budget, class_mask, flags)
    n_chunks = min(n_cand, workers * 8)
    bounds = np.linspace(0, n_cand, n_chunks + 1).astype(np.int64)
    prof = {k: profile[k] for k in ("n_models", "n_strategies", "wmax", "devices", "min_devices",
                                    "prefill_base_us", "prefill_q16", "step_us")}
    jobs = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        off = offsets[a:b + 1].astype(np.int64)
        sub_inst = inst[off[0]:off[-1]]
        jobs.append((prof, trace, classes, (off - off[0]).astype(np.uint32), sub_inst, budget,
                     None if class_mask is None else np.asarray(class_mask)[a:b], flags))
    own = pool is None
    if own:
        build()
        pool = mp.get_context("spawn").Pool(workers)
    try:
        parts = pool.map(_chunk, jobs)
    finally:
        if own:
            pool.close()
            pool.join()
    return np.concatenate(parts)


class _ScoreParams(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("gamma_t", C.c_double), ("gamma_l", C.c_double)]


def score(results, alpha, beta, gamma_t, gamma_l):
    """Composite serving score of every record (see orc_score)."""
    lib = _load()
    results = np.ascontiguousarray(results, dtype=_RES)
    out = np.zeros(len(results), dtype=np.float64)
    p = _ScoreParams(alpha, beta, gamma_t, gamma_l)
    rc = lib.orc_score(_ptr(results), C.c_uint64(len(results)), C.byref(p), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle score failed with code {rc}")
    return out


def rejected_by_model(profile, trace, classes, offsets, inst, budget, class_mask=None, flags=0):
    """[n_cand][16] requests of each model that every candidate left unserved."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint32)
    inst = np.ascontiguousarray(inst, dtype=np.uint32)
    if inst.size == 0:
        inst = np.zeros(1, dtype=np.uint32)
    mask = None if class_mask is None else np.ascontiguousarray(class_mask, dtype=np.uint32)
    out = np.zeros((len(offsets) - 1, 16), dtype=np.uint32)
    rc = lib.orc_rejected_by_model(C.byref(p), _ptr(trace), C.c_uint64(len(trace)), _ptr(classes),
                                   C.c_uint32(len(classes)), _ptr(offsets), _ptr(inst), _ptr(mask),
                                   C.c_uint64(len(offsets) - 1), C.c_uint32(budget), C.c_uint32(flags), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle rejected_by_model failed with code {rc}")
    del keep
    return out


def ttft_hist(profile, trace, classes, offsets, inst, budget, class_mask=None, flags=0):
    """[n_cand][64] histogram of the time to first token of the served requests (see orc_ttft_hist)."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint32)
    inst = np.ascontiguousarray(inst, dtype=np.uint32)
    if inst.size == 0:
        inst = np.zeros(1, dtype=np.uint32)
    mask = None if class_mask is None else np.ascontiguousarray(class_mask, dtype=np.uint32)
    out = np.zeros((len(offsets) - 1, 64), dtype=np.uint32)
    rc = lib.orc_ttft_hist(C.byref(p), _ptr(trace), C.c_uint64(len(trace)), _ptr(classes),
                           C.c_uint32(len(classes)), _ptr(offsets), _ptr(inst), _ptr(mask),
                           C.c_uint64(len(offsets) - 1), C.c_uint32(budget), C.c_uint32(flags), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle ttft_hist failed with code {rc}")
    del keep
    return out


def ttft_percentiles(hist, permille):
    """[n_cand][len(permille)] upper bounds in microseconds (see orc_ttft_percentile)."""
    lib = _load()
    hist = np.ascontiguousarray(hist, dtype=np.uint32).reshape(-1, 64)
    out = np.zeros((len(hist), len(permille)), dtype=np.int64)
    for c in range(len(hist)):
        for j, pm in enumerate(permille):
            out[c, j] = lib.orc_ttft_percentile(_ptr(hist[c]), C.c_uint32(int(pm)))
    return out


def ins_deploy(profile, trace, classes, gpus, configs, alpha, beta, gamma_t, gamma_l, class_mask=None, flags=0):
    """Alg. 1 (see orc_ins_deploy).  configs: list of (strategy, batch).  Returns (phi_star[gpus+1],
    list of gpus+1 instance-word arrays)."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    cfg = np.ascontiguousarray(np.asarray(configs, dtype=np.uint32).reshape(-1, 2))
    sp = _ScoreParams(alpha, beta, gamma_t, gamma_l)
    phi = np.zeros(gpus + 1, dtype=np.float64)
    ilen = np.zeros(gpus + 1, dtype=np.uint32)
    iinst = np.zeros((gpus + 1, 128), dtype=np.uint32)
    rc = lib.orc_ins_deploy(C.byref(p), _ptr(trace), C.c_uint64(len(trace)), _ptr(classes), C.c_uint32(len(classes)),
                            C.c_int(0 if class_mask is None else 1), C.c_uint32(class_mask or 0), C.c_uint32(gpus),
                            _ptr(cfg), C.c_uint32(len(cfg)), C.byref(sp), C.c_uint32(flags), _ptr(phi), _ptr(ilen),
                            _ptr(iinst))
    if rc != 0:
        raise RuntimeError(f"oracle ins_deploy failed with code {rc}")
    del keep
    return phi, [iinst[k, :ilen[k]].copy() for k in range(gpus + 1)]


def partition(profile, trace, classes, mask_t, mask_l, gpus, configs, alpha, beta, gamma_t, gamma_l, flags=0,
              baseline=False):
    """Alg. 2 (see orc_partition).  Returns dict(g_t, g_l, phi, inst_t, inst_l)."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    cfg = np.ascontiguousarray(np.asarray(configs, dtype=np.uint32).reshape(-1, 2))
    sp = _ScoreParams(alpha, beta, gamma_t, gamma_l)
    g = np.zeros(2, dtype=np.uint32)
    phi = C.c_double(0.0)
    lt, ll = C.c_uint32(0), C.c_uint32(0)
    it, il = np.zeros(128, dtype=np.uint32), np.zeros(128, dtype=np.uint32)
    rc = lib.orc_partition(C.byref(p), _ptr(trace), C.c_uint64(len(trace)), _ptr(classes), C.c_uint32(len(classes)),
                           C.c_uint32(mask_t), C.c_uint32(mask_l), C.c_uint32(gpus), _ptr(cfg), C.c_uint32(len(cfg)),
                           C.byref(sp), C.c_uint32(flags), C.c_int(1 if baseline else 0), _ptr(g), C.byref(phi),
                           C.byref(lt), _ptr(it), C.byref(ll), _ptr(il))
    if rc != 0:
        raise RuntimeError(f"oracle partition failed with code {rc}")
    del keep
    return {"g_t": int(g[0]), "g_l": int(g[1]), "phi": phi.value, "inst_t": it[:lt.value].copy(),
            "inst_l": il[:ll.value].copy()}


def prune_configs(profile, trace, classes, batches, class_mask=None, flags=0):
    """getPrunedConfigs (see orc_prune_configs): list of (strategy, batch) in tree order."""
    lib = _load()
    p, keep = _profile_struct(profile)
    trace = np.ascontiguousarray(trace, dtype=_REQ)
    classes = np.ascontiguousarray(classes, dtype=_SLO)
    b = np.ascontiguousarray(batches, dtype=np.uint32)
    out = np.zeros((int(profile["n_strategies"]) * len(b), 2), dtype=np.uint32)
    n_out = C.c_uint32(0)
    rc = lib.orc_prune_configs(C.byref(p), _ptr(trace), C.c_uint64(len(trace)), _ptr(classes),
                               C.c_uint32(len(classes)), C.c_int(0 if class_mask is None else 1),
                               C.c_uint32(class_mask or 0), _ptr(b), C.c_uint32(len(b)), C.c_uint32(flags),
                               _ptr(out), C.byref(n_out))
    if rc != 0:
        raise RuntimeError(f"oracle prune_configs failed with code {rc}")
    del keep
    return [tuple(int(x) for x in row) for row in out[:n_out.value]]


def topk_scores(scores, k):
    """Indices of the k highest scores, ties to the lower index, NaN last."""
    lib = _load()
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    out = np.zeros(min(k, len(scores)), dtype=np.uint32)
    rc = lib.orc_topk_scores(_ptr(scores), C.c_uint64(len(scores)), C.c_uint32(k), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle topk_scores failed with code {rc}")
    return out


def topk(results, k, order=0):
    """Indices of the k best candidates, best first (see orc_topk for the ordering)."""
    lib = _load()
    results = np.ascontiguousarray(results, dtype=_RES)
    out = np.zeros(min(k, len(results)), dtype=np.uint32)
    rc = lib.orc_topk(_ptr(results), C.c_uint64(len(results)), C.c_uint32(k), C.c_uint32(order),
                      _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle topk failed with code {rc}")
    return out

"""ctypes binding of libmaaso.so: same names as the C entry points, marshalling only.

Device buffers are torch tensors (torch is used for device memory and streams, nothing
else); host buffers are numpy arrays.  There is no CPU path: if the shared library is
missing it is built with nvcc, and if that fails the import raises.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

REQUEST_DTYPE = np.dtype([("arrival_us", "<i8"), ("in_tokens", "<u4"), ("out_tokens", "<u2"),
                          ("cls", "u1"), ("model", "u1")])
SLO_DTYPE = np.dtype([("ttft_us", "<i8"), ("tbt_us", "<i8"), ("e2e_us", "<i8")])
RESULT_DTYPE = np.dtype([
    ("status", "<u4"), ("n_counted", "<u4"), ("n_served", "<u4"), ("n_hit", "<u4"),
    ("n_rejected", "<u4"), ("n_cascade", "<u4"), ("hit_by_class", "<u4", (8,)),
    ("sum_ttft_us", "<i8"), ("max_ttft_us", "<i8"), ("sum_e2e_us", "<i8"), ("max_e2e_us", "<i8"),
    ("makespan_us", "<i8"), ("tokens_out", "<u8"), ("checksum", "<u8"), ("attempts", "<u8"),
    ("reserved", "<u8")])
assert REQUEST_DTYPE.itemsize == 16 and SLO_DTYPE.itemsize == 24 and RESULT_DTYPE.itemsize == 128

FLAG_PRED_OPTIMISTIC = 1
FLAG_ENGINE_FROZEN = 2
FLAG_TBT_MAXGAP = 4
FLAG_INSTANCE_QUEUES = 8
FLAG_TEST_STALL = 0x80000000
MAP_AUTO, MAP_BLOCK, MAP_GROUP, MAP_THREAD = 0, 1, 2, 3
CAND_STATUS = {"EBUDGET": 1, "EMEMFIT": 2, "ETOOMANY": 4, "EBADINST": 8, "ETIMEOUT": 16, "ELOOP": 32}


class MaasoError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {maaso_strerror(code)} ({code}) {detail}".strip())


class _ProfileDesc(C.Structure):
    _fields_ = [("n_models", C.c_uint32), ("n_strategies", C.c_uint32), ("wmax", C.c_uint32),
                ("devices", C.c_void_p), ("min_devices", C.c_void_p), ("prefill_base_us", C.c_void_p),
                ("prefill_q16", C.c_void_p), ("step_us", C.c_void_p)]


class _CandBatch(C.Structure):
    _fields_ = [("offsets", C.c_void_p), ("inst", C.c_void_p), ("class_mask", C.c_void_p),
                ("n_cand", C.c_uint64), ("n_inst", C.c_uint64), ("budget", C.c_uint32),
                ("reserved", C.c_uint32)]


class _EvalOpts(C.Structure):
    _fields_ = [("flags", C.c_uint32), ("mapping", C.c_uint32), ("dump_n", C.c_uint32),
                ("reserved", C.c_uint32), ("dump_cand_idx", C.c_void_p), ("dump_finish_us", C.c_void_p),
                ("dump_first_us", C.c_void_p), ("dump_inst", C.c_void_p), ("rejected_by_model", C.c_void_p),
                ("ttft_hist", C.c_void_p)]


class _ScoreParams(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("gamma_t", C.c_double), ("gamma_l", C.c_double)]


class _Timing(C.Structure):
    _fields_ = [("prep_ms", C.c_float), ("group_ms", C.c_float), ("block_ms", C.c_float),
                ("topk_ms", C.c_float), ("thread_ms", C.c_float)]


def lib_path():
    return _build.LIB


def _load():
    path = _build.LIB
    if not os.path.exists(path) or _build.stale():
        path = _build.build()          # raises if nvcc is missing or the build fails
    lib = C.CDLL(path)
    vp, u64, u32 = C.c_void_p, C.c_uint64, C.c_uint32
    lib.maaso_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.maaso_destroy.argtypes = [vp]
    lib.maaso_destroy.restype = None
    lib.maaso_load_profile.argtypes = [vp, C.POINTER(_ProfileDesc)]
    lib.maaso_load_trace.argtypes = [vp, vp, u64, vp, u32, C.POINTER(vp)]
    lib.maaso_free_trace.argtypes = [vp, vp]
    lib.maaso_free_trace.restype = None
    lib.maaso_eval_placements.argtypes = [vp, vp, C.POINTER(_CandBatch), C.POINTER(_EvalOpts), vp, vp]
    lib.maaso_eval_placements_host.argtypes = [vp, vp, C.POINTER(_CandBatch), C.POINTER(_EvalOpts), vp]
    lib.maaso_eval_placements_multi.argtypes = [vp, C.POINTER(vp), u32, C.POINTER(_CandBatch), C.POINTER(_EvalOpts), vp, vp]
    lib.maaso_eval_placements_multi.restype = C.c_int
    lib.maaso_topk.argtypes = [vp, vp, u64, u32, u32, vp, vp, vp]
    lib.maaso_score.argtypes = [vp, vp, u64, C.POINTER(_ScoreParams), vp, vp]
    lib.maaso_topk_scores.argtypes = [vp, vp, vp, u64, u32, vp, vp, vp]
    lib.maaso_ttft_percentiles.argtypes = [vp, vp, u64, vp, u32, vp, vp]
    lib.maaso_ttft_percentiles.restype = C.c_int
    lib.maaso_ins_deploy.argtypes = [vp, vp, u32, vp, u32, C.c_int, u32, C.POINTER(_ScoreParams), u32, vp, vp, vp]
    lib.maaso_ins_deploy.restype = C.c_int
    lib.maaso_prune_configs.argtypes = [vp, vp, C.c_int, u32, vp, u32, u32, vp, C.POINTER(u32)]
    lib.maaso_prune_configs.restype = C.c_int
    lib.maaso_partition.argtypes = [vp, vp, u32, u32, u32, vp, u32, C.POINTER(_ScoreParams), u32, C.c_int, vp,
                                    C.POINTER(C.c_double), C.POINTER(u32), vp, C.POINTER(u32), vp]
    lib.maaso_partition.restype = C.c_int
    lib.maaso_topk_noalloc.argtypes = [vp, u64, u32, u32, vp, vp, vp]
    lib.maaso_topk_noalloc.restype = C.c_int
    lib.maaso_set_timing.argtypes = [vp, C.c_int]
    lib.maaso_get_timing.argtypes = [vp, C.POINTER(_Timing)]
    lib.maaso_launch_count.argtypes = [vp]
    lib.maaso_test_fail_allocs.argtypes = [vp, C.c_int]
    lib.maaso_test_fail_allocs.restype = C.c_int
    lib.maaso_launch_count.restype = u64
    lib.maaso_strerror.argtypes = [C.c_int]
    lib.maaso_strerror.restype = C.c_char_p
    lib.maaso_last_error.argtypes = [vp]
    lib.maaso_last_error.restype = C.c_char_p
    for name in ("maaso_create", "maaso_load_profile", "maaso_load_trace", "maaso_eval_placements",
                 "maaso_eval_placements_host", "maaso_topk", "maaso_set_timing", "maaso_get_timing",
                 "maaso_score", "maaso_topk_scores"):
        getattr(lib, name).restype = C.c_int
    return lib


_lib = _load()


def maaso_strerror(code):
    return _lib.maaso_strerror(int(code)).decode()


def maaso_last_error(ctx):
    return _lib.maaso_last_error(ctx).decode()


def _check(rc, where, ctx=None):
    if rc != 0:
        raise MaasoError(rc, where, maaso_last_error(ctx) if ctx else "")


def _ptr(x):
    """device pointer of a torch tensor, host pointer of a numpy array, or NULL"""
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return getattr(stream, "cuda_stream", stream)


# ---- entry points, one per C function ---------------------------------------------------------
def maaso_create(cuda_device=0):
    ctx = C.c_void_p()
    _check(_lib.maaso_create(C.byref(ctx), int(cuda_device)), "maaso_create")
    return ctx


def maaso_destroy(ctx):
    _lib.maaso_destroy(ctx)


def maaso_load_profile(ctx, profile):
    """profile: dict with n_models, n_strategies, wmax and the int32 tables (host arrays)."""
    keep = {k: np.ascontiguousarray(profile[k], dtype=np.int32)
            for k in ("devices", "min_devices", "prefill_base_us", "prefill_q16", "step_us")}
    M, S, W = int(profile["n_models"]), int(profile["n_strategies"]), int(profile["wmax"])
    if keep["devices"].size != S or keep["min_devices"].size != M or \
            keep["prefill_base_us"].size != M * S or keep["prefill_q16"].size != M * S or \
            keep["step_us"].size != M * S * W:
        raise MaasoError(-1, "maaso_load_profile", "table sizes do not match n_models/n_strategies/wmax")
    d = _ProfileDesc(M, S, W, *(keep[k].ctypes.data for k in
                               ("devices", "min_devices", "prefill_base_us", "prefill_q16", "step_us")))
    _check(_lib.maaso_load_profile(ctx, C.byref(d)), "maaso_load_profile", ctx)


def maaso_load_trace(ctx, reqs, classes):
    """reqs: numpy array of REQUEST_DTYPE (host) or a torch uint8 CUDA tensor of 16-byte records;
    classes: numpy array of SLO_DTYPE (host).  Returns the trace handle."""
    classes = np.ascontiguousarray(classes, dtype=SLO_DTYPE)
    if isinstance(reqs, np.ndarray):
        reqs = np.ascontiguousarray(reqs, dtype=REQUEST_DTYPE)
        n = len(reqs)
    else:
        assert reqs.dtype.itemsize == 1 and reqs.numel() % 16 == 0
        n = reqs.numel() // 16
    out = C.c_void_p()
    _check(_lib.maaso_load_trace(ctx, _ptr(reqs), n, classes.ctypes.data, len(classes), C.byref(out)),
           "maaso_load_trace", ctx)
    return out


def maaso_free_trace(ctx, trace):
    _lib.maaso_free_trace(ctx, trace)


def _batch(offsets, inst, class_mask, budget):
    n_cand = int(offsets.shape[0]) - 1
    n_inst = int(inst.shape[0]) if inst is not None else 0
    return _CandBatch(_ptr(offsets), _ptr(inst) if n_inst else None, _ptr(class_mask), n_cand, n_inst,
                      int(budget), 0)


def maaso_eval_placements(ctx, trace, offsets, inst, budget, out_results, class_mask=None, flags=0,
                          mapping=MAP_AUTO, dump_cand_idx=None, dump_finish_us=None, dump_first_us=None,
                          dump_inst=None, rejected_by_model=None, ttft_hist=None, stream=None):
    """All array arguments are CUDA tensors (int32 views of the uint32 words; out_results a
    uint8 tensor of n_cand*128 bytes).  Work is enqueued on `stream` (default: torch's current)."""
    b = _batch(offsets, inst, class_mask, budget)
    o = _EvalOpts(int(flags), int(mapping), 0 if dump_cand_idx is None else int(dump_cand_idx.shape[0]), 0,
                  _ptr(dump_cand_idx), _ptr(dump_finish_us), _ptr(dump_first_us), _ptr(dump_inst),
                  _ptr(rejected_by_model), _ptr(ttft_hist))
    _check(_lib.maaso_eval_placements(ctx, trace, C.byref(b), C.byref(o), _ptr(out_results),
                                      _stream_ptr(stream)), "maaso_eval_placements", ctx)


def maaso_eval_placements_multi(ctx, traces, offsets, inst, budget, out_results, class_mask=None, flags=0,
                                rejected_by_model=None, ttft_hist=None, stream=None, mapping=MAP_AUTO):
    """traces: sequence of trace handles; out_results: uint8 CUDA tensor of len(traces)*n_cand*128 bytes."""
    b = _batch(offsets, inst, class_mask, budget)
    o = _EvalOpts(int(flags), int(mapping), 0, 0, None, None, None, None, _ptr(rejected_by_model), _ptr(ttft_hist))
    arr = (C.c_void_p * len(traces))(*[t if isinstance(t, int) else (t.value if hasattr(t, "value") else t) for t in traces])
    _check(_lib.maaso_eval_placements_multi(ctx, arr, len(traces), C.byref(b), C.byref(o), _ptr(out_results),
                                            _stream_ptr(stream)), "maaso_eval_placements_multi", ctx)


def maaso_eval_placements_host(ctx, trace, offsets, inst, budget, out_results, class_mask=None, flags=0,
                               mapping=MAP_AUTO):
    """Host (numpy) buffers in and out; copies happen inside the call, which synchronises."""
    b = _batch(offsets, inst, class_mask, budget)
    o = _EvalOpts(int(flags), int(mapping), 0, 0, None, None, None, None, None, None)
    _check(_lib.maaso_eval_placements_host(ctx, trace, C.byref(b), C.byref(o), _ptr(out_results)),
           "maaso_eval_placements_host", ctx)


def maaso_topk(ctx, results, n_cand, k, out_idx, out_res=None, order=0, stream=None):
    _check(_lib.maaso_topk(ctx, _ptr(results), int(n_cand), int(k), int(order), _ptr(out_idx), _ptr(out_res),
                           _stream_ptr(stream)), "maaso_topk", ctx)


def maaso_score(ctx, results, n_cand, alpha, beta, gamma_t, gamma_l, out_scores, stream=None):
    p = _ScoreParams(float(alpha), float(beta), float(gamma_t), float(gamma_l))
    _check(_lib.maaso_score(ctx, _ptr(results), int(n_cand), C.byref(p), _ptr(out_scores), _stream_ptr(stream)),
           "maaso_score", ctx)


def maaso_ttft_percentiles(ctx, ttft_hist, n_cand, permille, out, stream=None):
    pm = np.ascontiguousarray(permille, dtype=np.uint32)
    _check(_lib.maaso_ttft_percentiles(ctx, _ptr(ttft_hist), int(n_cand), pm.ctypes.data, len(pm), _ptr(out),
                                       _stream_ptr(stream)), "maaso_ttft_percentiles", ctx)


def maaso_topk_scores(ctx, results, scores, n_cand, k, out_idx, out_res=None, stream=None):
    _check(_lib.maaso_topk_scores(ctx, _ptr(results), _ptr(scores), int(n_cand), int(k), _ptr(out_idx),
                                  _ptr(out_res), _stream_ptr(stream)), "maaso_topk_scores", ctx)


def maaso_ins_deploy(ctx, trace, gpus, configs, alpha, beta, gamma_t, gamma_l, class_mask=None, flags=0):
    """Alg. 1 on the GPU.  configs: sequence of (strategy, batch).  Returns (phi_star[gpus+1] as a
    numpy array, list of gpus+1 arrays of packed instance words)."""
    cfg = np.ascontiguousarray(np.asarray(configs, dtype=np.uint32).reshape(-1, 2))
    p = _ScoreParams(float(alpha), float(beta), float(gamma_t), float(gamma_l))
    phi = np.zeros(gpus + 1, dtype=np.float64)
    ilen = np.zeros(gpus + 1, dtype=np.uint32)
    iinst = np.zeros((gpus + 1, 128), dtype=np.uint32)
    _check(_lib.maaso_ins_deploy(ctx, trace, int(gpus), cfg.ctypes.data, len(cfg), 0 if class_mask is None else 1,
                                 int(class_mask or 0), C.byref(p), int(flags), phi.ctypes.data, ilen.ctypes.data,
                                 iinst.ctypes.data), "maaso_ins_deploy", ctx)
    return phi, [iinst[k, :ilen[k]].copy() for k in range(gpus + 1)]


def maaso_prune_configs(ctx, trace, n_strategies, batches, class_mask=None, flags=0):
    """getPrunedConfigs: list of (strategy, batch) in configuration-tree order."""
    b = np.ascontiguousarray(batches, dtype=np.uint32)
    out = np.zeros((int(n_strategies) * len(b), 2), dtype=np.uint32)
    n_out = C.c_uint32(0)
    _check(_lib.maaso_prune_configs(ctx, trace, 0 if class_mask is None else 1, int(class_mask or 0),
                                    b.ctypes.data, len(b), int(flags), out.ctypes.data, C.byref(n_out)),
           "maaso_prune_configs", ctx)
    return [tuple(int(x) for x in row) for row in out[:n_out.value]]


def maaso_partition(ctx, trace, mask_t, mask_l, gpus, configs, alpha, beta, gamma_t, gamma_l, flags=0,
                    baseline=False):
    """Alg. 2 for two sub-clusters.  Returns dict(g_t, g_l, phi, inst_t, inst_l)."""
    cfg = np.ascontiguousarray(np.asarray(configs, dtype=np.uint32).reshape(-1, 2))
    p = _ScoreParams(float(alpha), float(beta), float(gamma_t), float(gamma_l))
    g = np.zeros(2, dtype=np.uint32)
    phi = C.c_double(0.0)
    lt, ll = C.c_uint32(0), C.c_uint32(0)
    it, il = np.zeros(128, dtype=np.uint32), np.zeros(128, dtype=np.uint32)
    _check(_lib.maaso_partition(ctx, trace, int(mask_t), int(mask_l), int(gpus), cfg.ctypes.data, len(cfg),
                                C.byref(p), int(flags), 1 if baseline else 0, g.ctypes.data, C.byref(phi),
                                C.byref(lt), it.ctypes.data, C.byref(ll), il.ctypes.data), "maaso_partition", ctx)
    return {"g_t": int(g[0]), "g_l": int(g[1]), "phi": phi.value, "inst_t": it[:lt.value].copy(),
            "inst_l": il[:ll.value].copy()}


NOALLOC_MAX_CAND = 1 << 20
NOALLOC_MAX_K = 64


def maaso_topk_noalloc(results, n_cand, k, out_idx, out_res=None, order=0, stream=None):
    """Top-k for callers that may not allocate device memory (pool-managed or latency-critical
    code): same result as maaso_topk, no context, scratch in a fixed array of the library;
    n_cand <= NOALLOC_MAX_CAND, k <= NOALLOC_MAX_K.  Returns the C return code unchanged so
    that the caller can tell a capacity refusal (-5) from other errors."""
    return int(_lib.maaso_topk_noalloc(_ptr(results), int(n_cand), int(k), int(order), _ptr(out_idx),
                                       _ptr(out_res), _stream_ptr(stream)))


def maaso_set_timing(ctx, enabled):
    _check(_lib.maaso_set_timing(ctx, 1 if enabled else 0), "maaso_set_timing", ctx)


def maaso_get_timing(ctx):
    """milliseconds per kernel family of the most recent eval / topk calls (waits for them)"""
    t = _Timing()
    _check(_lib.maaso_get_timing(ctx, C.byref(t)), "maaso_get_timing", ctx)
    return {"prep_ms": t.prep_ms, "group_ms": t.group_ms, "block_ms": t.block_ms, "topk_ms": t.topk_ms,
            "thread_ms": t.thread_ms}


def maaso_launch_count(ctx):
    return int(_lib.maaso_launch_count(ctx))


def maaso_test_fail_allocs(ctx, count):
    """test hook: the next `count` growths of the context's scratch buffers are refused"""
    _check(_lib.maaso_test_fail_allocs(ctx, int(count)), "maaso_test_fail_allocs", ctx)


# ---- convenience wrappers (allocation of outputs only) -------------------------------------------
class Trace:
    def __init__(self, ctx, handle, n):
        self.ctx, self.handle, self.n = ctx, handle, n


class Context:
    """Owns a library context on one CUDA device; allocates output tensors for the calls."""

    def __init__(self, device=0):
        import torch
        self.torch = torch
        self.device = torch.device("cuda", device)
        self.handle = maaso_create(device)

    def close(self):
        if self.handle is not None:
            maaso_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load_profile(self, profile):
        maaso_load_profile(self.handle, profile)

    def load_trace(self, reqs, classes):
        n = len(reqs) if isinstance(reqs, np.ndarray) else reqs.numel() // 16
        return Trace(self, maaso_load_trace(self.handle, reqs, classes), n)

    def free_trace(self, trace):
        maaso_free_trace(self.handle, trace.handle)
        trace.handle = None

    def to_device(self, words):
        """uint32 numpy words -> int32 CUDA tensor with the same bits"""
        t = self.torch.from_numpy(np.ascontiguousarray(words, dtype=np.uint32).view(np.int32))
        return t.to(self.device)

    def prune_configs(self, trace, n_strategies, batches, class_mask=None, flags=0):
        return maaso_prune_configs(self.handle, trace.handle, n_strategies, batches, class_mask, flags)

    def partition(self, trace, mask_t, mask_l, gpus, configs, alpha, beta, gamma_t, gamma_l, flags=0,
                  baseline=False):
        return maaso_partition(self.handle, trace.handle, mask_t, mask_l, gpus, configs, alpha, beta, gamma_t,
                               gamma_l, flags, baseline)

    def ins_deploy(self, trace, gpus, configs, alpha, beta, gamma_t, gamma_l, class_mask=None, flags=0):
        return maaso_ins_deploy(self.handle, trace.handle, gpus, configs, alpha, beta, gamma_t, gamma_l,
                                class_mask, flags)

    def eval_placements(self, trace, offsets, inst, budget, class_mask=None, flags=0, mapping=MAP_AUTO,
                        dump_idx=None, out=None, stream=None, rejected_by_model=None, ttft_hist=None):
        """offsets / inst / class_mask: CUDA int32 tensors (see to_device).  Returns the uint8
        result tensor [n_cand, 128] and, if dump_idx is given, a dict of dump tensors."""
        torch = self.torch
        n_cand = int(offsets.shape[0]) - 1
        if out is None:
            out = torch.empty((n_cand, 128), dtype=torch.uint8, device=self.device)
        dumps = None
        kw = {}
        if dump_idx is not None:
            d = self.to_device(np.asarray(dump_idx, dtype=np.uint32))
            dumps = {"finish_us": torch.empty((len(dump_idx), trace.n), dtype=torch.int64, device=self.device),
                     "first_us": torch.empty((len(dump_idx), trace.n), dtype=torch.int64, device=self.device),
                     "inst": torch.empty((len(dump_idx), trace.n), dtype=torch.int32, device=self.device)}
            kw = dict(dump_cand_idx=d, dump_finish_us=dumps["finish_us"], dump_first_us=dumps["first_us"],
                      dump_inst=dumps["inst"])
        maaso_eval_placements(self.handle, trace.handle, offsets, inst, budget, out, class_mask, flags,
                              mapping, stream=stream, rejected_by_model=rejected_by_model, ttft_hist=ttft_hist,
                              **kw)
        return (out, dumps) if dump_idx is not None else out

    def eval_placements_multi(self, traces, offsets, inst, budget, class_mask=None, flags=0, out=None, stream=None,
                              rejected_by_model=None, ttft_hist=None, mapping=MAP_AUTO):
        """One pass over several traces (at most 16, same SLO classes).  Returns a uint8 tensor
        [len(traces), n_cand, 128]: block t holds the records for traces[t]."""
        torch = self.torch
        n_cand = int(offsets.shape[0]) - 1
        if out is None:
            out = torch.empty((len(traces), n_cand, 128), dtype=torch.uint8, device=self.device)
        maaso_eval_placements_multi(self.handle, [t.handle for t in traces], offsets, inst, budget, out, class_mask,
                                    flags, rejected_by_model, ttft_hist, stream, mapping)
        return out

    def eval_placements_host(self, trace, offsets, inst, budget, class_mask=None, flags=0,
                             mapping=MAP_AUTO, out=None):
        offsets = np.ascontiguousarray(offsets, dtype=np.uint32)
        inst = np.ascontiguousarray(inst, dtype=np.uint32)
        if class_mask is not None:
            class_mask = np.ascontiguousarray(class_mask, dtype=np.uint32)
        if out is None:
            out = np.empty(len(offsets) - 1, dtype=RESULT_DTYPE)
        maaso_eval_placements_host(self.handle, trace.handle, offsets, inst, budget, out, class_mask,
                                   flags, mapping)
        return out

    def topk(self, results, k, order=0, with_records=True, stream=None):
        torch = self.torch
        n_cand = int(results.shape[0])
        idx = torch.empty(k, dtype=torch.int32, device=self.device)
        rec = torch.empty((k, 128), dtype=torch.uint8, device=self.device) if with_records else None
        maaso_topk(self.handle, results, n_cand, k, idx, rec, order, stream)
        return idx, rec

    def score(self, results, alpha, beta, gamma_t, gamma_l, stream=None):
        out = self.torch.empty(int(results.shape[0]), dtype=self.torch.float64, device=self.device)
        maaso_score(self.handle, results, int(results.shape[0]), alpha, beta, gamma_t, gamma_l, out, stream)
        return out

    def ttft_percentiles(self, ttft_hist, permille, stream=None):
        """ttft_hist: int32 CUDA tensor [n_cand, 64] filled by eval_placements(ttft_hist=...).
        Returns an int64 tensor [n_cand, len(permille)] of bin upper edges in microseconds."""
        n_cand = int(ttft_hist.shape[0])
        out = self.torch.empty((n_cand, len(permille)), dtype=self.torch.int64, device=self.device)
        maaso_ttft_percentiles(self.handle, ttft_hist, n_cand, permille, out, stream)
        return out

    def topk_scores(self, results, scores, k, with_records=True, stream=None):
        torch = self.torch
        idx = torch.empty(k, dtype=torch.int32, device=self.device)
        rec = torch.empty((k, 128), dtype=torch.uint8, device=self.device) if with_records else None
        maaso_topk_scores(self.handle, results, scores, int(results.shape[0]), k, idx, rec, stream)
        return idx, rec

    def set_timing(self, enabled):
        maaso_set_timing(self.handle, enabled)

    def get_timing(self):
        return maaso_get_timing(self.handle)

    def launch_count(self):
        return maaso_launch_count(self.handle)

    def test_fail_allocs(self, count):
        """test hook: refuse the next `count` growths of the context's scratch buffers"""
        maaso_test_fail_allocs(self.handle, count)

    @staticmethod
    def results_to_numpy(t):
        return t.cpu().numpy().reshape(-1).view(RESULT_DTYPE)

#!/usr/bin/env python
"""Throughput benchmark of the placement-scoring path.

One step = one pass of the whole path over one batch: candidate validation, trace replay
for every candidate (distributor + continuous batching) and the top-64 selection.  Default
workload: the multi-model sweep, 100,000 sampled placements of up to 32 devices x a
100,000-request trace.  With N GPUs the SAME sweep is sharded over the ranks in contiguous
candidate ranges (strong scaling); the only exchange is the gather of 64 records per rank.
Prints ONE JSON line.  `--impl reference` times the CPU oracle instead.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "candidate x request evaluations per second"
UNIT = "evals/s"
TOPK = 64

# ncu counters of the dominant kernel on the default workload (see profiles/).  They describe the
# kernels whose source hashes to `csrc_sha256`; with any other source they are not printed.
PROFILED = {
    "workload": "multimodel", "mapping": 0, "kernel": "eval_thread_kernel",
    # profiles/eval_thread_kernel_multimodel_sweep_counters.md: one launch of the default workload
    "warp_inst_per_launch": 46573414946,                 # smsp__inst_executed.sum
    "dram_bytes_per_launch": 8540173312 + 6593907712,    # dram__bytes_read.sum + dram__bytes_write.sum
    "csrc_sha256": "38d6462581e8b3e93e08ae6faacbcde5536639edd825c4f14a4a1d54dd9372cb",
}
SM_COUNT, ISSUE_PER_SM = 148, 4   # B200: 148 SMs x 4 warp schedulers, one warp instruction per cycle each


def csrc_sha256():
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2509_06362_b200", "csrc")
    for name in sorted(os.listdir(d)):
        if name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t_begin, t_end):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = [r for r in self.rows if t_begin - 0.05 <= r[0] <= t_end + 0.15] or self.rows
        for _, line in rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(cfg, evals):
    """Effective bytes of one pass: a 16-byte trace record per evaluation, the candidate
    words and offsets, one 128-byte record per candidate, the latency tables once."""
    n_cand = len(cfg["offsets"]) - 1
    prof = cfg["profile"]
    prof_bytes = prof["step_us"].nbytes + prof["prefill_base_us"].nbytes + prof["prefill_q16"].nbytes
    return evals * 16 + 4 * len(cfg["inst"]) + 8 * n_cand + 128 * n_cand + prof_bytes


FULL_CANDIDATES = {"tiny": 143, "node": 10_864, "bursty": 10_864, "multimodel": 100_000, "scale": 1_000_000, "large": 2_000}


def workload_label(name, n_cand, n_req, n_tr, budget):
    """One name for a workload, the same in both arms."""
    return (f"{name} sweep: {n_cand} placements x {n_req} requests"
            f"{f' x {n_tr} traces in one pass' if n_tr > 1 else ''}, budget {budget}, top-{TOPK}")


def oracle_pass(oracle, cfg, flags=0):
    res = oracle.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"],
                                 cfg["inst"], cfg["budget"], None, flags)
    oracle.topk(res, TOPK)
    return int(res["n_counted"][res["status"] == 0].astype(np.int64).sum())


def sample_of(gen, workload, n_cand, n_req, sample_cands):
    """A bounded sample of a workload for the CPU oracle: `sample_cands` placements spread evenly over
    the sweep, against the whole first trace."""
    if workload in ("tiny", "node", "bursty"):
        # enumerated sweeps are ordered from small to large placements: take every k-th one
        cfg = gen.make_config(workload, n_cand=n_cand, n_req=n_req)
        off = cfg["offsets"].astype(np.int64)
        stride = max(1, (len(off) - 1) // sample_cands)
        pick = np.arange(0, len(off) - 1, stride)[:sample_cands]
        parts = [cfg["inst"][off[c]:off[c + 1]] for c in pick]
        cfg["offsets"] = np.concatenate([[0], np.cumsum([len(x) for x in parts])]).astype(np.uint32)
        cfg["inst"] = np.concatenate(parts).astype(np.uint32)
        return cfg, f"every {stride}th placement ({len(pick)})"
    # sampled sweeps: the first placements of the seeded sample are as good as any
    cfg = gen.make_config(workload, n_cand=sample_cands if n_cand is None else min(n_cand, sample_cands), n_req=n_req)
    return cfg, f"the first {len(cfg['offsets']) - 1} placements of the seeded sample"


def run_reference(args):
    """The CPU oracle as it stands, one thread, on a bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import gen
    import oracle
    oracle.build()
    cfg, how = sample_of(gen, args.workload, args.n_cand, args.n_req, 256)
    times, evals = [], 0
    for step in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        ev = oracle_pass(oracle, cfg, args.flags)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            times.append(dt)
            evals = ev
    value = evals * len(times) / sum(times)
    n_full = args.n_cand or FULL_CANDIDATES.get(args.workload, 2000)   # Table I sweeps default to 2,000
    sample = f"{how} x all {len(cfg['traces'][0])} requests of the first trace per step, 1 thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": workload_label(cfg["name"], n_full, len(cfg["traces"][0]), len(cfg["traces"]),
                                              cfg["budget"]), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(args):
    """Oracle throughput on this host, one thread, on a bounded sample of the workload (10-30 s)."""
    import gen
    import oracle
    oracle.build()
    cfg, how = sample_of(gen, args.workload, args.n_cand, args.n_req, 4096 if args.workload != "scale" else 256)
    t0 = time.perf_counter()
    evals = oracle_pass(oracle, cfg, args.flags)
    dt = time.perf_counter() - t0
    return {"value": evals / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{how} x all {len(cfg['traces'][0])} requests, {dt:.1f} s, 1 thread; the rate is that of "
                      f"the sample, not an extrapolated run of the whole sweep"}


def scale_slice(m, torch, device_index, mapping):
    """One timed pass of a slice of the scale-stress configuration: the first 100,000 of its 10^6 sampled
    placements (budget 128) against the full 10^6-request trace, top-64.  The full pass takes too long to
    repeat inside a benchmark run; the slice is timed once, after a warm-up on a short trace."""
    import gen
    cfg = gen.make_config("scale", n_cand=100_000)
    ctx = m.Context(device_index)
    ctx.load_profile(cfg["profile"])
    warm = ctx.load_trace(cfg["traces"][0][:2000], cfg["classes"])
    trace = ctx.load_trace(cfg["traces"][0], cfg["classes"])
    d_off, d_inst = ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"])
    out = torch.empty((len(cfg["offsets"]) - 1, 128), dtype=torch.uint8, device=ctx.device)
    stream = torch.cuda.current_stream()
    ctx.eval_placements(warm, d_off, d_inst, cfg["budget"], mapping=mapping, out=out, stream=stream)
    ctx.topk(out, TOPK, stream=stream)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    ctx.eval_placements(trace, d_off, d_inst, cfg["budget"], mapping=mapping, out=out, stream=stream)
    ctx.topk(out, TOPK, stream=stream)
    b.record(stream)
    b.synchronize()
    ms = a.elapsed_time(b)
    rec = ctx.results_to_numpy(out)
    evals = int(rec["n_counted"][rec["status"] == 0].astype(np.int64).sum())
    ctx.close()
    return {"workload": workload_label("scale (slice)", len(rec), len(cfg["traces"][0]), 1, cfg["budget"]),
            "passes": 1, "ms": ms, "evals": evals, "value": evals / (ms * 1e-3), "unit": UNIT,
            "placements_over_32_instances": int((np.diff(cfg["offsets"].astype(np.int64)) > 32).sum())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mapping", type=int, default=0, help="0 auto, 1 block layout, 2 lane groups, 3 thread per placement")
    ap.add_argument("--workload", default="multimodel", help="multimodel (default) or another configuration name")
    ap.add_argument("--n-cand", type=int, default=None)
    ap.add_argument("--n-req", type=int, default=None)
    ap.add_argument("--flags", type=int, default=0, help="engine flags of maaso_eval_placements (0: the default engine)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-scale-slice", action="store_true")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import gen
    import paper_2509_06362_b200 as m
    from paper_2509_06362_b200.distributed import shard_range, shard_csr, global_topk

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = gen.make_config(args.workload, n_cand=args.n_cand, n_req=args.n_req)
    trace_np = cfg["traces"][0]
    n_total = len(cfg["offsets"]) - 1
    n_tr = len(cfg["traces"])     # more than one: the load sweep, all traces in one pass
    # ONE sweep: this rank scores the contiguous shard [lo, hi) of its candidates
    lo, hi = shard_range(n_total, rank, world)
    off_np, inst_np = shard_csr(cfg["offsets"], cfg["inst"], lo, hi)
    n_cand = hi - lo
    ctx = m.Context(local)
    ctx.load_profile(cfg["profile"])
    traces = [ctx.load_trace(t, cfg["classes"]) for t in cfg["traces"]]
    trace = traces[0]
    d_off, d_inst = ctx.to_device(off_np), ctx.to_device(inst_np)
    results = torch.empty((n_tr * n_cand, 128), dtype=torch.uint8, device=ctx.device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=ctx.device)  # > L2 (126 MB)
    stream = torch.cuda.current_stream()
    ctx.set_timing(True)

    def rank_topk(rec, k):
        return ctx.topk(rec, k, stream=stream)

    def step():
        if n_tr > 1:
            ctx.eval_placements_multi(traces, d_off, d_inst, cfg["budget"], flags=args.flags, out=results, stream=stream)
        else:
            ctx.eval_placements(trace, d_off, d_inst, cfg["budget"], flags=args.flags, mapping=args.mapping, out=results,
                                stream=stream)
        if world == 1:
            return ctx.topk(results, TOPK, stream=stream)
        return global_topk(rank_topk, rank_topk, results, lo, TOPK)   # local top-64, gather, merge

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # the clock sampler starts (and settles) before the warm-up, so that the timed steps follow the warm-up
    # steps directly and no idle gap lets the GPU leave its loaded state
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    for _ in range(args.warmup):
        flush.fill_(1)
        step()
    sync_all()
    rec = ctx.results_to_numpy(results)
    evals_rank = int(rec["n_counted"][rec["status"] == 0].astype(np.int64).sum())
    evals_t = torch.tensor([evals_rank], dtype=torch.int64, device=ctx.device)
    if dist is not None:
        dist.all_reduce(evals_t)
    evals_per_step = int(evals_t.item())      # of the whole sweep, all ranks

    launches0 = ctx.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    kernel_ms = []
    sync_all()
    t_begin = time.time()
    for a, b in ev:
        flush.fill_(2)               # L2 flush between timed iterations (not timed)
        a.record(stream)
        step()
        b.record(stream)
        b.synchronize()
        kernel_ms.append(ctx.get_timing())
    sync_all()
    t_end = time.time()
    launches = ctx.launch_count() - launches0
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = torch.tensor([sum(step_ms)], dtype=torch.float64, device=ctx.device)
    if dist is not None:
        dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None

    # End to end through the public calls with HOST buffers: every step copies this rank's candidate
    # arrays from pinned host memory to the device, scores them, selects the top-64 and copies all
    # records and the selection back to pinned host memory.
    off_pin = torch.from_numpy(off_np.view(np.int32)).pin_memory()
    inst_pin = torch.from_numpy(inst_np.view(np.int32)).pin_memory()
    out_pin = torch.empty((n_tr * n_cand, 128), dtype=torch.uint8).pin_memory()
    top_idx_pin = torch.empty(TOPK, dtype=torch.int32).pin_memory()
    top_rec_pin = torch.empty((TOPK, 128), dtype=torch.uint8).pin_memory()
    d_off2, d_inst2 = torch.empty_like(d_off), torch.empty_like(d_inst)

    def e2e_step():
        flush.fill_(3)               # same cache state as the timed steps: L2 flushed before every pass
        d_off2.copy_(off_pin, non_blocking=True)
        d_inst2.copy_(inst_pin, non_blocking=True)
        if n_tr > 1:
            ctx.eval_placements_multi(traces, d_off2, d_inst2, cfg["budget"], flags=args.flags, out=results, stream=stream)
        else:
            ctx.eval_placements(trace, d_off2, d_inst2, cfg["budget"], flags=args.flags, mapping=args.mapping, out=results, stream=stream)
        if world == 1:
            idx, top = ctx.topk(results, TOPK, stream=stream)
            top_idx_pin.copy_(idx, non_blocking=True)
            top_rec_pin.copy_(top, non_blocking=True)
        else:
            global_topk(rank_topk, rank_topk, results, lo, TOPK)
        out_pin.copy_(results.view(n_tr * n_cand, 128), non_blocking=True)
        torch.cuda.synchronize()

    for _ in range(2):
        e2e_step()
    sync_all()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device=ctx.device)
    if dist is not None:
        dist.all_reduce(e2e_s, op=dist.ReduceOp.MAX)
    e2e_value = evals_per_step * e2e_steps / float(e2e_s.item())
    assert out_pin.numpy().reshape(-1).view(m.RESULT_DTYPE).tobytes() == rec.tobytes(), \
        "the end-to-end pass disagrees with the device-resident pass"
    h2d = torch.tensor([off_np.nbytes + inst_np.nbytes], dtype=torch.int64, device=ctx.device)
    d2h = torch.tensor([n_tr * n_cand * 128 + TOPK * 132], dtype=torch.int64, device=ctx.device)
    if dist is not None:
        dist.all_reduce(h2d)
        dist.all_reduce(d2h)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = evals_per_step * args.steps / (total_ms * 1e-3)
    peak, peak_kind = measured_peak()
    mean_ms = {k: statistics.mean(x[k] for x in kernel_ms) for k in kernel_ms[0]}
    dom = max(("thread_ms", "group_ms", "block_ms"), key=lambda k: mean_ms[k])
    # block_ms covers the block kernels (block mapping) and the one-warp-per-placement kernel (other mappings)
    dom_kernel = {"thread_ms": "eval_thread_kernel", "group_ms": "eval_group_kernel",
                  "block_ms": "eval_block_kernel" if args.mapping == 1 else "eval_wide_kernel"}[dom]
    dom_ms = mean_ms[dom]
    # the dominant kernel's launch on rank 0 processes rank 0's shard
    abytes = algorithmic_bytes({"offsets": off_np, "inst": inst_np, "profile": cfg["profile"]}, evals_rank)
    achieved = abytes / (dom_ms * 1e-3) / 1e9
    profiled = None
    if (PROFILED and args.workload == PROFILED["workload"] and args.mapping == PROFILED["mapping"] and world == 1 and args.flags == 0
            and args.n_cand is None and args.n_req is None and PROFILED["kernel"] == dom_kernel
            and PROFILED["csrc_sha256"] == csrc_sha256()):
        profiled = PROFILED
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    alu_peak = SM_COUNT * ISSUE_PER_SM * sm_mhz * 1e6
    alu = None
    if profiled:
        ach = profiled["warp_inst_per_launch"] / (dom_ms * 1e-3)
        alu = {"bound": "alu", "kernel": dom_kernel, "achieved": ach / 1e9, "peak": alu_peak / 1e9,
               "unit": "G warp-instructions/s", "frac": ach / alu_peak,
               "peak_kind": f"{SM_COUNT} SMs x {ISSUE_PER_SM} issue slots x {sm_mhz:.0f} MHz sampled during the run",
               "warp_inst_per_eval": profiled["warp_inst_per_launch"] / evals_per_step,
               "source": "warp instructions per launch from the committed ncu summary of these kernel sources "
                         "(source hash checked); kernel time and clock measured in this run"}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": workload_label(cfg["name"], n_total, len(trace_np), n_tr, cfg["budget"]),
                   "evals_per_step": evals_per_step, "mapping": {0: "auto", 1: "block", 2: "lane groups", 3: "threads"}[args.mapping],
                   "engine_flags": args.flags,
                   "l2": "flushed between timed steps (256 MB write)",
                   "per_gpu": "one sweep, contiguous candidate shards" if world > 1 else "the whole sweep"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d.item()),
                "d2h_bytes_per_step": int(d2h.item()),
                "note": "candidate arrays copied in from pinned memory, scoring, top-64, all records and the selection "
                        "copied out, every step (after the same 256 MB L2 flush as the timed steps); host wall clock"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": dom_kernel,
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}",
                     "traffic": profiled["dram_bytes_per_launch"] if profiled else None,
                     "algorithmic_bytes_per_launch": abytes, "kernel_ms": dom_ms,
                     "note": "effective bytes (16 B trace record per evaluation); the path is bound by "
                             "integer issue of a dependent event chain, not by DRAM"},
        "roofline_alu": alu,
        "kernel_ms": mean_ms,
    }
    if not args.no_scale_slice and world == 1 and args.workload == "multimodel" and args.n_cand is None and args.n_req is None:
        ctx.close()
        del results, flush
        torch.cuda.empty_cache()
        line["scale_slice"] = scale_slice(m, torch, local, args.mapping)
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Throughput benchmark of the placement-scoring path.

One step = one pass of the whole path over one batch: candidate validation, trace replay
for every candidate (distributor + continuous batching) and the top-64 selection, on the
single-node sweep (10,864 placements of <= 8 devices x a 10,000-request trace).
Prints ONE JSON line.  `--impl reference` times the CPU oracle instead.
"""
import argparse
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

# ncu counters of eval_group_kernel on the default workload (profiles/eval_group_kernel_node_sweep.md).
# They describe the kernel as committed with that summary; set to None when the kernel changes.
PROFILED = {"workload": "node", "mapping": 0,
            "dram_bytes_per_launch": 49_585_664 + 36_903_424,
            "warp_inst_per_launch": 4_299_223_620,
            "alu_pipe_busy": 0.412}   # sm__inst_executed_pipe_alu, share of its peak while an SM is active
SM_COUNT, ISSUE_PER_SM = 148, 4   # B200: 148 SMs x 4 warp schedulers, one warp instruction per cycle each


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


FULL_CANDIDATES = {"tiny": 143, "node": 10_864, "bursty": 10_864, "multimodel": 100_000, "scale": 1_000_000}


def workload_label(name, n_cand, n_req, n_tr, budget):
    """One name for a workload, the same in both arms."""
    return (f"{name} sweep: {n_cand} placements x {n_req} requests"
            f"{f' x {n_tr} traces in one pass' if n_tr > 1 else ''}, budget {budget}, top-{TOPK}")


def oracle_pass(oracle, cfg):
    res = oracle.eval_placements(cfg["profile"], cfg["traces"][0], cfg["classes"], cfg["offsets"],
                                 cfg["inst"], cfg["budget"])
    oracle.topk(res, TOPK)
    return int(res["n_counted"][res["status"] == 0].astype(np.int64).sum())


def run_reference(args):
    """The CPU oracle as it stands, one thread, on a bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import gen
    import oracle
    oracle.build()
    sample_cands = 1024
    if args.workload in ("tiny", "node", "bursty"):
        # enumerated sweeps are ordered from small to large placements: take every k-th one
        cfg = gen.make_config(args.workload, n_cand=args.n_cand, n_req=args.n_req)
        off = cfg["offsets"].astype(np.int64)
        pick = np.arange(0, len(off) - 1, max(1, (len(off) - 1) // sample_cands))[:sample_cands]
        parts = [cfg["inst"][off[c]:off[c + 1]] for c in pick]
        cfg["offsets"] = np.concatenate([[0], np.cumsum([len(x) for x in parts])]).astype(np.uint32)
        cfg["inst"] = np.concatenate(parts).astype(np.uint32)
        how = f"every {max(1, (len(off) - 1) // sample_cands)}th placement ({len(pick)})"
    else:
        cfg = gen.make_config(args.workload, n_cand=sample_cands, n_req=args.n_req)
        how = f"{sample_cands} placements drawn like the sweep's"
    times, evals = [], 0
    for step in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        ev = oracle_pass(oracle, cfg)
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
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": workload_label(cfg["name"], n_full, len(cfg["traces"][0]), len(cfg["traces"]),
                                              cfg["budget"]), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(args):
    """Oracle throughput on this host, one thread.  The default workload is small enough for the
    oracle to run it whole (about 5 s); other workloads are cut to a bounded sample."""
    import gen
    import oracle
    oracle.build()
    sample_cands = args.n_cand if args.workload == "node" else min(args.n_cand or 512, 512)
    sample_req = args.n_req if args.workload == "node" else min(args.n_req or 20_000, 20_000)
    cfg = gen.make_config(args.workload, n_cand=sample_cands, n_req=sample_req)
    t0 = time.perf_counter()
    evals = oracle_pass(oracle, cfg)
    dt = time.perf_counter() - t0
    n_c = len(cfg["offsets"]) - 1
    return {"value": evals / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n_c} placements x {len(cfg['traces'][0])} requests of the same sweep"
                      f"{' (the whole workload)' if args.workload == 'node' and not args.n_cand and not args.n_req else ''}"
                      f", {dt:.1f} s, 1 thread"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mapping", type=int, default=0, help="0 auto (lane groups), 1 block layout")
    ap.add_argument("--workload", default="node", help="node (default) or another configuration name")
    ap.add_argument("--n-cand", type=int, default=None)
    ap.add_argument("--n-req", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import gen
    import paper_2509_06362_b200 as m

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
    n_cand = len(cfg["offsets"]) - 1
    n_tr = len(cfg["traces"])     # more than one: the load sweep, all traces in one pass
    ctx = m.Context(local)
    ctx.load_profile(cfg["profile"])
    traces = [ctx.load_trace(t, cfg["classes"]) for t in cfg["traces"]]
    trace = traces[0]
    d_off, d_inst = ctx.to_device(cfg["offsets"]), ctx.to_device(cfg["inst"])
    results = torch.empty((n_tr * n_cand, 128), dtype=torch.uint8, device=ctx.device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=ctx.device)  # > L2 (126 MB)
    stream = torch.cuda.current_stream()
    ctx.set_timing(True)

    from paper_2509_06362_b200.distributed import global_topk

    def rank_topk(rec, k):
        return ctx.topk(rec, k, stream=stream)

    def step():
        if n_tr > 1:
            ctx.eval_placements_multi(traces, d_off, d_inst, cfg["budget"], out=results, stream=stream)
        else:
            ctx.eval_placements(trace, d_off, d_inst, cfg["budget"], mapping=args.mapping, out=results,
                                stream=stream)
        if world == 1:
            return ctx.topk(results, TOPK, stream=stream)
        # every rank holds its own copy of the sweep: global index = rank * n_cand + local index
        return global_topk(rank_topk, rank_topk, results, rank * n_cand, TOPK)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.fill_(1)
        step()
    sync_all()
    rec = ctx.results_to_numpy(results)
    evals_per_step = int(rec["n_counted"][rec["status"] == 0].astype(np.int64).sum())

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
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

    # end to end through the host-buffer entry point: H2D of the candidates from pinned memory,
    # scoring, D2H of the records, every step
    off_pin = torch.from_numpy(cfg["offsets"].view(np.int32)).pin_memory()
    inst_pin = torch.from_numpy(cfg["inst"].view(np.int32)).pin_memory()
    out_pin = torch.empty((n_tr * n_cand, 128), dtype=torch.uint8).pin_memory()
    off_h, inst_h = off_pin.numpy().view(np.uint32), inst_pin.numpy().view(np.uint32)
    out_h = out_pin.numpy().reshape(-1).view(m.RESULT_DTYPE)

    def e2e_step():
        if n_tr > 1:   # the joint pass has no host-buffer entry point: same copies, made here
            d_off.copy_(off_pin, non_blocking=True)
            d_inst.copy_(inst_pin, non_blocking=True)
            ctx.eval_placements_multi(traces, d_off, d_inst, cfg["budget"], out=results, stream=stream)
            out_pin.copy_(results.view(n_tr * n_cand, 128), non_blocking=True)
            torch.cuda.synchronize()
        else:
            ctx.eval_placements_host(trace, off_h, inst_h, cfg["budget"], mapping=args.mapping, out=out_h)

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
    e2e_value = evals_per_step * world * e2e_steps / float(e2e_s.item())
    assert out_h.tobytes() == rec.tobytes(), "host entry point disagrees with the device entry point"

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = evals_per_step * world * args.steps / (total_ms * 1e-3)
    peak, peak_kind = measured_peak()
    dom = "group_ms" if args.mapping == 0 else "block_ms"
    dom_ms = statistics.mean(k[dom] for k in kernel_ms)
    abytes = algorithmic_bytes(cfg, evals_per_step)
    achieved = abytes / (dom_ms * 1e-3) / 1e9
    profiled = (PROFILED if PROFILED and args.workload == PROFILED["workload"] and args.mapping == PROFILED["mapping"]
                and args.n_cand is None and args.n_req is None else None)
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    alu_peak = SM_COUNT * ISSUE_PER_SM * sm_mhz * 1e6
    alu = None
    if profiled:
        ach = profiled["warp_inst_per_launch"] / (dom_ms * 1e-3)
        alu = {"bound": "alu", "kernel": "eval_group_kernel", "achieved": ach / 1e9, "peak": alu_peak / 1e9,
               "unit": "G warp-instructions/s", "frac": ach / alu_peak,
               "peak_kind": f"{SM_COUNT} SMs x {ISSUE_PER_SM} issue slots x {sm_mhz:.0f} MHz sampled during the run",
               "warp_inst_per_eval": profiled["warp_inst_per_launch"] / evals_per_step,
               "alu_pipe_busy_profiled": profiled["alu_pipe_busy"]}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": workload_label(cfg["name"], n_cand, len(trace_np), n_tr, cfg["budget"]),
                   "evals_per_step": evals_per_step, "mapping": "lane groups" if args.mapping == 0 else "block",
                   "l2": "flushed between timed steps (256 MB write)", "per_gpu": "same sweep on every rank"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": int(cfg["offsets"].nbytes + cfg["inst"].nbytes),
                "d2h_bytes_per_step": int(n_tr * n_cand * 128),
                "note": "host-buffer entry point: candidates copied in, all records copied out, every step; "
                        "no top-k pass and no L2 flush between steps, hence a little above the device-timed value"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "eval_group_kernel" if args.mapping == 0 else "eval_block_kernel",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}",
                     "traffic": profiled["dram_bytes_per_launch"] if profiled else None,
                     "algorithmic_bytes_per_launch": abytes, "kernel_ms": dom_ms,
                     "note": "effective bytes (16 B trace record per evaluation); the path is bound by "
                             "integer issue of a dependent event chain, not by DRAM"},
        "roofline_alu": alu,
        "kernel_ms": {k: statistics.mean(x[k] for x in kernel_ms) for k in kernel_ms[0]},
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the repair search on the thread-binding workload (256x256 matmul tile nest:
bx in [0,64), tx in [0,256), k in [0,8); 136 leaves; expression size <= 7; 213 939 625 416
candidates x 131 072 domain points).

A step is one complete search (every size, counts and least solution) of one seeded instance.
Prints one JSON line.  ``--impl reference`` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate_point_evals_per_s"
UNIT = "GInt-evals/s"
WORKLOAD = "config2_thread_binding_matmul256_size7"
# dram__bytes_read.sum + dram__bytes_write.sum of one eval_kernel launch on this workload, from the ncu capture
# summarised in profiles/eval_kernel_config2.md (local-memory frames; the path is bound by the integer ALUs).
# Set to None whenever eval_kernel changes, until the capture has been taken again.
EVAL_KERNEL_DRAM_BYTES = 5.02e9
ORACLE_SAMPLE_RANKS = 500_000_000          # ranks of size 7 the oracle is timed on (about 15-25 s of one core)


def oracle_sample(seed: int, n_ranks: int):
    """Times the CPU oracle, as it stands, on a rank window of the benchmark instance."""
    import oracle
    from xp_instances import config2
    sk = config2(seed)
    oracle.build()
    n7 = oracle.counts(sk.grammar, 0, 7)[7]
    lo = n7 // 3                            # a window inside the size-7 space, away from its first block
    t0 = time.perf_counter()
    r = oracle.repair_hole(sk, rank_ranges={1: (0, 0), 3: (0, 0), 5: (0, 0), 7: (lo, lo + n_ranks)})
    dt = time.perf_counter() - t0
    return r.evals, dt, f"size-7 ranks [{lo}, {lo + n_ranks}) of seed {seed}, single thread"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm = sorted(int(r[0]) for r in self.rows if r and r[0].isdigit())
        mx = [int(r[1]) for r in self.rows if len(r) > 1 and r[1].isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) > 3 + i and r[3 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(1_000_000, ORACLE_SAMPLE_RANKS // max(1, args.steps + args.warmup))
    for _ in range(args.warmup):
        oracle_sample(0, per_step // 8)
    evals, secs, sample = 0, 0.0, ""
    for _ in range(args.steps):
        e, dt, sample = oracle_sample(0, per_step)
        evals += e
        secs += dt
    value = evals / secs / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle on a bounded rank window per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample + " per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_batch(args, xp, torch, sketches, stream):
    """Profiling aid (single GPU): the batched workload, 4096 small instances in one
    ``xp_repair_batch`` call per step; prints a short JSON line of its own."""
    grammars, loaded = {}, []
    for sk in sketches:
        key = tuple(v.hi for v in sk.grammar.variables)
        if key not in grammars:
            grammars[key] = xp.xp_grammar_create(sk.grammar)
        loaded.append(xp.xp_sketch_load(grammars[key], sk))
    ws = torch.empty(xp.xp_workspace_bytes(loaded), dtype=torch.uint8, device="cuda")
    peak_add, _ = xp.xp_int32_peak()
    for _ in range(max(3, args.warmup)):
        xp.xp_repair_batch(loaded, workspace=ws, stream=stream.cuda_stream)
    torch.cuda.synchronize()
    dev_ms = kern_ms = 0.0
    evals = ops = cand = 0
    for _ in range(args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        res = xp.xp_repair_batch(loaded, workspace=ws, stream=stream.cuda_stream)
        e1.record(stream)
        e1.synchronize()
        dev_ms += e0.elapsed_time(e1)
        kern_ms += res[0][0].kernel_ms
        evals += sum(r[0].evals_executed for r in res)
        ops += sum(r[0].nominal_ops for r in res)
        cand += sum(sum(r[0].cand_count) for r in res)
    print(json.dumps({"metric": METRIC, "value": evals / (dev_ms * 1e-3) / 1e9, "unit": UNIT, "steps": args.steps,
                      "ms_per_step": dev_ms / args.steps, "kernel_ms_per_step": kern_ms / args.steps,
                      "time_to_solution_ms": res[0][0].total_ms,
                      "config": {"workload": "config5_batch_%d_instances" % len(loaded), "candidates_per_step": cand // args.steps},
                      "candidates_per_s": cand / (dev_ms * 1e-3),
                      "roofline": {"bound": "alu", "achieved": ops / (kern_ms * 1e-3) / 1e9, "peak": peak_add / 1e9,
                                   "unit": "G int32-op/s", "frac": ops / (kern_ms * 1e-3) / peak_add}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="config2", choices=["config2", "config3", "config4", "config5"],
                    help="profiling aid: time another config's instance instead (the bench line is config2's)")
    ap.add_argument("--instances", type=int, default=4096,
                    help="profiling aid: number of instances of the config5 batch (a small case of the same kernels)")
    ap.add_argument("--window", type=int, default=0,
                    help="profiling aid: search only the first WINDOW ranks of size 7 (a small case of the same kernel)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2505_02146_b200 as xp
    from xp_instances import config2, config3, config4, config5

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device: there is no CPU fallback"
    torch.cuda.set_device(local)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:      # launched by torchrun: one rank per GPU over NCCL
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    xp.load()

    # Independent problems shard with no data-path exchange.  Every rank searches its own copy of the seed-0
    # instance: the work per GPU is then the same at every N (instances of other seeds differ in cost by up to
    # 2.5x, which would measure the instances rather than the machine).
    stream = torch.cuda.current_stream()
    if args.workload == "config5":
        run_batch(args, xp, torch, config5(0, args.instances), stream)
        return
    sk = {"config2": config2, "config3": config3, "config4": config4}[args.workload](0)
    gr = xp.xp_grammar_create(sk.grammar)
    ls = xp.xp_sketch_load(gr, sk)
    ws = torch.empty(xp.xp_workspace_bytes([ls]), dtype=torch.uint8, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")      # > L2 (126 MB), written between steps

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peak_add, peak_mad = xp.xp_int32_peak()
    rr = [(0, 7, 0, args.window)] if args.window else None
    for _ in range(max(3, args.warmup)):
        res = xp.xp_repair(ls, workspace=ws, stream=stream.cuda_stream, rank_ranges=rr)[0]

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    dev_ms = kern_ms = 0.0
    evals = ops = launches = 0
    for _ in range(args.steps):
        flush.fill_(1)                                    # L2 flush, outside the events
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        res = xp.xp_repair(ls, workspace=ws, stream=stream.cuda_stream, rank_ranges=rr)[0]
        e1.record(stream)
        e1.synchronize()
        dev_ms += e0.elapsed_time(e1)
        kern_ms += res.kernel_ms
        evals += res.evals_executed
        ops += res.nominal_ops
        launches += res.n_launches
    barrier()
    clocks = sampler.stop() if rank == 0 else None

    # End to end through the public API with host buffers: grammar and sketch are encoded and
    # copied to the device, searched, and the result read back, every step.
    for _ in range(2):                                   # untimed: the first loads after the sampler exits are erratic
        l2 = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
        xp.xp_repair(l2, rank_ranges=rr)
        del l2
    barrier()
    t0 = time.perf_counter()
    e2e_evals = 0
    for _ in range(args.steps):
        g2 = xp.xp_grammar_create(sk.grammar)
        l2 = xp.xp_sketch_load(g2, sk)
        r2 = xp.xp_repair(l2, rank_ranges=rr)[0]
        e2e_evals += r2.evals_executed
        if os.environ.get("XP_BENCH_DEBUG"):
            print("e2e step: kernel_ms %.2f total_ms %.2f since start %.1f ms" % (r2.kernel_ms, r2.total_ms, 1e3 * (time.perf_counter() - t0)), file=sys.stderr)
        del l2, g2
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    # Bytes that cross the bus per end-to-end step (structure sizes of the library, 256-byte aligned pieces):
    # grammar block (header 1128, leaves 16 each, binary productions 152 each); sketch head (sketch record 824,
    # hole record 5008 and a flag word per hole); job list of the load; plan head of the search (counters,
    # segments 200 each, sketch pointer, accumulators 296 per hole).  Back: hole records and flags after the load,
    # accumulators after the search.  Host tables of a table domain would add their own size (config 2 is a box).
    al = lambda b: (b + 255) // 256 * 256
    n_bin = sum(1 for p in sk.grammar.productions if p.kind == 2)
    n_leaf = len(sk.grammar.productions) - n_bin
    nh, n_segs = len(sk.holes), 16
    h2d = (al(1128) + al(16 * (n_leaf + 1)) + 152 * (n_bin + 1)) + (al(824) + al(5012 * nh)) + (al(8) + 16 * nh) + \
          (256 + al(200 * (n_segs + 1)) + al(8 * 2) + al(296 * (nh + 1)))
    d2h = 5012 * nh + 296 * nh

    tot = torch.tensor([dev_ms, float(evals), e2e_s, float(e2e_evals), kern_ms, float(ops)], dtype=torch.float64, device="cuda")
    if dist is not None:
        mx = tot.clone(); dist.all_reduce(mx, op=dist.ReduceOp.MAX)
        sm = tot.clone(); dist.all_reduce(sm, op=dist.ReduceOp.SUM)
        dev_ms, e2e_s, kern_ms = float(mx[0]), float(mx[2]), float(mx[4])
        evals, e2e_evals, ops = float(sm[1]), float(sm[3]), float(sm[5])
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = evals / (dev_ms * 1e-3) / 1e9
    cand = sum(res.cand_count)
    achieved = (ops / world) / (kern_ms * 1e-3) / 1e9                  # per GPU, G int32-op/s
    peak = peak_add / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": dev_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int64", "data": "synthetic",
        "config": {"workload": (WORKLOAD if args.workload == "config2" else args.workload) +
                               (f"_first_{args.window}_ranks_of_size7" if args.window else ""),
                   "candidates_per_step": cand, "domain_points": sk.n_points,
                   "nominal_evals_per_step": cand * sk.n_points, "l2": "flushed between steps (256 MiB write)",
                   "time_to_solution_ms": res.total_ms, "kernel_ms_per_step": kern_ms / args.steps,
                   "candidates_per_s": cand * args.steps * world / (dev_ms * 1e-3),
                   "filter_survivors": res.filter_survivors, "probe_survivors": res.probe_survivors,
                   "least": res.least_text, "match_count": res.match_count},
        "clocks": clocks,
        "e2e": {"value": e2e_evals / e2e_s / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "G int32-op/s", "frac": achieved / peak,
                     "traffic": EVAL_KERNEL_DRAM_BYTES if args.workload == "config2" and not args.window else None,
                     "kernel": "eval_kernel",
                     "peak_source": "measured live: independent 32-bit add chains (xp_int32_peak); multiply-add chains reach %.0f" % (peak_mad / 1e9),
                     "model": "32-bit operations of one operation + one comparison per candidate-point evaluation of the filter stage"},
    }
    if not args.no_cpu_baseline and args.workload == "config2":
        e, dt, sample = oracle_sample(0, ORACLE_SAMPLE_RANKS)
        out["cpu_baseline"] = {"value": e / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                               "seconds": dt, "host_cores_present": os.cpu_count()}
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the fused GEMM-ReduceScatter hot path (one-rank emulation on one B200).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one entwine_gemm_rs call (schedule already planned; GEMM + per-tile flags + scatter
push + reduction in one launch) over one batch of seeded synthetic input.  The headline value
is 2*M*N*K_local / device time, with inputs resident in HBM and the L2 flushed between timed
steps.  One JSON line is printed on stdout by rank 0.

With --gpus N > 1 (under torchrun) every rank runs an independent replica of the same problem
on its own GPU (the path does not shard: "replicas only"); no data-path collective is issued.

--impl reference times the CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused GEMM-RS TFLOP/s and fraction of max(tensor peak, HBM) roofline"
# Peaks measured on this machine (used only if MEASURED_PEAKS.json is absent).
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch) of the fused kernel from
# the ncu capture of the named workload that profiles/ summarises; the summary file is carried
# beside the number so that a stale figure can be told from a fresh one.
NCU_TRAFFIC = {
    "attn_out_proj": {"bytes": 55.89e6, "summary": "profiles/fused_kernel_attn_out_proj.md"},
    "mlp_down_proj": {"bytes": 826.88e6, "summary": "profiles/fused_kernel_mlp_down_and_short_k.md"},
    "short_k_comm_bound": {"bytes": 514.21e6, "summary": "profiles/fused_kernel_mlp_down_and_short_k.md"},
}
# Launch configuration per workload: communication SMs, tile order.
# Launch configuration per workload (the best point of a budget x order scan on B200): number of
# dedicated communication SMs (0 = consumer warps co-located with the producer in every CTA),
# tile order (1 = interleaved, Eq. 1; 0 = row-major).
LAUNCH = {
    "attn_out_proj": dict(n_comm_sms=0, order=1, rank=1),
    "mlp_down_proj": dict(n_comm_sms=0, order=1, rank=5),
    "short_k_comm_bound": dict(n_comm_sms=0, order=1, rank=2),
    "tiny": dict(n_comm_sms=4, order=1, rank=0),
}


def apply_tuned_table():
    """Overlays the package's tuning table (written by paper_2609_11562_b200.autotune on a B200)
    on LAUNCH: tile order, budget, and the producer options the tuner chose."""
    from paper_2609_11562_b200 import autotune as T
    from paper_2609_11562_b200 import inputs as I
    path = os.path.join(ROOT, "paper_2609_11562_b200", "tuned_b200.json")
    if not os.path.exists(path):
        return
    table = T.load_table(path)
    for name, cfg in LAUNCH.items():
        wl = I.CONFIGS[name]
        if T.shape_key(wl.M, wl.N, wl.K, wl.W) not in table["shapes"]:
            continue
        order, n_comm, opts = T.launch_options(table, wl.M, wl.N, wl.K, wl.W)
        cfg.update(order=order, n_comm_sms=n_comm, opts=opts)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def roofline_seconds(wl, peaks):
    t_tc = wl.flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = wl.comm_bytes / (peaks["hbm_gbs"] * 1e9)
    return t_tc, t_hbm


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def lines(self):
        try:
            return sum(1 for _ in open(self.path))
        except Exception:
            return 0

    def wait_for_samples(self, n, timeout_s=10.0):
        t0 = time.perf_counter()
        while self.proc is not None and self.lines() < n and time.perf_counter() - t0 < timeout_s:
            time.sleep(0.02)

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [v.strip() for v in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def max_over_ranks(value, dist, device):
    """Largest per-rank value (ranks run independent replicas; the job is as slow as its slowest)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(world, flops_per_rank, seconds):
    """Aggregate throughput of `world` replicas that each did flops_per_rank in `seconds`."""
    return world * flops_per_rank / seconds / 1e12


def _dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), \
        int(os.environ.get("WORLD_SIZE", "1"))


def blas_threads():
    """Threads of the BLAS pool behind numpy's matmul (what the oracle's float64 GEMM runs on),
    after setting it to the cores this process may use."""
    cores = len(os.sched_getaffinity(0))
    try:
        import threadpoolctl
        threadpoolctl.threadpool_limits(limits=cores, user_api="blas")
        pools = [p for p in threadpoolctl.threadpool_info() if p.get("user_api") == "blas"]
        if pools:
            return max(int(p["num_threads"]) for p in pools)
    except Exception:
        pass
    return cores


def run_cpu_oracle(wl, launch, rows_per_pass, passes):
    """Times the oracle (float64 GEMM of the sampled rows + reduce-scatter definition + the
    whole integer schedule) and returns (seconds per pass, flops of one pass, threads used)."""
    import numpy as np
    from oracle import entwine_oracle as O
    from paper_2609_11562_b200 import inputs as I
    threads = blas_threads()
    A, Bm = I.make_operands(wl)
    P = I.make_peer_partials(wl)
    Ab, Bb, Pb = I.bits(A), I.bits(Bm), I.bits(P)
    r = launch["rank"]
    x = launch["n_comm_sms"] or 148
    full = rows_per_pass >= wl.M
    rows = None if full else np.linspace(0, wl.M - 1, rows_per_pass).astype(np.int64)
    times = []
    for _ in range(passes):
        t0 = time.perf_counter()
        O.gemm_rs(Ab, Bb, Pb, r, wl.W, 256, launch["order"], x, rows=rows)
        times.append(time.perf_counter() - t0)
    n_rows = wl.M if full else rows_per_pass
    return times, 2.0 * n_rows * wl.N * wl.K, threads


def main_reference(args, wl, launch):
    rank, _, world = _dist_env()
    if rank != 0:
        return 0
    # size the per-step sample so that the whole run stays within a couple of minutes
    probe, flops_probe, threads = run_cpu_oracle(wl, launch, min(256, wl.M), 1)
    sec_per_row = probe[0] / min(256, wl.M)
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = int(max(128, min(wl.M, (budget / max(sec_per_row, 1e-9)) // 128 * 128)))
    times, flops, threads = run_cpu_oracle(wl, launch, rows, args.steps + args.warmup)
    timed = times[args.warmup:]
    mean = sum(timed) / len(timed)
    value = flops / mean / 1e12
    sample = (f"{rows} of {wl.M} rows of the float64 partial GEMM and its magnitude sums + the full "
              f"integer schedule per step" + (" + reduce-scatter definition" if rows >= wl.M else ""))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "W": wl.W, "M": wl.M, "N": wl.N, "K_local": wl.K,
                   "tile_order": "interleaved" if launch["order"] else "row_major"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def time_steps(fn, steps, warmup, flush, torch, cold=True):
    """Device time of `steps` calls of fn with the L2 flushed before each (cold) or not; µs list."""
    for _ in range(warmup):
        if cold:
            flush.zero_()
        fn()
    torch.cuda.synchronize()
    evs = []
    for _ in range(steps):
        if cold:
            flush.zero_()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) * 1e3 for a, b in evs]


def measure_workload(wl, launch, steps, warmup, flush, torch, E, I, detailed):
    """All device-side numbers of one workload on the current device."""
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], launch["n_comm_sms"], rank=launch["rank"],
                  **launch.get("opts", {}))
    res = {}
    us = time_steps(lambda: plan.gemm_rs(A, Bm, P, out, send), steps, warmup, flush, torch)
    st = plan.last_status()
    res["fused_us"] = us
    res["status"] = st
    res["sm_mhz"] = plan.last_sm_clock_mhz()
    res["fused_hot_us"] = time_steps(lambda: plan.gemm_rs(A, Bm, P, out, send), steps, 3, flush, torch, cold=False)
    plan.last_status()
    # Back to back: `steps` calls queued between ONE event pair, no flush.  The queue hides the
    # launch latency of all calls but the first; a call's streamed data (partial C, incoming
    # partials, outputs) exceeds L2 for every configuration but the tiny one, so L2 holds at
    # most the operands when the next call starts.
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        plan.gemm_rs(A, Bm, P, out, send)
    e1.record()
    torch.cuda.synchronize()
    res["fused_back_to_back_us"] = e0.elapsed_time(e1) * 1e3 / steps
    plan.last_status()
    # CUDA-graph replay: the same queue of calls captured once (each preceded by the library's
    # reset kernel, see include/entwine.h) and replayed between one event pair.  A plan of its
    # own, so that the eager plan above keeps launching without the reset kernel.
    n_cap = min(steps, 50)
    gplan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], launch["n_comm_sms"], rank=launch["rank"],
                   **launch.get("opts", {}))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        gplan.gemm_rs(A, Bm, P, out, send)
        gplan.last_status()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(n_cap):
                gplan.gemm_rs(A, Bm, P, out, send)
        graph.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        side.synchronize()
        gplan.last_status()
    res["fused_graph_replay_us"] = e0.elapsed_time(e1) * 1e3 / n_cap
    del graph
    gplan.destroy()
    if detailed:
        time.sleep(0.5)  # the queued calls above are a sustained load: let the clock recover
        # the producer alone (uncontended GEMM time) and the consumer alone
        res["gemm_only_us"] = time_steps(lambda: plan.gemm_only(A, Bm), max(5, steps // 4), 3, flush, torch)
        plan.last_status()
        res["comm_only_us"] = time_steps(lambda: plan.comm_only(None, P, out, send, 0), max(5, steps // 4), 3,
                                         flush, torch)
        plan.last_status()
        # unfused sequence: library GEMM into a bf16 [M,N] buffer, then reduce + scatter on all SMs
        Cfull = torch.empty(wl.M, wl.N, dtype=torch.bfloat16, device="cuda")
        plan0 = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], 0, rank=launch["rank"])

        def unfused():
            torch.matmul(A, Bm.t(), out=Cfull)
            plan0.comm_only(Cfull, P, out, send, 0)
        res["unfused_us"] = time_steps(unfused, max(5, steps // 4), 3, flush, torch)
        plan0.last_status()
        res["cublas_gemm_us"] = time_steps(lambda: torch.matmul(A, Bm.t(), out=Cfull), max(5, steps // 4), 3,
                                           flush, torch)
        plan0.destroy()
        del Cfull
        # Pull mode (the rank's call when the W ranks have GPUs of their own): this rank's kernel
        # with the peers' contributions already in their heap segments and flagged, this GPU's
        # HBM standing in for the reads over NVLink.  No push tasks: a peer's pull is its own work.
        time.sleep(0.5)
        seg, flags_off = plan.heap_bytes()
        heap = torch.zeros(wl.W * seg, dtype=torch.uint8, device="cuda")
        r = launch["rank"]
        Q = plan.counts()["Q"]
        for w in range(wl.W):
            if w != r:
                heap[w * seg:w * seg + flags_off].view(torch.bfloat16).normal_()
        fl = heap[r * seg + flags_off:r * seg + flags_off + wl.W * Q * 4].view(torch.int32).view(wl.W, Q)
        fl.fill_(0x7fffffff)  # every peer is ahead of any call number used here
        fl[r].zero_()         # the rank's own flags are published by each call
        pplan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], launch["n_comm_sms"], rank=r,
                       **launch.get("opts", {}))
        calls = [0]

        def pull():
            calls[0] += 1
            pplan.gemm_rs_pull(A, Bm, heap, seg, calls[0], out)
        res["pull_us"] = time_steps(pull, max(5, steps // 4), 3, flush, torch)
        st = pplan.last_status()
        assert st["tiles_reduced"] == pplan.counts()["n_reduce"] and st["tiles_pushed"] == 0
        pplan.destroy()
        del heap, fl
    plan.destroy()
    return res


def run_sweep(args, peaks, flush, torch, E, I):
    """The sweep configuration: every shape x communication budget x tile order, fused call only.
    One JSON line per point goes to --sweep-out; stdout gets one summary line."""
    os.makedirs(os.path.dirname(args.sweep_out), exist_ok=True)
    n_points, best = 0, {}
    with open(args.sweep_out, "w") as f:
        for wl in I.sweep_workloads():
            A, Bm = I.make_operands(wl, device="cuda")
            P = I.make_peer_partials(wl, device="cuda")
            out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
            send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
            tc, hb = roofline_seconds(wl, peaks)
            for order in (1, 0):
                for n_comm in I.SWEEP_COMM_SMS:
                    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=wl.W - 1)
                    us = time_steps(lambda: plan.gemm_rs(A, Bm, P, out, send), args.sweep_iters, 2, flush, torch)
                    st = plan.last_status()
                    c = plan.counts()
                    assert st["tiles_reduced"] == c["n_reduce"] and st["tiles_pushed"] == c["n_push"]
                    if n_comm == I.SWEEP_COMM_SMS[0]:
                        # the properties that hold at any size, once per shape and order: what was
                        # pushed is the stored partial, what was reduced is its fp32 rank-order sum
                        r, R = wl.W - 1, wl.R
                        Cd = torch.empty(wl.M, wl.N, dtype=torch.bfloat16, device="cuda")
                        plan.read_partial(Cd)
                        torch.cuda.synchronize()
                        for slot, d in enumerate(dd for dd in range(wl.W) if dd != r):
                            assert torch.equal(send[slot], Cd[d * R:(d + 1) * R])
                        acc = Cd[r * R:(r + 1) * R].float()
                        for q in range(wl.W - 1):
                            acc = acc + P[q, r * R:(r + 1) * R].float()
                        assert torch.equal(out, acc.to(torch.bfloat16))
                        del Cd, acc
                    med = statistics.median(us)
                    rec = {"M": wl.M, "N": wl.N, "K_local": wl.K, "W": wl.W, "n_comm_sms": n_comm,
                           "tile_order": "interleaved" if order else "row_major", "fused_us": med,
                           "tflops": wl.flops / med / 1e6, "roofline_us": max(tc, hb) * 1e6,
                           "roofline_frac": max(tc, hb) * 1e6 / med, "bound": "tensor" if tc >= hb else "hbm",
                           "t_gemm_us": st["t_gemm_ns"] / 1e3, "t_end_us": st["t_end_ns"] / 1e3}
                    f.write(json.dumps(rec) + "\n")
                    n_points += 1
                    key = (wl.M, wl.K, wl.W)
                    if key not in best or med < best[key]["fused_us"]:
                        best[key] = rec
                    plan.destroy()
            del A, Bm, P, out, send
            torch.cuda.empty_cache()
    fr = [b["roofline_frac"] for b in best.values()]
    inter = sum(1 for b in best.values() if b["tile_order"] == "interleaved")
    print(json.dumps({"sweep_points": n_points, "shapes": len(best), "out": args.sweep_out,
                      "best_roofline_frac": {"min": min(fr), "median": statistics.median(fr), "max": max(fr)},
                      "shapes_where_interleaved_is_best": inter,
                      "best_budget_histogram": {str(k): sum(1 for b in best.values() if b["n_comm_sms"] == k)
                                                for k in I.SWEEP_COMM_SMS}}))
    return 0


def run_ablation(args, peaks, flush, torch, E, I):
    """The design ablations of Sec. 5 on this GPU: computation order, release granularity and
    SM sharing, each on a short-K and a long-K shape.  Every variant is the same kernel with
    another plan option; each line reports the variant's best communication budget."""
    iters = args.sweep_iters
    shapes = [I.Workload("ablation_short_K", 8, 8192, 8192, 1024, "normal_fanin", "normal_fanin", 6, 0),
              I.Workload("ablation_long_K", 8, 8192, 8192, 4096, "normal_fanin", "normal_fanin", 6, 1)]
    report = {}
    for wl in shapes:
        A, Bm = I.make_operands(wl, device="cuda")
        P = I.make_peer_partials(wl, device="cuda")
        out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")

        def fused(order, n_comm, **opts):
            # the slower of the first and the last rank: a collective ends with its slowest rank,
            # and in the grouped orders a rank's own tiles come early or late in the traversal
            worst = None
            for rank in (0, wl.W - 1):
                plan = E.Plan(wl.M, wl.N, wl.K, wl.W, order, n_comm, rank=rank, **opts)
                us = statistics.median(time_steps(lambda: plan.gemm_rs(A, Bm, P, out, send), iters, 3, flush, torch))
                st = plan.last_status()
                plan.destroy()
                if worst is None or us > worst["fused_us"]:
                    worst = {"fused_us": us, "t_gemm_us": st["t_gemm_ns"] / 1e3, "slowest_rank": rank,
                             "tail_us": (st["t_end_ns"] - st["t_gemm_ns"]) / 1e3, "n_comm_sms": n_comm}
            return worst

        def best(order, budgets, **opts):
            return min((fused(order, b, **opts) for b in budgets), key=lambda r: r["fused_us"])

        plan = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=wl.W - 1)
        gemm_us = statistics.median(time_steps(lambda: plan.gemm_only(A, Bm), iters, 3, flush, torch))
        plan.last_status()
        comm_us = statistics.median(time_steps(lambda: plan.comm_only(None, P, out, send, 0), iters, 3, flush, torch))
        plan.last_status()
        plan.destroy()
        base = gemm_us + comm_us  # the non-overlapped baseline: producer alone, then consumer alone
        budgets = (0, 8, 16, 32)
        rec = {"shape": {"W": wl.W, "M": wl.M, "N": wl.N, "K_local": wl.K},
               "non_overlapped_us": base, "gemm_alone_us": gemm_us, "comm_alone_us": comm_us}
        rec["computation_order"] = {name: best(order, budgets) for name, order in
                                    (("interleaved", 1), ("row_major", 0), ("m_major", 2))}
        gran = {}
        for name, g in (("block", 1), ("4_blocks", 4), ("16_blocks", 16), ("64_blocks", 64),
                        ("partition", E.RELEASE_PARTITION), ("whole_output", E.RELEASE_WHOLE)):
            r = best(1, (0, 16), release_group=g)
            r["speedup_vs_non_overlapped"] = base / r["fused_us"]
            gran[name] = r
        rec["release_granularity"] = gran
        rec["sm_sharing"] = {
            "shared_pool": best(1, budgets),
            "static_partition": best(1, (8, 16, 24, 32, 48, 64), colocate=0, tail_help=0),
        }
        report[wl.name] = rec
        del A, Bm, P, out, send
        torch.cuda.empty_cache()
    os.makedirs(args.out_dir, exist_ok=True)
    with open(os.path.join(args.out_dir, "ablation.json"), "w") as f:
        json.dump(report, f, indent=1)
    print(json.dumps({"ablation": report}))
    return 0


def run_layer_chain(args, peaks, flush, torch, E, I):
    """Layer-level chain of Sec. 5.2.3: the attention output of a Llama-3-70B-shaped layer at
    TP = 8 (hidden 8192, K_local = 1024): GEMM + ReduceScatter, residual addition, RMSNorm, at
    three sequence lengths.  One launch (entwine_gemm_rs_norm) against the fused GEMM-RS
    followed by library kernels for the rest, and against the fully unfused sequence."""
    import torch.nn.functional as F
    iters = max(args.sweep_iters, 10)
    report = {}
    for seq in (4096, 8192, 16384):
        wl = I.Workload(f"layer_seq{seq}", 8, seq, 8192, 1024, "normal", "normal_total_fanin", 7, seq // 4096)
        A, Bm = I.make_operands(wl, device="cuda")
        P = I.make_peer_partials(wl, device="cuda")
        res, w = I.make_layer_inputs(wl, device="cuda")
        hidden = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        normed = torch.empty_like(hidden)
        out = torch.empty_like(hidden)
        send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        Cfull = torch.empty(wl.M, wl.N, dtype=torch.bfloat16, device="cuda")
        plan = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=wl.W - 1)
        med = statistics.median

        def rest():
            h = out + res
            return h, F.rms_norm(h, (wl.N,), w, 1e-5)

        def fused_then_library():
            plan.gemm_rs(A, Bm, P, out, send)
            return rest()

        def unfused():
            torch.matmul(A, Bm.t(), out=Cfull)
            plan.comm_only(Cfull, P, out, send, 0)
            return rest()

        one_ring = med(time_steps(lambda: plan.gemm_rs_norm(A, Bm, P, res, w, 1e-5, hidden, normed, send),
                                 iters, 3, flush, torch))
        st = plan.last_status()
        # the same launch with the co-located consumer moving whole tiles through registers instead
        # of the shared-memory TMA ring (plan option reg_consumer = 1): which of the two is faster
        # depends on the shape (few, long reduce tasks per CTA favour the ring), so both are timed and
        # the faster is the chain's figure, as the tuner does for the plain call
        reg_plan = E.Plan(wl.M, wl.N, wl.K, wl.W, 1, 0, rank=wl.W - 1, reg_consumer=1)
        one_reg = med(time_steps(lambda: reg_plan.gemm_rs_norm(A, Bm, P, res, w, 1e-5, hidden, normed, send),
                                  iters, 3, flush, torch))
        st_reg = reg_plan.last_status()
        reg_plan.destroy()
        one = min(one_reg, one_ring)
        if one_reg < one_ring:
            st = st_reg
        two = med(time_steps(fused_then_library, iters, 3, flush, torch))
        plan.last_status()
        three = med(time_steps(unfused, iters, 3, flush, torch))
        plan.last_status()
        rs_only = med(time_steps(lambda: plan.gemm_rs(A, Bm, P, out, send), iters, 3, flush, torch))
        plan.last_status()
        # same numbers as the library chain applied to this launch's hidden stream
        plan.gemm_rs_norm(A, Bm, P, res, w, 1e-5, hidden, normed, send)
        plan.last_status()
        lib = F.rms_norm(hidden, (wl.N,), w, 1e-5)
        max_ulp_diff = float(((normed.float() - lib.float()).abs() / lib.float().abs().clamp_min(1e-3)).max())
        plan.destroy()
        report[f"seq_{seq}"] = {
            "shape": {"W": wl.W, "M": wl.M, "N": wl.N, "K_local": wl.K},
            "one_launch_us": one, "one_launch_consumer": "registers" if one_reg < one_ring else "tma_ring",
            "one_launch_registers_us": one_reg, "one_launch_tma_ring_us": one_ring,
            "gemm_rs_then_library_add_norm_us": two,
            "cublas_reduce_add_norm_us": three, "gemm_rs_alone_us": rs_only,
            "speedup_vs_gemm_rs_then_library": two / one, "speedup_vs_unfused": three / one,
            "chain_cost_over_gemm_rs_us": one - rs_only,
            "t_gemm_us": st["t_gemm_ns"] / 1e3, "t_end_us": st["t_end_ns"] / 1e3,
            "max_rel_diff_vs_library_rms_norm": max_ulp_diff,
        }
        del A, Bm, P, res, w, hidden, normed, out, send, Cfull
        torch.cuda.empty_cache()
    os.makedirs(args.out_dir, exist_ok=True)
    with open(os.path.join(args.out_dir, "layer_chain.json"), "w") as f:
        json.dump(report, f, indent=1)
    print(json.dumps({"layer_chain": report}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="mlp_down_proj",
                    help="default: the largest single-GPU configuration (MLP down-projection)")
    ap.add_argument("--out-dir", default=os.path.join(ROOT, "bench_out"),
                    help="where --sweep, --ablation and --layer-chain write their JSON files")
    ap.add_argument("--impl", default="entwine", choices=["entwine", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations and comparisons")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="run the sweep configuration (60 shapes x budgets 0..32 x both orders), write one "
                         "JSON line per point to --sweep-out and print a summary line")
    ap.add_argument("--sweep-out", default=None, help="default: <out-dir>/sweep.jsonl")
    ap.add_argument("--sweep-iters", type=int, default=8)
    ap.add_argument("--ablation", action="store_true",
                    help="the design ablations (computation order, release granularity, SM sharing) on a "
                         "short-K and a long-K shape; prints one JSON line and writes <out-dir>/ablation.json")
    ap.add_argument("--layer-chain", action="store_true",
                    help="GEMM-RS + residual add + RMSNorm in one launch against library kernels for the rest "
                         "(attention output of a 70B-shaped layer, three sequence lengths)")
    ap.add_argument("--comm-curve", action="store_true",
                    help="consumer bandwidth in isolation against the number of consumer CTAs (App. A)")
    ap.add_argument("--comm-ctas", type=int, default=0,
                    help="with --kernel-only comm: number of consumer CTAs (0 = one per SM)")
    ap.add_argument("--kernel-only", default=None, choices=["fused", "gemm", "comm"],
                    help="profiling aid: run warmup+steps launches of one mode on the workload and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "entwine" else args.warmup
    if args.sweep_out is None:
        args.sweep_out = os.path.join(args.out_dir, "sweep.jsonl")

    from paper_2609_11562_b200 import inputs as I
    apply_tuned_table()
    wl = I.CONFIGS[args.workload]
    launch = LAUNCH[args.workload]
    if args.impl == "reference":
        return main_reference(args, wl, launch)

    import torch
    rank, local_rank, world = _dist_env()
    if not torch.cuda.is_available():
        print("bench.py needs a CUDA device (there is no CPU fallback)", file=sys.stderr)
        return 2
    torch.cuda.set_device(local_rank % torch.cuda.device_count())
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    from paper_2609_11562_b200 import build as B
    if rank == 0:
        B.build()
    if dist is not None:
        dist.barrier()
    from paper_2609_11562_b200 import entwine as E

    peaks = load_peaks()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB of L2
    if args.sweep:
        return run_sweep(args, peaks, flush, torch, E, I)
    if args.ablation:
        return run_ablation(args, peaks, flush, torch, E, I)
    if args.layer_chain:
        return run_layer_chain(args, peaks, flush, torch, E, I)
    if args.comm_curve:
        # every input available, no competing producer: bandwidth against the budget (App. A)
        A, Bm = I.make_operands(wl, device="cuda")
        P = I.make_peer_partials(wl, device="cuda")
        out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        curve = []
        for x in (2, 4, 8, 12, 16, 20, 24, 32, 48, 64, 96, 128, 148):
            plan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], x if x <= 128 else 0, rank=launch["rank"])
            plan.gemm_only(A, Bm)
            us = statistics.median(time_steps(lambda: plan.comm_only(None, P, out, send, x), 6, 2, flush, torch))
            plan.last_status()
            curve.append({"consumer_ctas": x, "us": us, "GBps": wl.comm_bytes / us / 1e3,
                          "GBps_per_cta": wl.comm_bytes / us / 1e3 / x})
            plan.destroy()
        print(json.dumps({"comm_curve": wl.name, "comm_bytes": wl.comm_bytes, "points": curve}))
        return 0
    if args.kernel_only:
        A, Bm = I.make_operands(wl, device="cuda")
        P = I.make_peer_partials(wl, device="cuda")
        out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
        plan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], launch["n_comm_sms"], rank=launch["rank"],
                  **launch.get("opts", {}))
        plan.gemm_only(A, Bm)
        fn = {"fused": lambda: plan.gemm_rs(A, Bm, P, out, send), "gemm": lambda: plan.gemm_only(A, Bm),
              "comm": lambda: plan.comm_only(None, P, out, send, args.comm_ctas)}[args.kernel_only]
        us = time_steps(fn, args.steps, args.warmup, flush, torch)
        plan.last_status()
        print(json.dumps({"kernel_only": args.kernel_only, "workload": wl.name,
                          "median_us": statistics.median(us)}))
        plan.destroy()
        return 0
    dev_uuid = "GPU-" + str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
    sampler = ClockSampler(dev_uuid)

    # ---- headline: timed region of exactly `steps` fused calls -------------------------------
    A, Bm = I.make_operands(wl, device="cuda")
    P = I.make_peer_partials(wl, device="cuda")
    out = torch.empty(wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    send = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16, device="cuda")
    plan = E.Plan(wl.M, wl.N, wl.K, wl.W, launch["order"], launch["n_comm_sms"], rank=launch["rank"],
                  **launch.get("opts", {}))
    sampler.start()
    for _ in range(args.warmup):
        flush.zero_()
        plan.gemm_rs(A, Bm, P, out, send)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    lines_before = sampler.lines()
    t_wall0 = time.perf_counter()
    evs = []
    for _ in range(args.steps):
        flush.zero_()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        plan.gemm_rs(A, Bm, P, out, send)
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t_wall0
    status = plan.last_status()
    kernel_mhz = plan.last_sm_clock_mhz()  # cycle counter against the global timer inside the last timed launch
    # A short timed region can end before nvidia-smi's next sample: keep the same load running,
    # untimed, until two samples under load exist.
    extended = False
    t_ext = time.perf_counter()
    while sampler.proc is not None and sampler.lines() < lines_before + 2 and time.perf_counter() - t_ext < 5.0:
        extended = True
        for _ in range(20):
            flush.zero_()
            plan.gemm_rs(A, Bm, P, out, send)
        torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["sampled"] = ("during the timed region" if not extended else
                         "timed region shorter than the sampling period: same load continued untimed")
    us = [a.elapsed_time(b) * 1e3 for a, b in evs]
    total_us = max_over_ranks(sum(us), dist, "cuda")
    mean_us = total_us / args.steps
    value = whole_job_tflops(world, wl.flops, mean_us * 1e-6)

    # ---- end to end through the host-buffer entry point ---------------------------------------
    hA, hB, hP = A.cpu().pin_memory(), Bm.cpu().pin_memory(), P.cpu().pin_memory()
    hOut = torch.empty(wl.R, wl.N, dtype=torch.bfloat16).pin_memory()
    hSend = torch.empty(wl.W - 1, wl.R, wl.N, dtype=torch.bfloat16).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        plan.gemm_rs_host(hA, hB, hP, hOut, hSend)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        plan.gemm_rs_host(hA, hB, hP, hOut, hSend)
    sync_s = max_over_ranks((time.perf_counter() - t0) / e2e_steps, dist, "cuda")
    # the same steps as a pipeline of depth two: step i's copies up overlap step i-1's copies down
    hOut2 = [hOut, torch.empty_like(hOut).pin_memory()]
    hSend2 = [hSend, torch.empty_like(hSend).pin_memory()]
    for i in range(2):
        plan.gemm_rs_host_begin(hA, hB, hP, hOut2[i], hSend2[i])
    plan.gemm_rs_host_wait()
    plan.gemm_rs_host_wait()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        plan.gemm_rs_host_begin(hA, hB, hP, hOut2[i & 1], hSend2[i & 1])
        if i >= 1:
            plan.gemm_rs_host_wait()
    plan.gemm_rs_host_wait()
    e2e_s = max_over_ranks((time.perf_counter() - t0) / e2e_steps, dist, "cuda")
    plan.last_status()
    h2d = (wl.M * wl.K + wl.N * wl.K + (wl.W - 1) * wl.R * wl.N) * 2
    d2h = (wl.R * wl.N + (wl.W - 1) * wl.R * wl.N) * 2
    e2e = {"value": whole_job_tflops(world, wl.flops, e2e_s), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_s * 1e3,
           "api": "entwine_gemm_rs_host_begin / _wait, two steps in flight (pinned host buffers)",
           "one_step_at_a_time": {"value": whole_job_tflops(world, wl.flops, sync_s), "ms_per_step": sync_s * 1e3,
                                  "api": "entwine_gemm_rs_host"}}
    del hOut2, hSend2
    plan.destroy()
    del hA, hB, hP, hOut, hSend, A, Bm, P, out, send

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant (only) kernel of a step --------------------------------------
    t_tc, t_hbm = roofline_seconds(wl, peaks)
    tensor_bound = t_tc >= t_hbm
    if tensor_bound:
        achieved = wl.flops / (mean_us * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"]}
    else:
        achieved = wl.comm_bytes / (mean_us * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"]}
    # the same time against the other denominators: the seconds-long cuBLAS figure under the power
    # cap, and the nominal HBM bandwidth
    t_alt = max(wl.flops / (peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12), wl.comm_bytes / 8.0e12)
    roof["frac_vs_sustained_tensor_and_nominal_hbm"] = t_alt / (mean_us * 1e-6)
    if tensor_bound and kernel_mhz:
        # tensor-pipe cycles the FLOPs need (148 SMs x 8192 dense bf16 FLOP per cycle and SM: one
        # 128 x 256 x 16 tcgen05.mma per 128 cycles) over the cycles the call took at the clock measured
        # inside the kernel (the last timed launch: its own time and its own clock): the fraction with the
        # power-limited clock taken out
        props = torch.cuda.get_device_properties(torch.cuda.current_device())
        roof["tensor_cycles_ideal_over_measured"] = (wl.flops / (props.multi_processor_count * 8192.0)) / (us[-1] * kernel_mhz)
    roof["traffic"] = NCU_TRAFFIC.get(wl.name, {}).get("bytes")
    roof["traffic_source"] = NCU_TRAFFIC.get(wl.name, {}).get("summary")
    roof["peak_source"] = peaks["_source"] + (" burst" if tensor_bound else "")
    roof["roofline_us"] = max(t_tc, t_hbm) * 1e6
    roof["kernel"] = "entwine_fused_kernel<256, true, false, false, false>"

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": mean_us / 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "W": wl.W, "M": wl.M, "N": wl.N, "K_local": wl.K,
                   "n_comm_sms": launch["n_comm_sms"],
                   "tile_order": "interleaved" if launch["order"] else "row_major",
                   "plan_options": launch.get("opts", {}),
                   "block": "128x256 blocks on CTA pairs (256x256 pair tiles)",
                   "emulated_rank": launch["rank"], "l2": "flushed between timed steps (512 MiB memset)",
                   "multi_gpu": "replicas only"},
        "us_per_call": {"mean": mean_us, "median": statistics.median(us), "min": min(us),
                        "last_us": us[-1], "sm_mhz_inside_last_kernel": kernel_mhz, "last_us_times_sm_mhz": us[-1] * kernel_mhz},
        "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps, "roofline": roof,
        "device_status": {"t_gemm_us": status["t_gemm_ns"] / 1e3, "t_end_us": status["t_end_ns"] / 1e3,
                          "tail_us": (status["t_end_ns"] - status["t_gemm_ns"]) / 1e3},
        "wall_s_timed_region": wall,
    }

    # ---- comparisons and the other LLM-shaped configurations -----------------------------------
    if not args.no_extra:
        extra = {}
        names = [wl.name] + [n for n in ("attn_out_proj", "mlp_down_proj", "short_k_comm_bound") if n != wl.name]
        for name in names:
            time.sleep(1.0)  # let the part recover from the previous workload's sustained load
            w2 = I.CONFIGS[name]
            r = measure_workload(w2, LAUNCH[name], min(100, max(10, args.steps // 2)), 5, flush, torch, E, I, True)
            med = statistics.median
            fused = med(r["fused_us"])
            tc, hb = roofline_seconds(w2, peaks)
            e = {
                "fused_us": fused, "fused_tflops": w2.flops / fused / 1e6,
                "fused_hot_l2_us": med(r["fused_hot_us"]),
                "fused_back_to_back_us": r["fused_back_to_back_us"],
                "fused_graph_replay_us": r["fused_graph_replay_us"],
                "roofline_us": max(tc, hb) * 1e6, "roofline_frac": max(tc, hb) * 1e6 / fused,
                "roofline_frac_back_to_back": max(tc, hb) * 1e6 / r["fused_back_to_back_us"],
                "sm_mhz_inside_last_kernel": r["sm_mhz"], "last_fused_us_times_sm_mhz": r["fused_us"][-1] * r["sm_mhz"],
                "bound": "tensor" if tc >= hb else "hbm",
                "unfused_cublas_then_reduce_us": med(r["unfused_us"]),
                "speedup_vs_unfused": med(r["unfused_us"]) / fused,
                "cublas_gemm_us": med(r["cublas_gemm_us"]),
                "gemm_alone_us": med(r["gemm_only_us"]),
                "comm_alone_all_sms_us": med(r["comm_only_us"]),
                "comm_alone_GBps": w2.comm_bytes / med(r["comm_only_us"]) / 1e3,
                "pull_mode_us": med(r["pull_us"]),
                "overlap_efficiency": med(r["gemm_only_us"]) / fused,
                "tail_us": (r["status"]["t_end_ns"] - r["status"]["t_gemm_ns"]) / 1e3,
                "n_comm_sms": LAUNCH[name]["n_comm_sms"],
                "tile_order": "interleaved" if LAUNCH[name]["order"] else "row_major",
            }
            other = dict(LAUNCH[name], order=1 - LAUNCH[name]["order"])
            r2 = measure_workload(w2, other, min(100, max(10, args.steps // 2)), 5, flush, torch, E, I, False)
            e["other_tile_order_fused_us"] = med(r2["fused_us"])
            # Eq. 4 generalised to the emulation's push + reduce bytes, from the measured window
            t_g = r["status"]["t_gemm_ns"] * 1e-9
            if t_g > 0:
                e["b_req_GBps"] = w2.comm_bytes / t_g / 1e9
                e["b_measured_GBps"] = w2.comm_bytes / (r["status"]["t_end_ns"] * 1e-9) / 1e9
            extra[name] = e
        line["comparisons"] = extra

    # ---- CPU baseline: the oracle on the host cores --------------------------------------------
    if not args.no_cpu_baseline:
        rows = wl.M if wl.flops <= 5e10 else 512
        probe, _, _ = run_cpu_oracle(wl, launch, rows, 1)
        passes = int(max(3, min(80, 15.0 / max(probe[0], 1e-3))))  # about 15 s of CPU work
        times, flops, threads = run_cpu_oracle(wl, launch, rows, passes)
        line["cpu_baseline"] = {
            "value": flops / min(times) / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
            "sample": (f"{rows} of {wl.M} rows of the float64 partial GEMM and its magnitude sums"
                       + (" + reduce-scatter definition" if rows >= wl.M else "") +
                       f" + the full integer schedule, best of {passes} passes ({sum(times):.1f} s in total)")}
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

#!/usr/bin/env python
"""Benchmark of the split-FP4 linear layer (forward + input gradient + weight gradient).

One step = one pass of the whole hot path on one LLaMA-3-8B q_proj-shaped layer
(4096 tokens, 4096 -> 4096): split + quantize of X, W_t and dY, then Eq. 2, Eq. 3 and the weight
gradient.  Metric: effective TFLOP/s = 6*l*m*n / step time (low-rank extra flops not counted).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--weights split|requant]

N > 1 (launched by torchrun): every rank runs the same step on its own token shard (weak scaling)
and the weight gradient is summed across ranks with one NCCL all-reduce.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
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

L_TOKENS, D_IN, D_OUT, RANK_K, OVERSAMPLE_P = 4096, 4096, 4096, 32, 8
WORKLOAD = "llama3-8b q_proj linear fwd+bwd, tokens 4096 (2x2048), 4096->4096, k=32 p=8, SR on dY"
N_SETS = 3
FP4_OVER_BF16 = 4.0           # nominal dense FP4 : bf16 tensor throughput ratio
GEMM_DRAM_BYTES_NCU = 22.09e6 + 0.60e6   # per 4096^3 launch (profiles/gemm_nvfp4_2cta_4096x4096x4096.md)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.rows, self.proc = index, [], None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                self.rows.append([c.strip() for c in line.split(",")])
        except Exception:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        sm, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
def oracle_sample_step(sample_tokens, seed):
    """One pass of the oracle over a token sample of the workload.  Returns (seconds, flops credited)."""
    from oracle import layer as olay, nvfp4 as onv, split as osp
    from paper_2509_00404_b200 import synth
    x, _ = synth.llama_like(sample_tokens, D_IN, 1.0, seed)
    w, _ = synth.llama_like(D_OUT, D_IN, 0.02, seed + 1)
    d, _ = synth.llama_like(sample_tokens, D_OUT, 1e-4, seed + 2)
    t0 = time.perf_counter()
    xq = olay.quantize_operand(x, RANK_K, OVERSAMPLE_P, osp.MODE_SAMPLED, seed)
    wq = olay.quantize_operand(w, RANK_K, OVERSAMPLE_P, osp.MODE_FULL, seed + 1)
    dq = olay.quantize_operand(d, RANK_K, OVERSAMPLE_P, osp.MODE_SAMPLED, seed + 2, onv.ROUND_SR)
    y = olay.linear_fwd(xq, wq)
    dx = olay.linear_dgrad(dq, wq)
    dw = olay.linear_wgrad(dq, xq)
    dt = time.perf_counter() - t0
    assert np.isfinite(y).all() and np.isfinite(dx).all() and np.isfinite(dw).all()
    return dt, 6.0 * sample_tokens * D_IN * D_OUT


def cpu_threads():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = 256
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample_step(sample, 900)
    times, flops = [], 0.0
    for i in range(args.steps):
        dt, f = oracle_sample_step(sample, 1000 + 10 * i)
        times.append(dt)
        flops = f
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    sample_txt = "%d of %d tokens per step, full 4096x4096 weight, all operands split+quantized, 3 float64 products" % (sample, L_TOKENS)
    line = {"impl": "reference", "metric": "split_fp4_linear_fwd_bwd_effective_tflops", "value": value, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample_txt},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--weights", default="split", choices=["split", "requant"],
                    help="split: W_t is split (FULL sketch) and quantized every step; requant: W_t is split once, "
                         "its stored residual and factors are re-quantized every step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying CUDA graphs")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    from paper_2509_00404_b200 import binding as B, parallel, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    h = B.Handle(local_rank)
    sampler = ClockSampler(local_rank)

    l, m, n, k, p = L_TOKENS, D_IN, D_OUT, RANK_K, OVERSAMPLE_P
    bf = torch.bfloat16
    host_sets, dev_sets = [], []
    for s in range(N_SETS):
        c = synth.config_qproj(l, m, n, seed=2000 + 100 * s + 7 * rank)
        hs = {key: torch.from_numpy(c[key]).to(bf).pin_memory() for key in ("x", "w", "dy")}
        host_sets.append(hs)
        dev_sets.append({key: v.cuda() for key, v in hs.items()})
    xo, wo, do = B.Operand(l, m, k), B.Operand(n, m, k), B.Operand(l, n, k)
    y = torch.empty((l, n), dtype=bf, device="cuda")
    dx = torch.empty((l, m), dtype=bf, device="cuda")
    dw = torch.empty((n, m), dtype=bf, device="cuda")
    w_res_dense = None
    if args.weights == "requant":
        # weights held as (left, sigma, right, residual): split once, then only re-quantized per step
        wo0, w_res_dense = h.split(dev_sets[0]["w"], k, p, sketch=B.SKETCH_FULL, seed=2, want_residual=True)
        w_res_bf = w_res_dense.to(bf)

    # The three operand decompositions are independent of each other, and the dY chain is independent of the
    # forward product: they run on three streams and join by events (torch streams: plumbing only).
    side_w, side_d = torch.cuda.Stream(), torch.cuda.Stream()
    ev_start, ev_w, ev_d, ev_x, ev_b = (torch.cuda.Event() for _ in range(5))
    h_x, h_w, h_d = h, B.Handle(local_rank), B.Handle(local_rank)     # one workspace owner per stream

    stamps = torch.zeros(8, dtype=torch.int64, device="cuda")

    def step(bufs, i, stamp=False, outs=None):
        y_, dx_, dw_ = outs if outs is not None else (y, dx, dw)
        main = torch.cuda.current_stream()
        if stamp:
            h_x.timestamp(stamps[0:1], main)
        ev_start.record(main)
        side_w.wait_event(ev_start)
        side_d.wait_event(ev_start)
        with torch.cuda.stream(side_w):
            if args.weights == "split":
                h_w.split(bufs["w"], k, p, sketch=B.SKETCH_FULL, seed=3 * i + 2, rounding=B.ROUND_RNE, out=wo, stream=side_w)
            else:
                h_w.requantize_weight(wo0, w_res_bf, out=wo, stream=side_w)
            if stamp:
                h_w.timestamp(stamps[2:3], side_w)
            ev_w.record(side_w)
        with torch.cuda.stream(side_d):
            h_d.split(bufs["dy"], k, p, sketch=B.SKETCH_SAMPLED, seed=3 * i + 3, rounding=B.ROUND_SR, out=do, stream=side_d)
            if stamp:
                h_d.timestamp(stamps[3:4], side_d)
            ev_d.record(side_d)
        h_x.split(bufs["x"], k, p, sketch=B.SKETCH_SAMPLED, seed=3 * i + 1, rounding=B.ROUND_RNE, out=xo)
        ev_x.record(main)
        if stamp:
            h_x.timestamp(stamps[1:2], main)
        main.wait_event(ev_w)
        h_x.linear_fwd(xo, wo, out=y_)
        if stamp:
            h_x.timestamp(stamps[4:5], main)
        # The backward products need dY, X and W but not the forward product: they follow the dY decomposition on its
        # stream (in the forward's stream they would queue behind its GEMM, prologue included).
        side_d.wait_event(ev_x)
        side_d.wait_event(ev_w)
        with torch.cuda.stream(side_d):
            h_d.linear_bwd(do, xo, wo, out=(dx_, dw_), stream=side_d)
            if stamp:
                h_d.timestamp(stamps[5:6], side_d)
            parallel.allreduce_weight_grad_(dw_)     # token-sharded ranks: the one exchange of the path
            ev_b.record(side_d)
        main.wait_event(ev_b)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ------------------------------------------------------------------
    for i in range(args.warmup):
        step(dev_sets[i % N_SETS], i)
    barrier()
    assert h.device_status() == 0, "a bounded device wait expired during warm-up"
    l0 = B.launch_count()
    step(dev_sets[0], 0)
    barrier()
    launches_per_step = B.launch_count() - l0

    # One step is ~100 short kernels on three streams: replaying it as a CUDA graph (one per input set; the
    # seeds are baked in, all work is re-executed) takes the host's launch cost off the critical path.
    use_graph = world == 1 and not args.no_graph
    # end-to-end run: two staging sets (inputs and outputs), so that the copies of neighbouring steps overlap the compute
    stages = [{key: torch.empty_like(v) for key, v in dev_sets[0].items()} for _ in range(2)]
    out_sets = [(y, dx, dw), tuple(torch.empty_like(t) for t in (y, dx, dw))]
    graphs, graph_e2e = [], None
    if use_graph:
        try:
            for s_i in range(N_SETS):
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_):
                    step(dev_sets[s_i], s_i)
                graphs.append(g_)
            graph_e2e = []
            for b_ in range(2):
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_):
                    step(stages[b_], 0, outs=out_sets[b_])
                graph_e2e.append(g_)
            # the replay must reproduce the host-launched step bit for bit (all kernels are deterministic)
            step(dev_sets[0], 0)
            barrier()
            ref_out = [t.clone() for t in (y, dx, dw)]
            graphs[0].replay()
            barrier()
            assert all(torch.equal(a_, b_) for a_, b_ in zip(ref_out, (y, dx, dw))), "graph replay differs from host launches"
            del ref_out
        except AssertionError:
            raise
        except Exception as exc:                     # fall back to host launches, say so in the output
            sys.stderr.write("CUDA graph capture failed (%s); using host launches\n" % exc)
            use_graph, graphs, graph_e2e = False, [], None
            torch.cuda.synchronize()

    def run_step(i):
        if use_graph:
            graphs[i % N_SETS].replay()
        else:
            step(dev_sets[i % N_SETS], i)

    sampler.start()
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        run_step(i)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1) / args.steps
    launches = launches_per_step * args.steps
    status = h.device_status() | h_w.device_status() | h_d.device_status()

    # ---- end to end: pinned host inputs in, results out, every step ---------------------------------
    y_h, dx_h, dw_h = (torch.empty((l, n), dtype=bf).pin_memory(), torch.empty((l, m), dtype=bf).pin_memory(),
                       torch.empty((n, m), dtype=bf).pin_memory())

    # Step i uses staging set i % 2: its inputs go up on one copy stream while step i - 1 computes, its results come
    # down on another while step i + 1 computes (PCIe is full duplex).  Every step still copies all of its inputs
    # from pinned host memory and all of its results back.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in, ev_comp, ev_out = ([torch.cuda.Event() for _ in range(2)] for _ in range(3))

    def e2e_step(i):
        b_ = i & 1
        hs = host_sets[i % N_SETS]
        comp = torch.cuda.current_stream()
        s_in.wait_event(ev_comp[b_])                   # the compute of step i - 2 has read this staging set
        with torch.cuda.stream(s_in):
            for key in ("x", "w", "dy"):
                stages[b_][key].copy_(hs[key], non_blocking=True)
            ev_in[b_].record(s_in)
        comp.wait_event(ev_in[b_])
        comp.wait_event(ev_out[b_])                    # the results of step i - 2 have left this output set
        if use_graph:
            graph_e2e[b_].replay()
        else:
            step(stages[b_], i, outs=out_sets[b_])
        ev_comp[b_].record(comp)
        s_out.wait_event(ev_comp[b_])
        with torch.cuda.stream(s_out):
            for host_t, dev_t in zip((y_h, dx_h, dw_h), out_sets[b_]):
                host_t.copy_(dev_t, non_blocking=True)
            ev_out[b_].record(s_out)

    for i in range(4):
        e2e_step(i)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_e2e = max(4, args.steps)
    e2.record()
    for i in range(n_e2e):
        e2e_step(i)
    for b_ in range(2):
        torch.cuda.current_stream().wait_event(ev_out[b_])
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3) / n_e2e

    # ---- dominant kernel alone: the FP4 tensor-core GEMM on the three residual pairs ---------------------
    pairs = [(xo.res_by_cols, wo.res_by_cols), (do.res_by_cols, wo.res_by_rows), (do.res_by_rows, xo.res_by_rows)]
    outs = [y, dx, dw]
    for a, b_ in pairs:
        h.gemm_nvfp4(a, b_, out=y)
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 10
    g0.record()
    for r in range(reps):
        for (a, b_), o in zip(pairs, outs):
            h.gemm_nvfp4(a, b_, out=o)
    g1.record()
    torch.cuda.synchronize()
    gemm_ms = g0.elapsed_time(g1) / (3 * reps)
    # plain (k = 0) layer time for the overhead figure: three GEMMs only
    overhead = ms / (3 * gemm_ms) - 1.0

    # ---- split + quantize of each operand alone (algorithmic bytes: 2 B read + 2 x 0.5625 B written per element) ----
    def alone(fn, reps=10):
        """Mean device time of fn over `reps` calls; the calls are replayed as one CUDA graph where that is possible,
        so that a single short kernel is not timed by the host's launch rate."""
        fn(0)
        torch.cuda.synchronize()
        graph = None
        if use_graph:
            try:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for r_ in range(reps):
                        fn(r_)
                graph.replay()
                torch.cuda.synchronize()
            except Exception:
                graph = None
                torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        if graph is not None:
            graph.replay()
        else:
            for r_ in range(reps):
                fn(r_)
        a1.record()
        torch.cuda.synchronize()
        return a0.elapsed_time(a1) / reps
    ms_sx = alone(lambda i: h_x.split(dev_sets[i % N_SETS]["x"], k, p, sketch=B.SKETCH_SAMPLED, seed=i + 1, out=xo))
    ms_sw = alone(lambda i: h_x.split(dev_sets[i % N_SETS]["w"], k, p, sketch=B.SKETCH_FULL, seed=i + 2, out=wo))
    ms_sd = alone(lambda i: h_x.split(dev_sets[i % N_SETS]["dy"], k, p, sketch=B.SKETCH_SAMPLED, seed=i + 3, rounding=B.ROUND_SR, out=do))
    qc, qr = B.NvFp4(l, m), B.NvFp4(m, l)
    ms_q = alone(lambda i: h_x.quantize_nvfp4(dev_sets[i % N_SETS]["x"], B.BLOCKS_BOTH, B.ROUND_RNE, seed=1, tensor_scale=1.0, out=(qc, qr)))
    split_gbs = lambda elems, t_ms: 3.125 * elems / (t_ms * 1e-3) / 1e9

    # ---- where the step's time goes: GPU timer stamps at the end of each phase (their own graph, not the timed one) ----
    timeline = None
    try:
        if use_graph:
            g_t = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_t):
                step(dev_sets[0], 0, stamp=True)
            run_t = g_t.replay
        else:
            run_t = lambda: step(dev_sets[0], 0, stamp=True)
        acc_t = [0.0] * 6
        for _ in range(2):
            run_t()
        torch.cuda.synchronize()
        for _ in range(10):
            run_t()
            torch.cuda.synchronize()
            t_ = stamps.cpu().tolist()
            for j_ in range(6):
                acc_t[j_] += (t_[j_] - t_[0]) / 1e6 / 10
        timeline = {"unit": "ms after the step's start (one input set, ten replays)", "x_split_done": acc_t[1], "w_split_done": acc_t[2],
                    "dy_split_done": acc_t[3], "forward_done": acc_t[4], "backward_done": acc_t[5]}
    except Exception as exc:
        sys.stderr.write("timeline not measured (%s)\n" % exc)
    clocks = sampler.stop()

    times = torch.tensor([ms, ms_e2e], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms, ms_e2e = float(times[0]), float(times[1])

    flops_step = 6.0 * l * m * n
    peaks = measured_peaks()
    fp4_peak = peaks["bf16_tflops"] * FP4_OVER_BF16
    gemm_tflops = 2.0 * l * m * n / (gemm_ms * 1e-3) / 1e12
    line = {
        "metric": "split_fp4_linear_fwd_bwd_effective_tflops",
        "value": world * flops_step / (ms * 1e-3) / 1e12,
        "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4 (e2m1 x ue4m3, fp32 accumulate)",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "weights": args.weights, "cuda_graph": bool(use_graph),
                   "l2": "inputs rotate over %d sets (%d MB > 126 MB L2)" % (N_SETS, N_SETS * 3 * l * m * 2 // 2 ** 20),
                   "parallelism": "dp%d (token-sharded, dW all-reduce)" % world if world > 1 else "single GPU"},
        "e2e": {"value": world * flops_step / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": 3 * l * m * 2, "d2h_bytes_per_step": 3 * l * m * 2, "ms_per_step": ms_e2e,
                "overlap": "two staging sets: the copies of step i+1 / i-1 run on their own streams beside the compute of step i"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "two_cta::gemm_nvfp4_2cta_kernel (4096x4096x4096 residual GEMM, bf16 out)",
                     "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s", "frac": gemm_tflops / fp4_peak,
                     "traffic": GEMM_DRAM_BYTES_NCU, "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch, see profiles/",
                     "algorithmic_bytes": 0.5625 * 2 * l * m + 2.0 * l * n, "peak_source": "bf16 burst peak (%s) x %.0f nominal FP4:bf16 ratio" % (peaks["source"], FP4_OVER_BF16),
                     "ms_per_launch": gemm_ms},
        "split_overhead_vs_three_plain_gemms": overhead,
        "timeline": timeline,
        "split_quantize": {"unit": "GB/s of algorithmic bytes (3.125 B per element, both block orientations)",
                           "hbm_peak_gbs": peaks["hbm_gbs"],
                           "x_sampled": {"ms": ms_sx, "gbs": split_gbs(l * m, ms_sx)},
                           "w_full": {"ms": ms_sw, "gbs": split_gbs(n * m, ms_sw)},
                           "dy_sampled_sr": {"ms": ms_sd, "gbs": split_gbs(l * n, ms_sd)},
                           "plain_quantizer_rne_given_scale": {"ms": ms_q, "gbs": split_gbs(l * m, ms_q), "frac_of_hbm": split_gbs(l * m, ms_q) / peaks["hbm_gbs"]}},
        "device_status": status,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = 1024
        dt, f = oracle_sample_step(sample, 4242)
        line["cpu_baseline"] = {"value": f / dt / 1e12, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle",
                                "sample": "%d of %d tokens, full 4096x4096 weight, one pass (%.1f s)" % (sample, l, dt)}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the split-FP4 linear layer (forward + input gradient + weight gradient) at LLaMA-3 shapes.

One step = one pass of the whole hot path over the layers of a workload: split + quantize of every
activation X (once per group of projections that share it), of every weight W_t and of every output
gradient dY, then Eq. 2, Eq. 3 and the weight gradient of every layer.  Metric: effective TFLOP/s
= sum over layers of 6*l*m*n / step time (low-rank extra flops not counted).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--weights split|requant]
                  [--workloads name,name,...]

Workloads (all timed in one run, one sub-record each; the headline is the decoder block):
  qproj_4096tok        one q_proj-shaped layer, 4096 tokens, 4096 -> 4096, k = 32
  ffn_8192tok          SwiGLU FFN layers at 8192 tokens: gate, up 4096 -> 14336 (shared X), down 14336 -> 4096
  block_16384tok       all seven linear layers of a decoder block at 16384 tokens (q, k, v share X; gate, up share X)
  proj70b_16384tok_k*  rank sweep k = 0, 16, 64, 256 on an 8192 -> 28672 projection at 16384 tokens

N > 1: every rank runs the same steps on its own token shard (weak scaling) and the weight gradients are
summed across ranks with NCCL all-reduces that overlap the next step.  Started without a torchrun
environment, `--gpus N` starts its own N ranks on this node.
`--impl reference` times the CPU oracle on a bounded sample of the headline workload.
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FP4_OVER_BF16 = 4.0           # nominal dense FP4 : bf16 tensor throughput ratio
BYTES_PER_ELEM_BOTH = 3.125   # split / quantize: 2 B read + 2 x 0.5625 B written per operand element


# DRAM bytes of ONE launch of the two-CTA GEMM (dram__bytes_read.sum + dram__bytes_write.sum), per (M, N, K), from an
# ncu capture of this program's block workload (a profiler cannot run inside the timed program).  Reads are 4.3 x the
# operand bytes at K = 4096 (the B panels are fetched once per group of eight tile rows); the bf16 output is written once.
NCU_DRAM_BYTES = {(16384, 14336, 4096): 304.8e6 + 416.3e6, (16384, 4096, 14336): 321.3e6 + 113.2e6,
                  (14336, 4096, 16384): 374.7e6 + 98.3e6}
NCU_DRAM_SOURCE = ("ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum -k regex:gemm_nvfp4_2cta on "
                   "`bench.py --workloads block_16384tok --no-graph`, one launch of this shape")


def layer(name, d_in, d_out, x_group):
    return {"name": name, "d_in": d_in, "d_out": d_out, "x": x_group}


WORKLOADS = {
    "qproj_4096tok": {"tokens": 4096, "k": 32, "p": 8, "rank": 32, "layers": [layer("q", 4096, 4096, "x")],
                      "text": "llama3-8b q_proj linear fwd+bwd, tokens 4096 (2x2048), 4096->4096, k=32 p=8, SR on dY"},
    "ffn_8192tok": {"tokens": 8192, "k": 32, "p": 8, "rank": 32,
                    "layers": [layer("gate", 4096, 14336, "x_ffn"), layer("up", 4096, 14336, "x_ffn"), layer("down", 14336, 4096, "x_down")],
                    "text": "llama3-8b SwiGLU FFN linears fwd+bwd, tokens 8192: gate, up 4096->14336 (X shared, split once), down 14336->4096, k=32 p=8, SR on dY"},
    "block_16384tok": {"tokens": 16384, "k": 32, "p": 8, "rank": 32,
                       "layers": [layer("q", 4096, 4096, "x_attn"), layer("k", 4096, 1024, "x_attn"), layer("v", 4096, 1024, "x_attn"),
                                  layer("o", 4096, 4096, "x_o"), layer("gate", 4096, 14336, "x_ffn"), layer("up", 4096, 14336, "x_ffn"),
                                  layer("down", 14336, 4096, "x_down")],
                       "text": "llama3-8b decoder block, all seven linears fwd+bwd, tokens 16384 (8x2048): q,o 4096->4096; k,v 4096->1024; "
                               "gate,up 4096->14336; down 14336->4096; X shared by q/k/v and by gate/up split once; k=32 p=8, SR on dY"},
}
for _k in (0, 16, 64, 256):
    WORKLOADS["proj70b_16384tok_k%d" % _k] = {
        "tokens": 16384, "k": _k, "p": 8 if _k else 0, "rank": 64, "layers": [layer("proj", 8192, 28672, "x")],
        "text": "llama3-70b-shaped projection fwd+bwd, tokens 16384, 8192->28672, planted rank 64, k=%d p=%d, SR on dY" % (_k, 8 if _k else 0)}
HEADLINE = "block_16384tok"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through nvidia-smi while timed regions run."""

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
                self.rows.append((time.time(), [c.strip() for c in line.split(",")]))
        except Exception:
            pass

    def summary(self, t0=None, t1=None):
        sm, power, reasons, mx = [], [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in list(self.rows):
            if (t0 is not None and t < t0) or (t1 is not None and t > t1):
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                power.append(float(r[2]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "power_w_max": max(power) if power else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)


# ------------------------------------------------------------------------------------------------
def oracle_sample_step(sample_tokens, seed, d_in=4096, d_out=4096, k=32, p=8):
    """One pass of the oracle over a token sample of one q_proj-shaped layer.  Returns (seconds, flops credited, seconds per phase)."""
    from oracle import layer as olay, nvfp4 as onv, split as osp
    from paper_2509_00404_b200 import synth
    x, _ = synth.llama_like(sample_tokens, d_in, 1.0, seed)
    w, _ = synth.llama_like(d_out, d_in, 0.02, seed + 1)
    d, _ = synth.llama_like(sample_tokens, d_out, 1e-4, seed + 2)
    t0 = time.perf_counter()
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, seed)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, seed + 1)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, seed + 2, onv.ROUND_SR)
    t1 = time.perf_counter()
    y = olay.linear_fwd(xq, wq)
    dx = olay.linear_dgrad(dq, wq)
    dw = olay.linear_wgrad(dq, xq)
    dt = time.perf_counter() - t0
    assert np.isfinite(y).all() and np.isfinite(dx).all() and np.isfinite(dw).all()
    return dt, 6.0 * sample_tokens * d_in * d_out, {"split_and_quantize_s": t1 - t0, "three_products_s": dt - (t1 - t0)}


def cpu_threads():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample = 256
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample_step(sample, 900)
    times, flops = [], 0.0
    for i in range(args.steps):
        dt, f, _ = oracle_sample_step(sample, 1000 + 10 * i)
        times.append(dt)
        flops = f
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    sample_txt = ("the q projection of the block (4096->4096) on %d of 16384 tokens per step: all three operands split+quantized, "
                  "3 float64 products" % sample)
    line = {"impl": "reference", "metric": "split_fp4_linear_fwd_bwd_effective_tflops", "value": value, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOADS[HEADLINE]["text"], "sample": sample_txt},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
def spawn_ranks(n):
    """`python bench.py --gpus N` without a torchrun environment: start the N ranks of this node ourselves."""
    import torch
    have = torch.cuda.device_count()
    if have < n:
        sys.stderr.write("bench.py: --gpus %d asked for, %d CUDA device(s) visible: refusing to report a %d-GPU number\n" % (n, have, n))
        sys.exit(2)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--local-addr", "127.0.0.1", "--nnodes=1",
           "--nproc-per-node", str(n), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


class Workload:
    """Device buffers and the enqueue order of one workload on one rank."""

    def __init__(self, name, spec, B, synth, handles, streams, weights_mode, world, rank, dw_sets=1, act_sketch=None):
        import torch
        self.torch, self.B, self.name, self.spec = torch, B, name, spec
        self.act_sketch = B.SKETCH_SAMPLED if act_sketch is None else act_sketch      # sketch mode of the activation and gradient operands
        self.amax = None                                     # optional: amax|operand| as its producer would hand it over
        # handles / streams: one for the activations and the forward products (the caller's current stream), N_SIDE
        # for the weights and N_SIDE for the output gradients and the backward products (layer j uses side j % N_SIDE,
        # so that the latency-bound start of one layer's decomposition runs beside the previous layer's big kernels)
        self.h_x, self.h_ws, self.h_ds = handles
        self.side_ws, self.side_ds = streams
        self.h_w, self.h_d = self.h_ws[0], self.h_ds[0]
        self.l, self.k, self.p = spec["tokens"], spec["k"], spec["p"]
        self.layers = spec["layers"]
        self.weights_mode = weights_mode
        bf = torch.bfloat16
        l, k, rk = self.l, self.k, spec["rank"]
        seed0 = 7000 + 977 * rank
        self.x_in, self.xo = {}, {}
        for i, ly in enumerate(self.layers):
            g = ly["x"]
            if g not in self.x_in:
                self.x_in[g] = synth.planted_device(l, ly["d_in"], rk, 1.0, seed0 + 31 * i)
                self.xo[g] = B.Operand(l, ly["d_in"], k)
        self.w_in = [synth.planted_device(ly["d_out"], ly["d_in"], rk, 0.02, seed0 + 31 * i + 1) for i, ly in enumerate(self.layers)]
        self.d_in = [synth.planted_device(l, ly["d_out"], rk, 1e-4, seed0 + 31 * i + 2) for i, ly in enumerate(self.layers)]
        self.wo = [B.Operand(ly["d_out"], ly["d_in"], k) for ly in self.layers]
        self.do = [B.Operand(l, ly["d_out"], k) for ly in self.layers]
        self.y = [torch.empty((l, ly["d_out"]), dtype=bf, device="cuda") for ly in self.layers]
        self.dx = [torch.empty((l, ly["d_in"]), dtype=bf, device="cuda") for ly in self.layers]
        # several ranks: FP32 weight gradients (summed across ranks in FP32), two sets so that the all-reduce of one
        # step overlaps the next step
        dw_dt = torch.float32 if world > 1 else bf
        self.dw_sets = [[torch.empty((ly["d_out"], ly["d_in"]), dtype=dw_dt, device="cuda") for ly in self.layers] for _ in range(dw_sets)]
        self.w_stored = None
        if weights_mode == "requant" and k:
            # weights held as (left, sigma, right, residual): split once, re-quantized every step
            self.w_stored = []
            for i, ly in enumerate(self.layers):
                _, dense = self.h_w.split(self.w_in[i], k, self.p, sketch=B.SKETCH_FULL, seed=2, out=self.wo[i], want_residual=True)
                self.w_stored.append(dense)
        n_x = len(self.x_in)
        self.ev_start = torch.cuda.Event()
        self.ev_x = {g: torch.cuda.Event() for g in self.x_in}
        self.ev_w = [torch.cuda.Event() for _ in self.layers]
        self.ev_b = [torch.cuda.Event() for _ in self.side_ds]
        self.flops = sum(6.0 * l * ly["d_in"] * ly["d_out"] for ly in self.layers)
        self.elements = {"x": sum(l * t.shape[1] for t in self.x_in.values()), "w": sum(t.numel() for t in self.w_in),
                         "dy": sum(t.numel() for t in self.d_in)}
        self.input_bytes = 2 * sum(self.elements.values())
        self.output_bytes = sum(t.numel() * t.element_size() for t in self.y + self.dx + self.dw_sets[0])
        del n_x

    def with_producer_amax(self):
        """amax|x| of every operand, found once outside any timed region: what the kernel that wrote the operand would
        pass along (the split then runs no reduction of its own when k = 0)."""
        am = lambda t: t.float().abs().max().reshape(1)
        self.amax = ({g: am(t) for g, t in self.x_in.items()}, [am(t) for t in self.w_in], [am(t) for t in self.d_in])
        return self

    def step(self, i, inputs=None, outs=None, dw_set=0):
        """Enqueues one step on the current stream and the two side streams (joined before it returns)."""
        torch, B = self.torch, self.B
        k, p = self.k, self.p
        x_in, w_in, d_in = inputs if inputs is not None else (self.x_in, self.w_in, self.d_in)
        y, dx, dw = outs if outs is not None else (self.y, self.dx, self.dw_sets[dw_set])
        main = torch.cuda.current_stream()
        self.ev_start.record(main)
        n_w, n_d = len(self.side_ws), len(self.side_ds)
        for st in self.side_ws + self.side_ds:
            st.wait_event(self.ev_start)
        for j in range(len(self.layers)):
            sw, hw = self.side_ws[j % n_w], self.h_ws[j % n_w]
            with torch.cuda.stream(sw):
                if self.w_stored is not None:
                    hw.requantize_operand(self.wo[j], self.w_stored[j], seed=3 * i + 2, stream=sw)
                else:
                    hw.split(w_in[j], k, p, sketch=B.SKETCH_FULL, seed=3 * i + 2, rounding=B.ROUND_RNE, out=self.wo[j], stream=sw,
                             src_amax=self.amax[1][j] if self.amax else None)
                self.ev_w[j].record(sw)
        done_x = set()
        for j, ly in enumerate(self.layers):
            g = ly["x"]
            if g not in done_x:
                self.h_x.split(x_in[g], k, p, sketch=self.act_sketch, seed=3 * i + 1, rounding=B.ROUND_RNE, out=self.xo[g],
                                 src_amax=self.amax[0][g] if self.amax else None)
                self.ev_x[g].record(main)
                done_x.add(g)
            main.wait_event(self.ev_w[j])
            self.h_x.linear_fwd(self.xo[g], self.wo[j], out=y[j])
            # the backward products need dY, X and W but not the forward product: they follow the dY decomposition on
            # its stream
            sd, hd = self.side_ds[j % n_d], self.h_ds[j % n_d]
            with torch.cuda.stream(sd):
                hd.split(d_in[j], k, p, sketch=self.act_sketch, seed=3 * i + 3, rounding=B.ROUND_SR, out=self.do[j], stream=sd,
                         src_amax=self.amax[2][j] if self.amax else None)
                sd.wait_event(self.ev_x[g])
                sd.wait_event(self.ev_w[j])
                hd.linear_bwd(self.do[j], self.xo[g], self.wo[j], out=(dx[j], dw[j]), stream=sd)
        for ev, sd in zip(self.ev_b, self.side_ds):
            ev.record(sd)
            main.wait_event(ev)

    def gemm_pairs(self):
        out = []
        for j, ly in enumerate(self.layers):
            xo, wo, do = self.xo[ly["x"]], self.wo[j], self.do[j]
            out += [(xo.res_by_cols, wo.res_by_cols, self.y[j]), (do.res_by_cols, wo.res_by_rows, self.dx[j]),
                    (do.res_by_rows, xo.res_by_rows, self.dw_sets[0][j])]
        return out


def timed_ms(torch, fn, reps):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(reps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--weights", default="split", choices=["split", "requant"],
                    help="split: every W_t is split (FULL sketch) and quantized every step; requant: W_t is split once, "
                         "its stored residual and factors are re-quantized every step (the paper's per-step work for weights)")
    ap.add_argument("--workloads", default="all", help="comma-separated workload names (default: all)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp4-probe", action="store_true", help="skip the 16384^3 product that measures the GEMM kernel's own best rate")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying CUDA graphs")
    ap.add_argument("--side-streams", type=int, default=4, help="streams (and library handles) per operand kind for the weight and gradient decompositions")
    ap.add_argument("--sustain-seconds", type=float, default=1.0, help="length of the sustained timing loop of every workload")
    ap.add_argument("--dry-run-ranks-on-one-gpu", action="store_true",
                    help="control-flow check of the multi-rank path on a one-GPU box: every rank uses device 0 and the weight "
                         "gradients are summed over gloo (host-staged, so no kernel of one rank waits for another); "
                         "the line is marked and its numbers mean nothing")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    from paper_2509_00404_b200 import binding as B, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        sys.stderr.write("bench.py: --gpus %d does not match WORLD_SIZE %d\n" % (args.gpus, world))
        sys.exit(2)
    if args.dry_run_ranks_on_one_gpu:
        local_rank = 0
    torch.cuda.set_device(local_rank)
    if world > 1:
        if args.dry_run_ranks_on_one_gpu:
            dist.init_process_group("gloo")
        else:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    n_side = max(1, args.side_streams)
    handles = (B.Handle(local_rank), [B.Handle(local_rank) for _ in range(n_side)], [B.Handle(local_rank) for _ in range(n_side)])   # one workspace owner per stream
    streams = ([torch.cuda.Stream() for _ in range(n_side)], [torch.cuda.Stream() for _ in range(n_side)])
    all_handles = [handles[0]] + handles[1] + handles[2]
    comm_stream = torch.cuda.Stream()
    sampler = ClockSampler(local_rank)
    sampler.start()
    peaks = measured_peaks()
    fp4_peak = peaks["bf16_tflops"] * FP4_OVER_BF16
    names = list(WORKLOADS) if args.workloads == "all" else [n for n in args.workloads.split(",") if n]
    for n in names:
        if n not in WORKLOADS:
            sys.stderr.write("unknown workload %s; known: %s\n" % (n, ", ".join(WORKLOADS)))
            sys.exit(2)
    if HEADLINE not in names:
        names.append(HEADLINE)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(values):
        t = torch.tensor(values, dtype=torch.float64, device="cuda")
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return [float(v) for v in t]

    records, headline = {}, None
    for name in names:
        spec = WORKLOADS[name]
        wl = Workload(name, spec, B, synth, handles, streams, args.weights, world, rank, dw_sets=2 if world > 1 else 1)
        is_head = name == HEADLINE
        for i in range(args.warmup):
            wl.step(i)
        barrier()
        status = 0
        for h in all_handles:
            status |= h.device_status()
        assert status == 0, "device status %d after warm-up of %s" % (status, name)
        l0 = B.launch_count()
        wl.step(0)
        barrier()
        launches_per_step = B.launch_count() - l0

        # The step is hundreds of short kernels on three streams: replaying it as a CUDA graph takes the host's launch
        # cost off the critical path (the seeds are baked in, all work is re-executed).  Inputs exceed the L2 by
        # themselves at every workload but the smallest, which rotates over three input sets.
        n_sets = 3 if wl.input_bytes < 2 * 126e6 else 1
        in_sets = [(wl.x_in, wl.w_in, wl.d_in)]
        for s_i in range(1, n_sets):
            in_sets.append(({g: synth.planted_device(wl.l, t.shape[1], spec["rank"], 1.0, 9000 + 100 * s_i + 7 * rank) for g, t in wl.x_in.items()},
                            [synth.planted_device(t.shape[0], t.shape[1], spec["rank"], 0.02, 9001 + 100 * s_i + 7 * rank) for t in wl.w_in],
                            [synth.planted_device(t.shape[0], t.shape[1], spec["rank"], 1e-4, 9002 + 100 * s_i + 7 * rank) for t in wl.d_in]))
        n_dw = len(wl.dw_sets)
        use_graph = not args.no_graph
        graphs = {}
        if use_graph:
            try:
                for s_i in range(n_sets):
                    for b_ in range(n_dw):
                        g_ = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(g_):
                            wl.step(s_i, inputs=in_sets[s_i], dw_set=b_)
                        graphs[(s_i, b_)] = g_
                # the replay must reproduce the host-launched step bit for bit (all kernels are deterministic)
                wl.step(0, inputs=in_sets[0], dw_set=0)
                barrier()
                ref_out = [t.clone() for t in (wl.y[0], wl.dx[0], wl.dw_sets[0][0])]
                graphs[(0, 0)].replay()
                barrier()
                assert all(torch.equal(a_, b_) for a_, b_ in zip(ref_out, (wl.y[0], wl.dx[0], wl.dw_sets[0][0]))), "graph replay differs from host launches (%s)" % name
                del ref_out
            except AssertionError:
                raise
            except Exception as exc:
                sys.stderr.write("CUDA graph capture failed for %s (%s); using host launches\n" % (name, exc))
                use_graph, graphs = False, {}
                torch.cuda.synchronize()

        comm_done = [torch.cuda.Event() for _ in range(n_dw)]
        comp_done = [torch.cuda.Event() for _ in range(n_dw)]

        def run_step(i):
            b_ = i % n_dw
            main = torch.cuda.current_stream()
            if world > 1:
                main.wait_event(comm_done[b_])            # the all-reduce that last used this weight-gradient set is over
            if use_graph:
                graphs[(i % n_sets, b_)].replay()
            else:
                wl.step(i, inputs=in_sets[i % n_sets], dw_set=b_)
            if world > 1:
                # the one exchange of the path: sum of the weight gradients over the token shards, on its own stream so
                # that it overlaps the next step's decompositions and products
                comp_done[b_].record(main)
                comm_stream.wait_event(comp_done[b_])
                with torch.cuda.stream(comm_stream):
                    for t in wl.dw_sets[b_]:
                        dist.all_reduce(t, op=dist.ReduceOp.SUM)
                    comm_done[b_].record(comm_stream)

        def drain():
            if world > 1:
                for ev in comm_done:
                    torch.cuda.current_stream().wait_event(ev)

        # ---- timed region: exactly K steps, device-resident inputs --------------------------------------
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_wall0 = time.time()
        e0.record()
        for i in range(args.steps):
            run_step(i)
        drain()
        e1.record()
        barrier()
        t_wall1 = time.time()
        ms = e0.elapsed_time(e1) / args.steps
        clocks_timed = sampler.summary(t_wall0, t_wall1)

        # ---- sustained: the same loop for about a second (clocks settle under the power cap) ----------------
        n_sus = max(args.steps, int(math.ceil(args.sustain_seconds * 1e3 / ms)))
        barrier()
        t_s0 = time.time()
        e0.record()
        for i in range(n_sus):
            run_step(i)
        drain()
        e1.record()
        barrier()
        t_s1 = time.time()
        ms_sus = e0.elapsed_time(e1) / n_sus
        clocks_sus = sampler.summary(t_s0, t_s1)
        for h in all_handles:
            status |= h.device_status()
        ms, ms_sus = max_over_ranks([ms, ms_sus])

        # ---- the FP4 GEMMs of the same layers alone (k = 0 work: the denominator of the split overhead) -------
        pairs = wl.gemm_pairs()
        h_x = handles[0]

        def gemms(i):
            for a_, b_, o_ in pairs:
                h_x.gemm_nvfp4(a_, b_, out=o_)
        gemms(0)
        ms_gemm = timed_ms(torch, gemms, 5)
        # the largest single GEMM of the workload, alone: the roofline record of the tensor-core kernel
        big = max(pairs, key=lambda t: t[0].rows * t[1].rows * t[0].k_len)
        h_x.gemm_nvfp4(big[0], big[1], out=big[2])
        ms_big = timed_ms(torch, lambda i: h_x.gemm_nvfp4(big[0], big[1], out=big[2]), 10)
        big_flops = 2.0 * big[0].rows * big[1].rows * big[0].k_len
        big_bytes = 0.5625 * (big[0].rows + big[1].rows) * big[0].k_len + big[2].element_size() * big[0].rows * big[1].rows

        # ---- split + quantize of each operand kind alone, at the workload's largest operand --------------------
        def alone(fn, reps=12):
            for w_i in range(3):
                fn(w_i)
            torch.cuda.synchronize()
            return timed_ms(torch, fn, reps)
        k, p = wl.k, wl.p
        gx = max(wl.x_in, key=lambda g: wl.x_in[g].numel())
        jw = max(range(len(wl.layers)), key=lambda j: wl.w_in[j].numel())
        jd = max(range(len(wl.layers)), key=lambda j: wl.d_in[j].numel())
        ms_sx = alone(lambda i: h_x.split(wl.x_in[gx], k, p, sketch=B.SKETCH_SAMPLED, seed=i + 1, out=wl.xo[gx]))
        ms_sw = alone(lambda i: h_x.split(wl.w_in[jw], k, p, sketch=B.SKETCH_FULL, seed=i + 2, out=wl.wo[jw]))
        ms_sd = alone(lambda i: h_x.split(wl.d_in[jd], k, p, sketch=B.SKETCH_SAMPLED, seed=i + 3, rounding=B.ROUND_SR, out=wl.do[jd]))
        xq = wl.xo[gx]
        ms_q = alone(lambda i: h_x.quantize_nvfp4(wl.x_in[gx], B.BLOCKS_BOTH, B.ROUND_RNE, seed=1, tensor_scale=1.0, out=(xq.res_by_cols, xq.res_by_rows)), reps=30)
        ms_qsr = alone(lambda i: h_x.quantize_nvfp4(wl.x_in[gx], B.BLOCKS_BOTH, B.ROUND_SR, seed=1, tensor_scale=1.0, out=(xq.res_by_cols, xq.res_by_rows)), reps=30)
        gbs = lambda elems, t_ms: BYTES_PER_ELEM_BOTH * elems / (t_ms * 1e-3) / 1e9
        ex, ew, ed = wl.x_in[gx].numel(), wl.w_in[jw].numel(), wl.d_in[jd].numel()
        hbm = peaks["hbm_gbs"]
        rec = {
            "workload": spec["text"], "ms_per_step": ms, "effective_tflops": world * wl.flops / (ms * 1e-3) / 1e12,
            "sustained": {"steps": n_sus, "ms_per_step": ms_sus, "effective_tflops": world * wl.flops / (ms_sus * 1e-3) / 1e12,
                          "clocks": clocks_sus, "ms_x_median_mhz": (ms_sus * clocks_sus["sm_mhz"]) if clocks_sus["sm_mhz"] else None},
            "clocks": clocks_timed, "launches_per_step": int(launches_per_step), "cuda_graph": bool(use_graph),
            "input_sets": n_sets, "side_streams_per_kind": n_side, "input_bytes_per_step": int(wl.input_bytes),
            "plain_fp4_gemms": {"ms": ms_gemm, "tflops": wl.flops / (ms_gemm * 1e-3) / 1e12, "frac_of_fp4_peak": wl.flops / (ms_gemm * 1e-3) / 1e12 / fp4_peak},
            "split_overhead_vs_plain_gemms": ms / ms_gemm - 1.0,
            "largest_gemm": {"shape_mnk": [int(big[0].rows), int(big[1].rows), int(big[0].k_len)], "ms": ms_big,
                             "tflops": big_flops / (ms_big * 1e-3) / 1e12, "frac_of_fp4_peak": big_flops / (ms_big * 1e-3) / 1e12 / fp4_peak,
                             "algorithmic_bytes": big_bytes},
            "split_quantize": {"unit": "GB/s of algorithmic bytes (3.125 B per element, both block orientations); largest operand of each kind, alone",
                               "x_sampled": {"shape": list(wl.x_in[gx].shape), "ms": ms_sx, "gbs": gbs(ex, ms_sx), "frac_of_hbm": gbs(ex, ms_sx) / hbm},
                               "w_full": {"shape": list(wl.w_in[jw].shape), "ms": ms_sw, "gbs": gbs(ew, ms_sw), "frac_of_hbm": gbs(ew, ms_sw) / hbm},
                               "dy_sampled_sr": {"shape": list(wl.d_in[jd].shape), "ms": ms_sd, "gbs": gbs(ed, ms_sd), "frac_of_hbm": gbs(ed, ms_sd) / hbm},
                               "plain_quantizer_rne": {"shape": list(wl.x_in[gx].shape), "ms": ms_q, "gbs": gbs(ex, ms_q), "frac_of_hbm": gbs(ex, ms_q) / hbm},
                               "plain_quantizer_sr": {"shape": list(wl.x_in[gx].shape), "ms": ms_qsr, "gbs": gbs(ex, ms_qsr), "frac_of_hbm": gbs(ex, ms_qsr) / hbm}},
            "device_status": int(status),
        }
        records[name] = rec

        if wl.k == 0:
            # plain quantization with amax|x| supplied by the producer of each operand: no reduction pass inside the step
            wa = Workload(name, spec, B, synth, handles, streams, args.weights, world, rank, dw_sets=1).with_producer_amax()
            for i in range(args.warmup):
                wa.step(i)
            barrier()
            ms_a = max_over_ranks([timed_ms(torch, wa.step, args.steps)])[0]
            rec["amax_supplied_by_the_producer"] = {"ms_per_step": ms_a, "effective_tflops": world * wa.flops / (ms_a * 1e-3) / 1e12,
                                                    "split_overhead_vs_plain_gemms": ms_a / ms_gemm - 1.0, "cuda_graph": False}
            del wa
            torch.cuda.empty_cache()

        if is_head and args.weights == "split" and wl.k:
            # The same block with the weights held as stored factors + residual and only re-quantized each step (the
            # paper's per-step work for weights, Section 3.2), activations and gradients split as before.
            wr = Workload(name, spec, B, synth, handles, streams, "requant", world, rank, dw_sets=1)
            for i in range(args.warmup):
                wr.step(i)
            barrier()
            g_r = None
            if use_graph:
                try:
                    g_r = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g_r):
                        wr.step(0)
                except Exception:
                    g_r = None
                    torch.cuda.synchronize()
            ms_r = timed_ms(torch, (lambda i: g_r.replay()) if g_r is not None else wr.step, args.steps)
            ms_r = max_over_ranks([ms_r])[0]
            rec["weights_requantized_each_step"] = {"ms_per_step": ms_r, "effective_tflops": world * wr.flops / (ms_r * 1e-3) / 1e12,
                                                    "split_overhead_vs_plain_gemms": ms_r / ms_gemm - 1.0,
                                                    "stored_residual": "float32, re-quantized with its own amax/2688"}
            del wr, g_r
            torch.cuda.empty_cache()
            # The same block with every operand decomposed from all of its rows (the paper's "without sparse random
            # sampling" ablation, Section 4 / Table 2): sketch, orthonormalisation and projection run over 16384 rows.
            wf = Workload(name, spec, B, synth, handles, streams, args.weights, world, rank, dw_sets=1, act_sketch=B.SKETCH_FULL)
            for i in range(args.warmup):
                wf.step(i)
            barrier()
            ms_f = max_over_ranks([timed_ms(torch, wf.step, max(3, args.steps // 4))])[0]
            rec["every_operand_full_sketch"] = {"ms_per_step": ms_f, "effective_tflops": world * wf.flops / (ms_f * 1e-3) / 1e12,
                                                "split_overhead_vs_plain_gemms": ms_f / ms_gemm - 1.0, "cuda_graph": False}
            del wf
            torch.cuda.empty_cache()

        if is_head:
            # ---- end to end: pinned host inputs in, results out, every step -------------------------------
            host_in = ({g: t.cpu().pin_memory() for g, t in wl.x_in.items()}, [t.cpu().pin_memory() for t in wl.w_in],
                       [t.cpu().pin_memory() for t in wl.d_in])
            stage = ({g: torch.empty_like(t) for g, t in wl.x_in.items()}, [torch.empty_like(t) for t in wl.w_in],
                     [torch.empty_like(t) for t in wl.d_in])
            host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in wl.y + wl.dx + wl.dw_sets[0]]
            s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
            # Two landing sets for the inputs and two take-off sets for the results, so that the copies of steps i + 1
            # (in) and i - 1 (out) run while step i computes: the step reads its inputs from `stage` and writes the
            # workload's output buffers (the captured graph has those addresses), a device copy on the compute stream
            # moves a landed set in and the finished results out (2.7 + 3.1 GB at HBM speed: ~2 ms of the step).
            flat = lambda st: list(st[0].values()) + st[1] + st[2]
            land = [[torch.empty_like(t) for t in flat(stage)] for _ in range(2)]
            outs_dev = wl.y + wl.dx + wl.dw_sets[0]
            takeoff = [[torch.empty_like(t) for t in outs_dev] for _ in range(2)]
            host_flat = flat(host_in)
            ev_in = [torch.cuda.Event() for _ in range(2)]       # landing set b holds step i's inputs
            ev_free = [torch.cuda.Event() for _ in range(2)]     # landing set b has been copied into `stage`
            ev_ready = [torch.cuda.Event() for _ in range(2)]    # take-off set b holds step i's results
            ev_out = [torch.cuda.Event() for _ in range(2)]      # take-off set b has reached the host
            g_e2e = None
            if use_graph:
                g_e2e = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_e2e):
                    wl.step(0, inputs=stage)

            def e2e_step(i):
                b_ = i & 1
                comp = torch.cuda.current_stream()
                s_in.wait_event(ev_free[b_])                 # the step that last used this landing set has taken it over
                with torch.cuda.stream(s_in):
                    for dst, src in zip(land[b_], host_flat):
                        dst.copy_(src, non_blocking=True)
                    ev_in[b_].record(s_in)
                comp.wait_event(ev_in[b_])
                for dst, src in zip(flat(stage), land[b_]):
                    dst.copy_(src, non_blocking=True)
                ev_free[b_].record(comp)
                if g_e2e is not None:
                    g_e2e.replay()
                else:
                    wl.step(i, inputs=stage)
                comp.wait_event(ev_out[b_])                  # the results of step i - 2 have left this take-off set
                for dst, src in zip(takeoff[b_], outs_dev):
                    dst.copy_(src, non_blocking=True)
                ev_ready[b_].record(comp)
                s_out.wait_event(ev_ready[b_])
                with torch.cuda.stream(s_out):
                    for host_t, dev_t in zip(host_out, takeoff[b_]):
                        host_t.copy_(dev_t, non_blocking=True)
                    ev_out[b_].record(s_out)

            for i in range(2):
                e2e_step(i)
            barrier()
            n_e2e = max(4, min(args.steps, 20))
            e0.record()
            for i in range(n_e2e):
                e2e_step(i)
            for ev in ev_out:
                torch.cuda.current_stream().wait_event(ev)
            e1.record()
            barrier()
            ms_e2e = max_over_ranks([e0.elapsed_time(e1) / n_e2e])[0]
            headline = {"rec": rec, "ms": ms, "ms_e2e": ms_e2e, "flops": wl.flops, "launches": int(launches_per_step) * args.steps,
                        "h2d": int(wl.input_bytes), "d2h": int(wl.output_bytes), "n_e2e": n_e2e,
                        "ms_big": ms_big, "big_flops": big_flops, "big_bytes": big_bytes, "big_shape": rec["largest_gemm"]["shape_mnk"],
                        "quant": rec["split_quantize"]}
            del host_in, stage, host_out, g_e2e, land, takeoff
        del wl, graphs, in_sets, pairs, big
        torch.cuda.empty_cache()

    sampler.stop()
    hd = headline
    gemm_tflops = hd["big_flops"] / (hd["ms_big"] * 1e-3) / 1e12
    q = hd["quant"]
    line = {
        "metric": "split_fp4_linear_fwd_bwd_effective_tflops",
        "value": world * hd["flops"] / (hd["ms"] * 1e-3) / 1e12,
        "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": hd["ms"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4 (e2m1 x ue4m3, fp32 accumulate)",
        "data": "synthetic",
        "config": {"workload": WORKLOADS[HEADLINE]["text"], "weights": args.weights, "cuda_graph": hd["rec"]["cuda_graph"],
                   "l2": "inputs of one step are %d MB, far above the 126 MB L2 (no rotation needed)" % (hd["h2d"] // 2 ** 20),
                   "parallelism": ("dp%d (token-sharded, FP32 dW all-reduce overlapping the next step)" % world) if world > 1 else "single GPU"},
        "e2e": {"value": world * hd["flops"] / (hd["ms_e2e"] * 1e-3) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": hd["h2d"], "d2h_bytes_per_step": hd["d2h"], "ms_per_step": hd["ms_e2e"], "steps": hd["n_e2e"],
                "overlap": "copies in, compute and copies out of consecutive steps run on three streams, two buffer sets each way"},
        "gpu_launches": hd["launches"],
        "clocks": hd["rec"]["clocks"],
        "roofline": {"bound": "tensor", "kernel": "two_cta::gemm_nvfp4_2cta_kernel, the largest residual GEMM of the block (M, N, K = %s), bf16 out" % hd["big_shape"],
                     "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s", "frac": gemm_tflops / fp4_peak,
                     "traffic": NCU_DRAM_BYTES.get(tuple(hd["big_shape"])), "traffic_source": NCU_DRAM_SOURCE,
                     "algorithmic_bytes": hd["big_bytes"],
                     "peak_source": "bf16 burst peak (%s) x %.0f nominal FP4:bf16 ratio" % (peaks["source"], FP4_OVER_BF16),
                     "ms_per_launch": hd["ms_big"]},
        "rooflines_hbm": {"peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "algorithmic_bytes_per_element": BYTES_PER_ELEM_BOTH,
                          "fused_residual_quantizer_chain_x": q["x_sampled"], "fused_residual_quantizer_chain_dy_sr": q["dy_sampled_sr"],
                          "quantize_kernel_rne": q["plain_quantizer_rne"], "quantize_kernel_sr": q["plain_quantizer_sr"]},
        "split_overhead_vs_plain_gemms": hd["rec"]["split_overhead_vs_plain_gemms"],
        "sustained": hd["rec"]["sustained"],
        "workloads": records,
    }
    if rank == 0 and not args.no_fp4_probe:
        # the kernel's own best rate: one 16384^3 product (221 tiles of 256 x 256 per CTA pair and 64 K blocks per tile), random codes
        n_p = 16384
        src = torch.randn((n_p, n_p), dtype=torch.bfloat16, device="cuda")
        qa, qb = B.NvFp4(n_p, n_p), B.NvFp4(n_p, n_p)
        handles[0].quantize_nvfp4(src, B.BLOCKS_BOTH, B.ROUND_RNE, seed=1, out=(qa, qb))
        del src
        out_p = torch.empty((n_p, n_p), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            handles[0].gemm_nvfp4(qa, qb, out=out_p)
        torch.cuda.synchronize()
        ms_p = timed_ms(torch, lambda i: handles[0].gemm_nvfp4(qa, qb, out=out_p), 10)
        tf_p = 2.0 * n_p ** 3 / (ms_p * 1e-3) / 1e12
        line["roofline"]["same_kernel_16384_cubed"] = {"ms": ms_p, "tflops": tf_p, "frac_of_peak": tf_p / fp4_peak,
                                                       "frac_of_nominal_9000": tf_p / 9000.0}
        del qa, qb, out_p
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = 4096
        dt, f, phases = oracle_sample_step(sample, 4242)
        line["cpu_baseline"] = {"value": f / dt / 1e12, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle",
                                "sample": "the q projection of the block (4096->4096) on %d of 16384 tokens, one pass (%.1f s)" % (sample, dt),
                                "phases": phases}
    if args.dry_run_ranks_on_one_gpu:
        line["dry_run"] = "%d ranks on one GPU, gloo: control flow only, not a measurement" % world
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

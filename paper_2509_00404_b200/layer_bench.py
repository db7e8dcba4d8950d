"""Times one split-FP4 linear layer of any shape on one GPU (forward + input gradient + weight gradient,
all three operands split and quantized inside the timed step) and prints one JSON line.

    python -m paper_2509_00404_b200.layer_bench --tokens 8192 --d-in 4096 --d-out 14336 --k 32 --p 8

Besides the step it times, each alone: the decomposition of every operand (algorithmic bytes = 2 B read +
2 x 0.5625 B written per element, both block orientations), the plain quantizer on X, and the three FP4 GEMMs
of the same layer without any split (the denominator of the split overhead).  Inputs are planted-spectrum
matrices generated on the device (rank-r spike, top singular value 100x the bulk edge, 10:1 span, Gaussian
bulk); they are regenerated from the seed, never read from disk.  Timing: CUDA events on the launching stream,
inputs rotate over enough sets to exceed the L2; the step (about 90 kernels on three streams) is replayed as one
CUDA graph per input set unless --no-graph is given, so that the host's launch rate does not bound the smaller layers.
"""
import argparse
import json
import math

import torch

from . import binding as B

L2_BYTES = 126e6


def planted_device(rows, cols, rank, sigma, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    u, _ = torch.linalg.qr(torch.randn((rows, rank), generator=g, device="cuda"))
    v, _ = torch.linalg.qr(torch.randn((cols, rank), generator=g, device="cuda"))
    s_top = 100.0 * sigma * (math.sqrt(rows) + math.sqrt(cols))
    s = torch.logspace(math.log10(s_top), math.log10(s_top / 10.0), rank, device="cuda")
    m = (u * s) @ v.T
    m += sigma * torch.randn((rows, cols), generator=g, device="cuda")
    return m.to(torch.bfloat16)


def timed(fn, reps, stream=None):
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
    ap.add_argument("--tokens", type=int, required=True)
    ap.add_argument("--d-in", type=int, required=True)
    ap.add_argument("--d-out", type=int, required=True)
    ap.add_argument("--k", type=int, default=32)
    ap.add_argument("--p", type=int, default=8)
    ap.add_argument("--rank", type=int, default=32, help="planted rank of the synthetic inputs")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--no-graph", action="store_true", help="time host launches instead of CUDA graph replays")
    a = ap.parse_args()
    l, m, n, k, p = a.tokens, a.d_in, a.d_out, a.k, a.p
    bf = torch.bfloat16
    per_set = 2 * (l * m + n * m + l * n)
    n_sets = max(1, min(3, int(math.ceil(2 * L2_BYTES / per_set))))
    sets = [{"x": planted_device(l, m, a.rank, 1.0, 5000 + 10 * s), "w": planted_device(n, m, a.rank, 0.02, 5001 + 10 * s),
             "dy": planted_device(l, n, a.rank, 1e-4, 5002 + 10 * s)} for s in range(n_sets)]
    h_x, h_w, h_d = B.Handle(0), B.Handle(0), B.Handle(0)
    xo, wo, do = B.Operand(l, m, k), B.Operand(n, m, k), B.Operand(l, n, k)
    y = torch.empty((l, n), dtype=bf, device="cuda")
    dx = torch.empty((l, m), dtype=bf, device="cuda")
    dw = torch.empty((n, m), dtype=bf, device="cuda")
    side_w, side_d = torch.cuda.Stream(), torch.cuda.Stream()
    ev0, ev_w, ev_d = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

    def split_x(i): h_x.split(sets[i % n_sets]["x"], k, p, sketch=B.SKETCH_SAMPLED, seed=3 * i + 1, out=xo)
    def split_w(i, st=None): h_w.split(sets[i % n_sets]["w"], k, p, sketch=B.SKETCH_FULL, seed=3 * i + 2, out=wo, stream=st)
    def split_d(i, st=None): h_d.split(sets[i % n_sets]["dy"], k, p, sketch=B.SKETCH_SAMPLED, seed=3 * i + 3, rounding=B.ROUND_SR, out=do, stream=st)

    ev_x, ev_b = torch.cuda.Event(), torch.cuda.Event()

    def step(i):
        main_s = torch.cuda.current_stream()
        ev0.record(main_s)
        side_w.wait_event(ev0)
        side_d.wait_event(ev0)
        with torch.cuda.stream(side_w):
            split_w(i, side_w)
            ev_w.record(side_w)
        with torch.cuda.stream(side_d):
            split_d(i, side_d)
            ev_d.record(side_d)
        split_x(i)
        ev_x.record(main_s)
        main_s.wait_event(ev_w)
        h_x.linear_fwd(xo, wo, out=y)
        # the backward products need dY, X and W but not the forward product: they follow dY's decomposition on its stream
        side_d.wait_event(ev_x)
        side_d.wait_event(ev_w)
        with torch.cuda.stream(side_d):
            h_d.linear_bwd(do, xo, wo, out=(dx, dw), stream=side_d)
            ev_b.record(side_d)
        main_s.wait_event(ev_b)

    for i in range(a.warmup):
        step(i)
    torch.cuda.synchronize()
    status = h_x.device_status() | h_w.device_status() | h_d.device_status()
    graphs = []
    if not a.no_graph:
        try:
            for s_i in range(n_sets):
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_):
                    step(s_i)
                graphs.append(g_)
            graphs[0].replay()
            torch.cuda.synchronize()
        except Exception:
            graphs = []
            torch.cuda.synchronize()
    ms_step = timed((lambda i: graphs[i % n_sets].replay()) if graphs else step, a.steps)
    ms_sx, ms_sw, ms_sd = timed(split_x, a.steps), timed(split_w, a.steps), timed(split_d, a.steps)

    # plain NVFP4 layer (k = 0): the three GEMMs alone, and the plain quantizer on X (both orientations)
    pairs = [(xo.res_by_cols, wo.res_by_cols, y), (do.res_by_cols, wo.res_by_rows, dx), (do.res_by_rows, xo.res_by_rows, dw)]
    def gemms(i):
        for a_, b_, o_ in pairs:
            h_x.gemm_nvfp4(a_, b_, out=o_)
    gemms(0)
    ms_gemm = timed(gemms, a.steps)
    qc, qr = B.NvFp4(l, m), B.NvFp4(m, l)
    def quant(i): h_x.quantize_nvfp4(sets[i % n_sets]["x"], B.BLOCKS_BOTH, B.ROUND_RNE, seed=1, out=(qc, qr))
    quant(0)
    ms_q = timed(quant, a.steps)

    gb = lambda elems, ms: 3.125 * elems / (ms * 1e-3) / 1e9
    line = {
        "layer": {"tokens": l, "d_in": m, "d_out": n, "k": k, "p": p},
        "ms_step": ms_step, "effective_tflops": 6.0 * l * m * n / (ms_step * 1e-3) / 1e12,
        "ms_three_plain_gemms": ms_gemm, "gemm_tflops": 6.0 * l * m * n / (ms_gemm * 1e-3) / 1e12,
        "split_overhead_vs_three_plain_gemms": ms_step / ms_gemm - 1.0,
        "split_ms": {"x_sampled": ms_sx, "w_full": ms_sw, "dy_sampled_sr": ms_sd},
        "split_gbs": {"x_sampled": gb(l * m, ms_sx), "w_full": gb(n * m, ms_sw), "dy_sampled_sr": gb(l * n, ms_sd)},
        "quantizer_both_orientations_gbs": gb(l * m, ms_q),
        "input_sets": n_sets, "cuda_graph": bool(graphs), "device_status": int(status),
    }
    print(json.dumps(line))


if __name__ == "__main__":
    main()

"""GPU parity: the split-FP4 linear layer end to end (Eq. 2, Eq. 3, weight gradient) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import layer as olay, nvfp4 as onv, split as osp
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 2e-3        # relative Frobenius error of layer outputs / gradients against the oracle's own split-FP4 result


@pytest.fixture(scope="module")
def ctx():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    yield B, h
    h.close()


def _check_e2e(case, errors, *pairs, base_tol=TOL):
    from gpu_util import check_e2e
    return check_e2e(case, errors, pairs, base_tol)


def _oracle_from_gpu_operand(op, k):
    """Dequantize the library's own quantized pieces in float64 (isolates the GEMM composition from the split)."""
    from gpu_util import nv_dequant
    res_c = nv_dequant(op.res_by_cols) if op.res_by_cols else None
    res_r = nv_dequant(op.res_by_rows).T if op.res_by_rows else None
    if k == 0:
        z = np.zeros((op.rows, op.cols))
        return z, res_c, res_r
    lq, rq = nv_dequant(op.left_q)[:k].T, nv_dequant(op.right_q)[:k].T
    low = (lq * op.sigma.cpu().numpy().astype(np.float64)) @ rq.T
    return low, res_c, res_r


def test_small_config_forward(ctx):
    from gpu_util import to_dev_bf16, rel_fro
    B, h = ctx
    c = synth.config_small()
    xo = h.split(to_dev_bf16(c["x"]), 4, 4, sketch=B.SKETCH_FULL, seed=1)
    wo = h.split(to_dev_bf16(c["w"]), 4, 4, sketch=B.SKETCH_FULL, seed=2)
    y = h.linear_fwd(xo, wo)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    xq = olay.quantize_operand(c["x"], 4, 4, osp.MODE_FULL, 1)
    wq = olay.quantize_operand(c["w"], 4, 4, osp.MODE_FULL, 2)
    _check_e2e("small_config_forward_128tok_256to256_k4", {"y": rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq))}, (xo, xq), (wo, wq))
    # composition alone, on the library's own codes: tight
    lx, rxc, _ = _oracle_from_gpu_operand(xo, 4)
    lw, rwc, _ = _oracle_from_gpu_operand(wo, 4)
    assert rel_fro(y.cpu().numpy(), (lx + rxc) @ (lw + rwc).T) < 2e-5


@pytest.mark.parametrize("k", [0, 8])
def test_forward_and_backward_medium(ctx, k):
    from gpu_util import to_dev_bf16, rel_fro
    B, h = ctx
    l, m, n, p = 512, 384, 256, 8 if k else 0
    x, _ = synth.llama_like(l, m, 1.0, 51, rank=8)
    w, _ = synth.llama_like(n, m, 0.02, 52, rank=8)
    d, _ = synth.llama_like(l, n, 1e-4, 53, rank=8)
    xo = h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
    wo = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2)
    do = h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
    y = h.linear_fwd(xo, wo)
    dx, dw = h.linear_bwd(do, xo, wo)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, 2)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    _check_e2e("medium_512tok_384to256_k%d" % k,
               {"y": rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq)), "dx": rel_fro(dx.cpu().numpy(), olay.linear_dgrad(dq, wq)),
                "dw": rel_fro(dw.cpu().numpy(), olay.linear_wgrad(dq, xq))}, (xo, xq), (wo, wq), (do, dq))
    lx, rxc, rxr = _oracle_from_gpu_operand(xo, k)
    lw, rwc, rwr = _oracle_from_gpu_operand(wo, k)
    ld, rdc, rdr = _oracle_from_gpu_operand(do, k)
    assert rel_fro(y.cpu().numpy(), (lx + rxc) @ (lw + rwc).T) < 2e-5
    assert rel_fro(dx.cpu().numpy(), (ld + rdc) @ (lw + rwr)) < 2e-5
    assert rel_fro(dw.cpu().numpy(), (ld + rdr).T @ (lx + rxr)) < 2e-5


@pytest.mark.parametrize("k", [0, 8, 128])
def test_layer_on_the_oracles_own_bytes(ctx, k):
    """No discontinuity in the way: the ORACLE's codes, scale bytes, tensor scales and singular values are uploaded
    into the library's operands, so both sides multiply exactly the same quantized tensors.  Eq. 2, Eq. 3 and the
    weight gradient must then agree with the oracle's float64 evaluation to FP32-accumulation accuracy, with no
    allowance of any kind."""
    from gpu_util import rel_fro, operand_from_oracle
    B, h = ctx
    l, m, n, p = (512, 384, 256, 8 if k else 0) if k <= 64 else (1024, 768, 640, 8)      # k = 128: the wide-rank composition
    x, _ = synth.llama_like(l, m, 1.0, 51, rank=max(k, 8))
    w, _ = synth.llama_like(n, m, 0.02, 52, rank=max(k, 8))
    d, _ = synth.llama_like(l, n, 1e-4, 53, rank=max(k, 8))
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, 2)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    xo, wo, do = (operand_from_oracle(B, q) for q in (xq, wq, dq))
    y = h.linear_fwd(xo, wo)
    fg = tuple(torch.full(sh, float("nan"), device="cuda") for sh in ((k, n), (k,), (k, m))) if k else None
    dx, dw = h.linear_bwd(do, xo, wo, factor_grads=fg)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    errs = (rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq)), rel_fro(dx.cpu().numpy(), olay.linear_dgrad(dq, wq)),
            rel_fro(dw.cpu().numpy(), olay.linear_wgrad(dq, xq)))
    print("layer on the oracle's bytes, k = %d: y %.2e dx %.2e dw %.2e" % (k, *errs))
    assert max(errs) < 2e-5
    if k:
        du, ds, dv = olay.factor_grads(olay.linear_wgrad(dq, xq), wq)
        d_left, d_sigma, d_right = fg
        assert rel_fro(d_right.cpu().numpy().T, du) < 2e-5 and rel_fro(d_left.cpu().numpy().T, dv) < 2e-5
        assert rel_fro(d_sigma.cpu().numpy(), ds) < 2e-5


@pytest.mark.parametrize("dw_dtype", [torch.float32, torch.bfloat16])
def test_factor_gradients(ctx, dw_dtype):
    """dL/dU, dL/dS, dL/dV of the weight factors (Section 3.2) against the oracle."""
    from gpu_util import to_dev_bf16, rel_fro, nv_dequant
    B, h = ctx
    l, m, n, k, p = 256, 448, 192, 12, 4
    x, _ = synth.llama_like(l, m, 1.0, 61, rank=8)
    w, _ = synth.llama_like(n, m, 0.02, 62, rank=8)
    d, _ = synth.llama_like(l, n, 1e-4, 63, rank=8)
    xo = h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
    wo = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2)
    do = h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
    d_left = torch.full((k, n), float("nan"), device="cuda")
    d_sigma = torch.full((k,), float("nan"), device="cuda")
    d_right = torch.full((k, m), float("nan"), device="cuda")
    dx, dw = h.linear_bwd(do, xo, wo, out_dtype=dw_dtype, factor_grads=(d_left, d_sigma, d_right))
    torch.cuda.synchronize()
    assert h.device_status() == 0
    # (a) the three contractions themselves, from the library's own dw and dequantized factors, in float64
    dwn = dw.float().cpu().numpy().astype(np.float64)
    lq, rq = nv_dequant(wo.left_q)[:k].T, nv_dequant(wo.right_q)[:k].T            # n x k (V), m x k (U)
    sig = wo.sigma.cpu().numpy().astype(np.float64)
    assert rel_fro(d_left.cpu().numpy().T, (dwn @ rq) * sig) < 1e-5
    assert rel_fro(d_right.cpu().numpy().T, (dwn.T @ lq) * sig) < 1e-5
    assert rel_fro(d_sigma.cpu().numpy(), np.einsum("jt,ji,it->t", lq, dwn, rq)) < 1e-5
    # (b) end to end against the oracle's own split, quantization and weight gradient
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, 2)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    du, ds, dv = olay.factor_grads(olay.linear_wgrad(dq, xq), wq)
    base = TOL if dw_dtype == torch.float32 else 3 * TOL                          # a BF16 dw carries 2^-9 per entry
    _check_e2e("factor_gradients_256tok_448to192_k12_dw_%s" % ("fp32" if dw_dtype == torch.float32 else "bf16"),
               {"dU": rel_fro(d_right.cpu().numpy().T, du), "dV": rel_fro(d_left.cpu().numpy().T, dv),
                "dS": rel_fro(d_sigma.cpu().numpy(), ds)}, (xo, xq), (wo, wq), (do, dq), base_tol=base)


def test_factor_gradients_need_the_weight_gradient(ctx):
    from gpu_util import to_dev_bf16
    B, h = ctx
    c = synth.config_small()
    xo = h.split(to_dev_bf16(c["x"]), 4, 4, sketch=B.SKETCH_FULL, seed=1)
    wo = h.split(to_dev_bf16(c["w"]), 4, 4, sketch=B.SKETCH_FULL, seed=2)
    do = h.split(torch.randn(128, 256, device="cuda").to(torch.bfloat16), 4, 4, sketch=B.SKETCH_FULL, seed=3)
    g = torch.zeros((4, 256), device="cuda")
    with pytest.raises(RuntimeError):
        h.linear_bwd(do, xo, wo, need_dw=False, factor_grads=(g, None, None))


@pytest.mark.parametrize("kp", [(12, 4), (24, 8), (40, 0), (48, 8), (64, 8)])
def test_rank_and_oversampling_range(ctx, kp):
    """Ranks that are not multiples of 16 (padded coefficient blocks), no oversampling, and the largest rank."""
    from gpu_util import to_dev_bf16, rel_fro
    B, h = ctx
    k, p = kp
    l, m, n = 512, 768, 640
    x, _ = synth.llama_like(l, m, 1.0, 91, rank=max(k, 8))
    w, _ = synth.llama_like(n, m, 0.02, 92, rank=max(k, 8))
    d, _ = synth.llama_like(l, n, 1e-4, 93, rank=max(k, 8))
    xo = h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
    wo = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2)
    do = h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
    y = h.linear_fwd(xo, wo)
    dx, dw = h.linear_bwd(do, xo, wo)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, 2)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    for op, q in ((xo, xq), (wo, wq), (do, dq)):
        assert np.max(np.abs(op.sigma.cpu().numpy()[:k] - q.sigma) / q.sigma) < 1e-3
    _check_e2e("rank_range_512tok_768to640_k%d_p%d" % (k, p),
               {"y": rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq)), "dx": rel_fro(dx.cpu().numpy(), olay.linear_dgrad(dq, wq)),
                "dw": rel_fro(dw.cpu().numpy(), olay.linear_wgrad(dq, xq))}, (xo, xq), (wo, wq), (do, dq))


def test_ragged_layer_through_the_two_cta_gemm(ctx):
    """l, m, n above 256 but not multiples of the 256-wide GEMM tiles: ragged tiles in every product, the fused
    low-rank correction boxes, tensor stores clipped at the matrix edge."""
    from gpu_util import to_dev_bf16, rel_fro
    B, h = ctx
    l, m, n, k, p = 320, 448, 320, 8, 4
    x, _ = synth.llama_like(l, m, 1.0, 81, rank=8)
    w, _ = synth.llama_like(n, m, 0.02, 82, rank=8)
    d, _ = synth.llama_like(l, n, 1e-4, 83, rank=8)
    xo = h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
    wo = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2)
    do = h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
    y = h.linear_fwd(xo, wo)
    dx, dw = h.linear_bwd(do, xo, wo)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    lx, rxc, rxr = _oracle_from_gpu_operand(xo, k)
    lw, rwc, rwr = _oracle_from_gpu_operand(wo, k)
    ld, rdc, rdr = _oracle_from_gpu_operand(do, k)
    assert rel_fro(y.cpu().numpy(), (lx + rxc) @ (lw + rwc).T) < 2e-5
    assert rel_fro(dx.cpu().numpy(), (ld + rdc) @ (lw + rwr)) < 2e-5
    assert rel_fro(dw.cpu().numpy(), (ld + rdr).T @ (lx + rxr)) < 2e-5
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = olay.quantize_operand(w, k, p, osp.MODE_FULL, 2)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    _check_e2e("ragged_320tok_448to320_k8",
               {"y": rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq)), "dx": rel_fro(dx.cpu().numpy(), olay.linear_dgrad(dq, wq)),
                "dw": rel_fro(dw.cpu().numpy(), olay.linear_wgrad(dq, xq))}, (xo, xq), (wo, wq), (do, dq))


def test_bf16_output(ctx):
    from gpu_util import to_dev_bf16, rel_fro
    B, h = ctx
    c = synth.config_small()
    xo = h.split(to_dev_bf16(c["x"]), 4, 4, sketch=B.SKETCH_FULL, seed=1)
    wo = h.split(to_dev_bf16(c["w"]), 4, 4, sketch=B.SKETCH_FULL, seed=2)
    y32 = h.linear_fwd(xo, wo)
    y16 = h.linear_fwd(xo, wo, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert rel_fro(y16.float().cpu().numpy(), y32.cpu().numpy()) < 4e-3


def test_repeated_calls_are_bit_identical(ctx):
    """Same inputs, same seeds: every byte of every output is the same from call to call.  The decomposition, the
    forward and the backward fork into the handle's side streams (the backward into all of them), so a missing join
    or a shared intermediate would show up here as a changed bit."""
    from gpu_util import to_dev_bf16
    B, h = ctx
    l, m, n, k, p = 1024, 768, 512, 16, 8
    x, _ = synth.llama_like(l, m, 1.0, 61, rank=16)
    w, _ = synth.llama_like(n, m, 0.02, 62, rank=16)
    d, _ = synth.llama_like(l, n, 1e-4, 63, rank=16)
    xd, wd, dd = to_dev_bf16(x), to_dev_bf16(w), to_dev_bf16(d)

    def run():
        xo = h.split(xd, k, p, sketch=B.SKETCH_SAMPLED, seed=1)
        wo = h.split(wd, k, p, sketch=B.SKETCH_FULL, seed=2)
        do = h.split(dd, k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
        y = h.linear_fwd(xo, wo, out_dtype=torch.bfloat16)
        dx, dw = h.linear_bwd(do, xo, wo)
        torch.cuda.synchronize()
        return [y, dx, dw, xo.left, xo.right, xo.sigma, do.res_by_cols.codes, do.res_by_rows.codes, wo.left_q.codes]

    first = [t.clone() for t in run()]
    for _ in range(5):
        again = run()
        assert all(torch.equal(a, b) for a, b in zip(first, again))
    assert h.device_status() == 0


def test_concurrent_step_replayed_many_times_is_bit_identical():
    """The whole step of a 4096-token layer - three decompositions on three streams, forward and backward - captured
    once and replayed 1500 times: every replay must reproduce the first one bit for bit.  Kernels of different
    operands overlap differently from replay to replay, which is what exposes a missing ordering between a buffer's
    readers and the copy that refills it (such a gap once let one step in a few hundred through with a 32 x 8 patch of
    wrong residual values)."""
    from paper_2509_00404_b200 import binding as B
    l = m = n = 4096
    k, p = 32, 8
    x, w, d = synth.planted_device(l, m, 32, 1.0, 11), synth.planted_device(n, m, 32, 0.02, 12), synth.planted_device(l, n, 32, 1e-4, 13)
    hx, hw, hd = B.Handle(0), B.Handle(0), B.Handle(0)
    try:
        xo, wo, do = B.Operand(l, m, k), B.Operand(n, m, k), B.Operand(l, n, k)
        y = torch.empty((l, n), dtype=torch.bfloat16, device="cuda")
        dx, dw = torch.empty((l, m), dtype=torch.bfloat16, device="cuda"), torch.empty((n, m), dtype=torch.bfloat16, device="cuda")
        sw, sd = torch.cuda.Stream(), torch.cuda.Stream()
        e0, ew, ex, eb = (torch.cuda.Event() for _ in range(4))

        def step():
            main = torch.cuda.current_stream()
            e0.record(main); sw.wait_event(e0); sd.wait_event(e0)
            with torch.cuda.stream(sw):
                hw.split(w, k, p, sketch=B.SKETCH_FULL, seed=2, out=wo, stream=sw)
                ew.record(sw)
            hx.split(x, k, p, sketch=B.SKETCH_SAMPLED, seed=1, out=xo)
            ex.record(main)
            main.wait_event(ew)
            hx.linear_fwd(xo, wo, out=y)
            with torch.cuda.stream(sd):
                hd.split(d, k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR, out=do, stream=sd)
                sd.wait_event(ex); sd.wait_event(ew)
                hd.linear_bwd(do, xo, wo, out=(dx, dw), stream=sd)
                eb.record(sd)
            main.wait_event(eb)

        for _ in range(2):
            step()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        g.replay()
        torch.cuda.synchronize()
        watched = [y, dx, dw, xo.res_by_cols.codes, xo.res_by_rows.codes, wo.res_by_cols.codes, wo.res_by_rows.codes,
                   do.res_by_cols.codes, do.res_by_rows.codes, xo.res_by_cols.scales, do.res_by_rows.scales]
        first = [t.clone() for t in watched]
        bad = 0
        for _ in range(1500):
            g.replay()
            bad += int(not all(torch.equal(a, b) for a, b in zip(first, watched)))
        torch.cuda.synchronize()
        assert bad == 0, "%d of 1500 replays differ from the first" % bad
        assert (hx.device_status() | hw.device_status() | hd.device_status()) == 0
    finally:
        for h in (hx, hw, hd):
            h.close()

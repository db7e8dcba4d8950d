"""GPU parity at the benchmark's full size and launch configuration (one LLaMA-3-8B q_proj-shaped layer,
4096 tokens, 4096 -> 4096, k=32, p=8, SR on dY), checked on sampled output rows the oracle computes exactly."""
import numpy as np
import pytest
import torch

from oracle import layer as olay, nvfp4 as onv, split as osp
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 2e-3


def test_qproj_layer_forward_and_backward_on_sampled_rows():
    from gpu_util import rel_fro, check_e2e, operand_from_oracle
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    try:
        c = synth.config_qproj(seed=2000)
        k, p = c["k"], c["p"]
        dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
        xo = h.split(dev(c["x"]), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
        wo = h.split(dev(c["w"]), k, p, sketch=B.SKETCH_FULL, seed=2)
        do = h.split(dev(c["dy"]), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
        y = h.linear_fwd(xo, wo, out_dtype=torch.float32)
        d_left, d_sigma, d_right = (torch.empty(sh, device="cuda") for sh in ((k, 4096), (k,), (k, 4096)))
        dx, dw = h.linear_bwd(do, xo, wo, out_dtype=torch.float32, factor_grads=(d_left, d_sigma, d_right))
        torch.cuda.synchronize()
        assert h.device_status() == 0
        xq = olay.quantize_operand(c["x"], k, p, osp.MODE_SAMPLED, 1)
        wq = olay.quantize_operand(c["w"], k, p, osp.MODE_FULL, 2)
        dq = olay.quantize_operand(c["dy"], k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
        # top-k singular values of all three operands
        for op, q in ((xo, xq), (wo, wq), (do, dq)):
            sig = op.sigma.cpu().numpy().astype(np.float64)
            assert np.max(np.abs(sig - q.sigma) / q.sigma) < 1e-3
        rows = np.random.default_rng(0).choice(4096, 192, replace=False)
        xd, wd_c = xq.dense(onv.AXIS_COLS), wq.dense(onv.AXIS_COLS)
        dd_c, wd_r = dq.dense(onv.AXIS_COLS), wq.dense(onv.AXIS_ROWS)
        dd_r, xd_r = dq.dense(onv.AXIS_ROWS), xq.dense(onv.AXIS_ROWS)
        # factor gradients of the weight operand (sampled rows of dL/dV, all of dL/dS and dL/dU) from the oracle's dW
        dw_o = dd_r.T @ xd_r
        du, ds, dv = olay.factor_grads(dw_o, wq)
        check_e2e("bench_workload_qproj_4096tok_4096to4096_k32_sampled_rows",
                  {"y": rel_fro(y.cpu().numpy()[rows], xd[rows] @ wd_c.T), "dx": rel_fro(dx.cpu().numpy()[rows], dd_c[rows] @ wd_r),
                   "dw": rel_fro(dw.cpu().numpy()[rows], dw_o[rows]), "dV": rel_fro(d_left.cpu().numpy().T[rows], dv[rows]),
                   "dU": rel_fro(d_right.cpu().numpy().T, du), "dS": rel_fro(d_sigma.cpu().numpy(), ds)},
                  [(xo, xq), (wo, wq), (do, dq)])
        # the same three products on the ORACLE's own bytes (uploaded codes, scales, singular values): no rounding
        # decision can differ, so the comparison is at FP32-accumulation accuracy and needs no allowance
        del xo, wo, do, y, dx, dw
        xo, wo, do = (operand_from_oracle(B, q) for q in (xq, wq, dq))
        y = h.linear_fwd(xo, wo, out_dtype=torch.float32)
        dx, dw = h.linear_bwd(do, xo, wo, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        assert rel_fro(y.cpu().numpy()[rows], xd[rows] @ wd_c.T) < 2e-5
        assert rel_fro(dx.cpu().numpy()[rows], dd_c[rows] @ wd_r) < 2e-5
        assert rel_fro(dw.cpu().numpy()[rows], dw_o[rows]) < 2e-5
    finally:
        h.close()

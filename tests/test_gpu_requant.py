"""GPU parity: metis_requantize_operand, the per-step work of an operand that is kept as stored factors and residual
(Section 3.2 holds a weight as U, S, V and W_R and refreshes only their NVFP4 forms), against the oracle."""
import numpy as np
import pytest
import torch

from oracle import layer as olay, nvfp4 as onv, split as osp
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    yield B, h
    h.close()


def _bytes(t):
    from gpu_util import nv_to_numpy
    return nv_to_numpy(t)


@pytest.mark.parametrize("case", [(384, 512, 8, 8, 0), (640, 448, 24, 8, 1), (1024, 768, 128, 8, 0), (256, 320, 0, 0, 1)],
                         ids=lambda c: "%dx%d_k%d_%s" % (c[0], c[1], c[2], "sr" if c[4] else "rne"))
def test_requantized_operand_matches_the_oracle_byte_for_byte(ctx, case):
    from gpu_util import to_dev_bf16
    B, h = ctx
    n, m, k, p, rounding = case
    w, _ = synth.llama_like(n, m, 0.02, 300 + k, rank=max(k, 8))
    wo, dense = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2, rounding=rounding, want_residual=True)
    if k == 0:
        dense = to_dev_bf16(w).float()                   # a plain operand has no residual of its own: the tensor itself
    torch.cuda.synchronize()
    s_src = onv.tensor_scale_from_amax(np.max(np.abs(w)))
    first = {name: _bytes(getattr(wo, name)) for name in ("res_by_cols", "res_by_rows", "left_q", "right_q")}
    left32, right32, sig = wo.left.cpu().numpy()[:k].T, wo.right.cpu().numpy()[:k].T, wo.sigma.cpu().numpy()[:k]
    res32 = dense.cpu().numpy()
    # (a) stored pieces + the scale of the original split: every byte of the split comes back
    for t in (wo.res_by_cols, wo.res_by_rows, wo.left_q, wo.right_q):
        t.codes.fill_(0x5A); t.scales.fill_(0x11)
    h.requantize_operand(wo, dense, rounding=rounding, seed=2, given_scale=float(s_src))
    torch.cuda.synchronize()
    assert h.device_status() == 0
    for name in ("res_by_cols", "res_by_rows") + (("left_q", "right_q") if k else ()):
        c, s, ts = _bytes(getattr(wo, name))
        rows_valid = k if name.endswith("_q") else c.shape[0]
        assert ts == first[name][2] and np.array_equal(c[:rows_valid], first[name][0][:rows_valid]) and np.array_equal(s[:rows_valid], first[name][1][:rows_valid]), name
    # (b) the stored-weight default (own amax as the residual's tensor scale) against the oracle on the same values
    ref = olay.requantize_operand(left32, sig, right32, res32, rounding, seed=2)
    h.requantize_operand(wo, dense, rounding=rounding, seed=2)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    pairs = [("res_by_cols", "res_by_cols"), ("res_by_rows", "res_by_rows")] + ([("left_q", "left"), ("right_q", "right")] if k else [])
    for name, oname in pairs:
        c, s, ts = _bytes(getattr(wo, name))
        oc, os_, ots = ref.raw[oname]
        assert ts == ots and np.array_equal(c[: oc.shape[0]], oc) and np.array_equal(s[: oc.shape[0]], os_), name
    # (c) a BF16 copy of the residual as the stored form: bytes of the oracle on the rounded values
    res_bf = dense.to(torch.bfloat16)
    ref_bf = olay.requantize_operand(left32, sig, right32, res_bf.float().cpu().numpy(), rounding, seed=2)
    h.requantize_operand(wo, res_bf, rounding=rounding, seed=2)
    torch.cuda.synchronize()
    for name in ("res_by_cols", "res_by_rows"):
        c, s, ts = _bytes(getattr(wo, name))
        oc, os_, ots = ref_bf.raw[name]
        assert ts == ots and np.array_equal(c, oc) and np.array_equal(s, os_), name


def test_layer_with_a_requantized_weight_matches_the_oracle(ctx):
    """The step the paper describes for weights: the stored pieces are re-quantized, then Eq. 2, Eq. 3 and the weight
    gradient run on them.  Both sides hold the same bytes, so the products agree to FP32-accumulation accuracy."""
    from gpu_util import to_dev_bf16, rel_fro, operand_from_oracle
    B, h = ctx
    l, m, n, k, p = 512, 384, 320, 8, 8
    x, _ = synth.llama_like(l, m, 1.0, 51, rank=8)
    w, _ = synth.llama_like(n, m, 0.02, 52, rank=8)
    d, _ = synth.llama_like(l, n, 1e-4, 53, rank=8)
    wo, dense = h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2, want_residual=True)
    # an "optimizer step" on the stored pieces, then the refresh
    dense.mul_(0.97); wo.sigma.mul_(1.01)
    h.requantize_operand(wo, dense, seed=9)
    torch.cuda.synchronize()
    wq = olay.requantize_operand(wo.left.cpu().numpy()[:k].T, wo.sigma.cpu().numpy()[:k], wo.right.cpu().numpy()[:k].T,
                                 dense.cpu().numpy(), seed=9)
    xq = olay.quantize_operand(x, k, p, osp.MODE_SAMPLED, 1)
    dq = olay.quantize_operand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    xo, do = operand_from_oracle(B, xq), operand_from_oracle(B, dq)
    y = h.linear_fwd(xo, wo)
    dx, dw = h.linear_bwd(do, xo, wo)
    torch.cuda.synchronize()
    assert h.device_status() == 0
    assert rel_fro(y.cpu().numpy(), olay.linear_fwd(xq, wq)) < 2e-5
    assert rel_fro(dx.cpu().numpy(), olay.linear_dgrad(dq, wq)) < 2e-5
    assert rel_fro(dw.cpu().numpy(), olay.linear_wgrad(dq, xq)) < 2e-5


def test_requantize_rejects_bad_arguments(ctx):
    B, h = ctx
    op = B.Operand(128, 256, 4)
    res = torch.zeros((128, 256), device="cuda")
    with pytest.raises(B.MetisError):
        h.requantize_operand(op, res, axes=0)
    with pytest.raises(B.MetisError):
        h.requantize_operand(B.Operand(120, 256, 4), torch.zeros((120, 256), device="cuda"))

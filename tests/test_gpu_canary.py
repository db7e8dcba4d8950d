"""Guard bytes around every output of the ragged-shape cases (the stand-in for a memory checker, which is not
available where these tests run): codes, scale bytes, factors and layer outputs sit inside larger buffers whose
borders must come back untouched."""
import numpy as np
import pytest
import torch

from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


def _guarded_nvfp4(B, G, rows, k_len, keep):
    t = B.NvFp4.__new__(B.NvFp4)
    t.rows, t.k_len, t.layout = rows, k_len, B.SF_TILED
    gc, gs, gt = G((rows, k_len // 2), torch.uint8, 0), G((max(B.sf_bytes(rows, k_len, B.SF_TILED), 16),), torch.uint8, 0), G((1,), torch.float32, 0)
    t.codes, t.scales, t.tensor_scale = gc.view, gs.view, gt.view
    keep += [(gc, "codes %dx%d" % (rows, k_len)), (gs, "scales %dx%d" % (rows, k_len)), (gt, "tensor scale")]
    return t


def _guarded_operand(B, G, rows, cols, k, keep):
    op = B.Operand.__new__(B.Operand)
    op.rows, op.cols, op.k, op.axes = rows, cols, k, B.BLOCKS_BOTH
    gl, gg, gr = G((k, rows), torch.float32, 0), G((k,), torch.float32, 0), G((k, cols), torch.float32, 0)
    op.left, op.sigma, op.right = gl.view, gg.view, gr.view
    keep += [(gl, "left"), (gg, "sigma"), (gr, "right")]
    op.left_q, op.right_q = _guarded_nvfp4(B, G, k, rows, keep), _guarded_nvfp4(B, G, k, cols, keep)
    op.res_by_cols, op.res_by_rows = _guarded_nvfp4(B, G, rows, cols, keep), _guarded_nvfp4(B, G, cols, rows, keep)
    return op


@pytest.mark.parametrize("shape", [(320, 448, 320, 8, 4), (192, 576, 832, 12, 4), (1088, 320, 256, 0, 0)])
def test_ragged_layer_writes_nothing_outside_its_outputs(shape):
    from gpu_util import to_dev_bf16, Guarded
    from paper_2509_00404_b200 import binding as B
    l, m, n, k, p = shape
    x, _ = synth.llama_like(l, m, 1.0, 81, rank=8)
    w, _ = synth.llama_like(n, m, 0.02, 82, rank=8)
    d, _ = synth.llama_like(l, n, 1e-4, 83, rank=8)
    h = B.Handle(0)
    try:
        keep = []
        if k:
            xo, wo, do = (_guarded_operand(B, Guarded, r, c, k, keep) for r, c in ((l, m), (n, m), (l, n)))
        else:
            xo, wo, do = (B.Operand(r, c, 0) for r, c in ((l, m), (n, m), (l, n)))
            for op, (r, c) in zip((xo, wo, do), ((l, m), (n, m), (l, n))):
                op.res_by_cols, op.res_by_rows = _guarded_nvfp4(B, Guarded, r, c, keep), _guarded_nvfp4(B, Guarded, c, r, keep)
        h.split(to_dev_bf16(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1, out=xo)
        h.split(to_dev_bf16(w), k, p, sketch=B.SKETCH_FULL, seed=2, out=wo)
        h.split(to_dev_bf16(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR, out=do)
        for dt in (torch.float32, torch.bfloat16):
            gy, gdx, gdw = Guarded((l, n), dt, 0), Guarded((l, m), dt, 0), Guarded((n, m), dt, 0)
            h.linear_fwd(xo, wo, out=gy.view)
            h.linear_bwd(do, xo, wo, out=(gdx.view, gdw.view))
            torch.cuda.synchronize()
            assert h.device_status() == 0
            for g, name in ((gy, "y"), (gdx, "dx"), (gdw, "dw")):
                g.check(name)
                assert float(g.view.float().abs().max()) > 0
        for g, name in keep:
            g.check(name)
    finally:
        h.close()

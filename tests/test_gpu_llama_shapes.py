"""GPU parity on the other LLaMA-3 layer shapes of the workload list (SwiGLU FFN projections, GQA key/value
projections, a 70B-shaped projection with a rank sweep), checked on sampled outputs: the oracle splits every
operand in full and encodes only the residual rows / columns that the sampled outputs read (oracle_partial).
Every shape of the workload list is run at its full size (the decoder block's other projections have the shapes of
the q projection and of the FFN layers).  The quarter-scale rank-sweep cases are
small enough for the whole output to be compared, which matters for k = 16: the cut then falls inside the
planted rank-64 cluster (neighbouring singular values 3.7 % apart), FP32-level differences in the factors
flip more FP4 roundings than elsewhere, and a 64 x 64 sample of the output is too noisy a statistic."""
import numpy as np
import pytest
import torch

from oracle import nvfp4 as onv, split as osp
from oracle_partial import PartialOperand
from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 2e-3
N_SAMPLE = 256        # sampled rows and columns per output: a 64 x 64 sample is dominated by whichever re-rounded factor block it happens to contain

CASES = [
    # id, tokens, in, out, k, p, planted rank, compare the whole output
    ("ffn_up_8192tok_4096to14336", 8192, 4096, 14336, 32, 8, 32, False),
    ("ffn_down_8192tok_14336to4096", 8192, 14336, 4096, 32, 8, 32, False),
    ("gqa_kv_16384tok_4096to1024", 16384, 4096, 1024, 32, 8, 32, False),
    ("ffn_up_16384tok_4096to14336", 16384, 4096, 14336, 32, 8, 32, False),
    ("ffn_down_16384tok_14336to4096", 16384, 14336, 4096, 32, 8, 32, False),
    ("70b_proj_16384tok_8192to28672_k64", 16384, 8192, 28672, 64, 8, 64, False),
    ("70b_proj_16384tok_8192to28672_k256", 16384, 8192, 28672, 256, 8, 64, False),
    ("70b_proj_quarter_scale_2048to7168_k64", 1024, 2048, 7168, 64, 8, 64, True),
    ("70b_proj_quarter_scale_2048to7168_k16", 1024, 2048, 7168, 16, 8, 64, True),
    ("70b_proj_quarter_scale_2048to7168_k0", 1024, 2048, 7168, 0, 0, 64, True),
    ("70b_proj_quarter_scale_2048to7168_k128", 1024, 2048, 7168, 128, 8, 64, True),
    ("70b_proj_quarter_scale_2048to7168_k256", 2048, 2048, 7168, 256, 8, 64, True),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_layer_on_sampled_outputs(case):
    from gpu_util import rel_fro, nv_to_numpy, check_e2e
    from paper_2509_00404_b200 import binding as B
    _, l, m, n, k, p, rank, whole = case
    x, _ = synth.llama_like(l, m, 1.0, 3000, rank=rank)
    w, _ = synth.llama_like(n, m, 0.02, 3001, rank=rank)
    d, _ = synth.llama_like(l, n, 1e-4, 3002, rank=rank)
    h = B.Handle(0)
    try:
        dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
        xo = h.split(dev(x), k, p, sketch=B.SKETCH_SAMPLED, seed=1)
        wo = h.split(dev(w), k, p, sketch=B.SKETCH_FULL, seed=2)
        do = h.split(dev(d), k, p, sketch=B.SKETCH_SAMPLED, seed=3, rounding=B.ROUND_SR)
        y = h.linear_fwd(xo, wo, out_dtype=torch.float32)
        dx, dw = h.linear_bwd(do, xo, wo, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        rng = np.random.default_rng(11)
        rl, rn, cm = (np.arange(dim) if whole else np.sort(rng.choice(dim, N_SAMPLE, replace=False)) for dim in (l, n, m))
        y_s = y[torch.from_numpy(rl).cuda()][:, torch.from_numpy(rn).cuda()].cpu().numpy()
        dx_s = dx[torch.from_numpy(rl).cuda()][:, torch.from_numpy(cm).cuda()].cpu().numpy()
        dw_s = dw[torch.from_numpy(rn).cuda()][:, torch.from_numpy(cm).cuda()].cpu().numpy()
        sig = [o.sigma.cpu().numpy().astype(np.float64) for o in (xo, wo, do)] if k else []
        rights = [o.right.cpu().numpy()[:k].T.astype(np.float64) for o in (xo, wo, do)] if k > rank else []
        factors = [(nv_to_numpy(o.left_q), nv_to_numpy(o.right_q)) for o in (xo, wo, do)] if k else []
        del y, dx, dw
    finally:
        h.close()
    xq = PartialOperand(x, k, p, osp.MODE_SAMPLED, 1)
    wq = PartialOperand(w, k, p, osp.MODE_FULL, 2)
    dq = PartialOperand(d, k, p, osp.MODE_SAMPLED, 3, onv.ROUND_SR)
    for s_gpu, q in zip(sig, (xq, wq, dq)):
        assert np.max(np.abs(s_gpu - q.sigma) / q.sigma) < 1e-3
    for r_gpu, q in zip(rights, (xq, wq, dq)):
        # rank cut inside the bulk: single vectors are not unique to working precision, the spanned subspace is
        # (mean squared canonical correlation, the paper's subspace-alignment measure)
        from oracle import metrics
        align = metrics.subspace_alignment(q.right, r_gpu)
        print("subspace alignment of the right factors: %.6f" % align)
        assert align > 0.9999
    check_e2e(case[0], {"y": rel_fro(y_s, xq.dense_by_cols(rl) @ wq.dense_by_cols(rn).T),
                        "dx": rel_fro(dx_s, dq.dense_by_cols(rl) @ wq.dense_by_rows(cm)),
                        "dw": rel_fro(dw_s, dq.dense_by_rows(rn).T @ xq.dense_by_rows(cm))},
              list(zip(factors, (xq, wq, dq))) if k else [], TOL, cut_in_bulk=k > rank)

"""GPU test of metis_linear_fwd_static_ws, the forward layer for callers that cannot provide scratch memory
(a process whose pool already owns all device memory, a plug-in barred from allocating).  It must give the
same output as metis_linear_fwd, call after call, although every call reuses one built-in scratch array.

Collected last on purpose (file name): a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


def _operands(B, h, seed, l=256, n=320):
    dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
    x, _ = synth.planted(l, 384, 8, 300.0, 30.0, 1.0, seed)
    w, _ = synth.planted(n, 384, 8, 6.0, 0.6, 0.02, seed + 1)
    xo = h.split(dev(x), 8, 8, sketch=B.SKETCH_SAMPLED, seed=seed)
    wo = h.split(dev(w), 8, 8, sketch=B.SKETCH_FULL, seed=seed + 1)
    return xo, wo


def test_static_workspace_forward_matches_regular_forward_twice_in_a_row():
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    try:
        for call, seed in enumerate((61, 73)):          # two calls in a row, different data: the array is reused
            xo, wo = _operands(B, h, seed)
            want = h.linear_fwd(xo, wo)
            got = h.linear_fwd_static_ws(xo, wo)
            torch.cuda.synchronize()
            assert h.device_status() == 0
            assert torch.equal(got, want), "call %d differs from metis_linear_fwd" % call
            assert float(want.abs().max()) > 0
        # a layer below 256 rows takes the other internal route (FP32 staging of the main product inside the array)
        for call, seed in enumerate((81, 95)):
            xo, wo = _operands(B, h, seed, l=128, n=192)
            want = h.linear_fwd(xo, wo)
            got = h.linear_fwd_static_ws(xo, wo)
            torch.cuda.synchronize()
            assert torch.equal(got, want), "staged route, call %d differs from metis_linear_fwd" % call
        # the call itself takes no device memory: free memory is the same before and after (output supplied by the caller)
        xo, wo = _operands(B, h, 61)
        out = torch.empty((xo.rows, wo.rows), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        h.linear_fwd_static_ws(xo, wo, out=out)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
        # plain NVFP4 operands (k = 0) need no scratch at all and must work too
        dev = lambda a: torch.from_numpy(a).to(torch.bfloat16).cuda()
        c = synth.config_small()
        x0, w0 = h.split(dev(c["x"]), 0, 0), h.split(dev(c["w"]), 0, 0)
        assert torch.equal(h.linear_fwd_static_ws(x0, w0), h.linear_fwd(x0, w0))
        # a layer that needs more than the built-in array is refused, not truncated
        big_x, big_w = B.Operand(8192, 256, 64, axes=B.BLOCKS_ALONG_COLS), B.Operand(8192, 256, 64, axes=B.BLOCKS_ALONG_COLS)
        with pytest.raises(B.MetisError) as err:
            h.linear_fwd_static_ws(big_x, big_w)
        assert err.value.code == 4                       # METIS_ERR_WORKSPACE
    finally:
        h.close()

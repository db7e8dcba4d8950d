"""GPU test of the bounded-wait give-up path (failure detection without a fault): a wait on a barrier that nobody
completes must run out, report METIS_DEV_TIMEOUT through the status word and leave the context usable."""
import numpy as np
import pytest
import torch

from paper_2509_00404_b200 import synth

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_the_timeout_bit_and_the_next_call_is_clean():
    from gpu_util import to_dev_bf16
    from paper_2509_00404_b200 import binding as B
    h = B.Handle(0)
    try:
        assert h.device_status() == 0
        seen = h.wait_timeout(polls=256)
        torch.cuda.synchronize()                      # the kernel returned by itself
        s = seen.cpu().tolist()
        assert s[0] & 1, "the first warp's wait should have expired"
        assert s[0] & 2 and s[1] & 2, "both warps should have seen the give-up flag"
        assert s[1] & 1, "the second warp must stop waiting once the flag is up"
        st = h.device_status()
        assert st & B.DEV_TIMEOUT
        assert h.device_status() == 0                 # reading the word clears it
        # an ordinary call on the same handle afterwards: correct result, clean status
        c = synth.config_small()
        xo = h.split(to_dev_bf16(c["x"]), 4, 4, sketch=B.SKETCH_FULL, seed=1)
        wo = h.split(to_dev_bf16(c["w"]), 4, 4, sketch=B.SKETCH_FULL, seed=2)
        y = h.linear_fwd(xo, wo)
        torch.cuda.synchronize()
        assert h.device_status() == 0
        ref = c["x"].astype(np.float64) @ c["w"].astype(np.float64).T
        assert np.linalg.norm(y.cpu().numpy() - ref) / np.linalg.norm(ref) < 0.3
        with pytest.raises(B.MetisError):
            h.wait_timeout(polls=0)
    finally:
        h.close()

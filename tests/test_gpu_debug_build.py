"""GPU: the debug build of the library (METIS_DEBUG=1) - every store of codes and scales of the quantizing kernels is
checked against the extent of its buffer; a store that would fall outside is skipped and reported through the device
status word.  compute-sanitizer is not available, so this build is what stands in for it.  The library is loaded once
per process, so the debug library runs in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %(root)r); sys.path.insert(0, %(root)r + "/tests")
import numpy as np, torch
from oracle import nvfp4 as onv
from paper_2509_00404_b200 import binding as B, synth
from gpu_util import to_dev_bf16, nv_to_numpy
assert B.debug_build()
h = B.Handle(0)
# the check itself, on made-up stores: inside, touching the end, one byte over, negative
for off, n, ext, bad in ((0, 8, 64, False), (56, 8, 64, False), (57, 8, 64, True), (-1, 1, 64, True), (0, 16, 8, True)):
    h.index_check(off, n, ext)
    st = h.device_status()
    assert st == (B.DEV_INDEX if bad else 0), (off, n, ext, st)
assert h.device_status() == 0                                   # reading the word clears it
# the stand-alone quantizer on ragged shapes, both layouts and rounding modes: bit-exact and no store out of range
rng = np.random.default_rng(5)
for rows, cols, layout in ((336, 400, B.SF_LINEAR), (320, 448, B.SF_TILED), (128, 128, B.SF_TILED), (16, 16, B.SF_LINEAR)):
    x = synth.to_bf16_values((rng.standard_normal((rows, cols)) * 3).astype(np.float32))
    for rounding in (B.ROUND_RNE, B.ROUND_SR):
        bc, br = h.quantize_nvfp4(to_dev_bf16(x), B.BLOCKS_BOTH, rounding, seed=9, layout=layout)
        assert h.device_status() == 0
        for t, axis in ((bc, onv.AXIS_COLS), (br, onv.AXIS_ROWS)):
            c, s, ts = nv_to_numpy(t)
            oc, os_, ots = onv.quantize(x, axis, rounding, seed=9)
            assert ts == ots and np.array_equal(s, os_) and np.array_equal(c, oc)
# a split (fused residual + quantizer, whole tiles and ragged tiles) and the layer on top of it
for rows, cols, k in ((512, 768, 8), (320, 448, 8), (1024, 512, 80)):
    xs, _ = synth.llama_like(rows, cols, 1.0, 7, rank=16)
    a = h.split(to_dev_bf16(xs), k, 8, seed=3, rounding=B.ROUND_SR)
    assert h.device_status() == 0
x, _ = synth.llama_like(512, 768, 1.0, 11, rank=8); w, _ = synth.llama_like(640, 768, 0.02, 12, rank=8); d, _ = synth.llama_like(512, 640, 1e-4, 13, rank=8)
xo = h.split(to_dev_bf16(x), 8, 8, seed=1); wo = h.split(to_dev_bf16(w), 8, 8, sketch=B.SKETCH_FULL, seed=2); do = h.split(to_dev_bf16(d), 8, 8, seed=3, rounding=B.ROUND_SR)
y = h.linear_fwd(xo, wo); dx, dw = h.linear_bwd(do, xo, wo)
torch.cuda.synchronize()
assert h.device_status() == 0 and bool(torch.isfinite(y).all()) and bool(torch.isfinite(dx).all()) and bool(torch.isfinite(dw).all())
print("debug build ok")
"""


def test_debug_build_checks_every_output_store_and_finds_none_out_of_range():
    env = dict(os.environ, METIS_DEBUG="1")
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]

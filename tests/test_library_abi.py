"""CPU-side checks of the boundary: the library builds, loads and exports every symbol the header declares."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "metis.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(metis_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2509_00404_b200 import build, binding
    build.build()
    lib = binding.lib()
    names = _declared()
    assert "metis_split" in names and "metis_quantize_nvfp4" in names
    assert "metis_linear_fwd" in names and "metis_linear_bwd" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTED) == names
    # the debug build (index checks on every output store) is the same sources with one macro: same symbols
    import ctypes
    dbg = ctypes.CDLL(build.LIB_DEBUG)
    for n in names:
        assert hasattr(dbg, n), n
    dbg.metis_debug_build.restype = ctypes.c_int32
    lib.metis_debug_build.restype = ctypes.c_int32
    assert dbg.metis_debug_build() == 1 and lib.metis_debug_build() == 0


def test_host_only_helpers():
    from paper_2509_00404_b200 import binding as B
    from oracle import split as osp
    assert B.sf_bytes(128, 64, B.SF_TILED) == 512 and B.sf_bytes(129, 64, B.SF_TILED) == 1024
    assert B.sf_bytes(100, 160, B.SF_LINEAR) == 1000
    for rows, q in ((4096, 40), (16384, 40), (16384, 72), (128, 8), (200, 8)):
        assert B.default_sample_count(rows, q) == osp.default_sample_count(rows, q)
    assert B.workspace_bytes(1, 4096, 4096, 32, 8) > 0 and B.workspace_bytes(2, 4096, 4096, 32, 0) >= 4 * 4096 * 4096
    with pytest.raises(B.MetisError):
        B.workspace_bytes(9, 1, 1, 0, 0)


def test_no_cpu_path():
    import torch
    from paper_2509_00404_b200 import binding as B
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        B.Handle(0)


def test_tiled_scale_layout_helper_matches_the_header_formula():
    import numpy as np
    import torch
    from paper_2509_00404_b200 import binding as B
    rows, k_len = 256, 128
    nb = k_len // 16
    t = B.NvFp4.__new__(B.NvFp4)
    t.rows, t.k_len, t.layout = rows, k_len, B.SF_TILED
    raw = np.zeros(B.sf_bytes(rows, k_len, B.SF_TILED), dtype=np.uint8)
    for r in range(rows):
        for b in range(nb):
            off = ((r // 128) * (k_len // 64) + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
            raw[off] = (r * 7 + b * 3) % 251
    t.scales = torch.from_numpy(raw)
    lin = t.linear_scales().numpy()
    want = (np.arange(rows)[:, None] * 7 + np.arange(nb)[None, :] * 3) % 251
    assert np.array_equal(lin, want)


def test_launch_helpers_keep_no_process_wide_state():
    """Kernel attributes and occupancy figures belong to a device; a `static` flag or counter inside a launch helper
    would be shared by every device and thread of the process.  They live in the context (set in metis_create)."""
    csrc = os.path.join(ROOT, "paper_2509_00404_b200", "csrc")
    bad = []
    for name in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, name)).read()
        for i, line in enumerate(text.splitlines(), 1):
            if re.match(r"\s+static\s+(bool|int|unsigned|size_t|long)\b", line) and "(" not in line.split("=")[0]:
                bad.append("%s:%d: %s" % (name, i, line.strip()))
    assert not bad, bad

"""Helpers shared by the GPU parity tests: move tensors between the oracle's numpy world and the library."""
import numpy as np
import torch

from oracle import nvfp4 as onv


def to_dev_bf16(a):
    """float32 numpy array holding bf16-representable values -> cuda bfloat16 tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()


def nv_to_numpy(t):
    """NvFp4 device object -> (codes [rows, k_len] one per byte, scales [rows, k_len/16], tensor scale)."""
    packed = t.codes.cpu().numpy()
    return onv.unpack(packed), t.linear_scales().numpy(), np.float32(t.tensor_scale.item())


def nv_dequant(t):
    c, s, ts = nv_to_numpy(t)
    return onv.dequantize(c, s, ts)


def nv_from_numpy(binding, codes, scales, ts, layout=None):
    """Upload oracle-quantized (codes one per byte, linear scales, tensor scale) into an NvFp4 device object."""
    layout = binding.SF_TILED if layout is None else layout
    rows, k_len = codes.shape
    t = binding.NvFp4(rows, k_len, layout)
    t.codes.copy_(torch.from_numpy(onv.pack(codes)))
    nb = k_len // 16
    if layout == binding.SF_LINEAR:
        flat = torch.from_numpy(np.ascontiguousarray(scales)).reshape(-1)
        t.scales[: flat.numel()].copy_(flat)
    else:
        r = np.arange(rows).reshape(-1, 1)
        b = np.arange(nb).reshape(1, -1)
        off = ((r // 128) * (nb // 4) + b // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + b % 4
        host = np.zeros(t.scales.numel(), dtype=np.uint8)
        host[off] = scales
        t.scales.copy_(torch.from_numpy(host))
    t.tensor_scale.fill_(float(ts))
    return t


def rel_fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))

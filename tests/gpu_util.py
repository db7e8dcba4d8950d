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


def flip_allowance(pairs, gain=1.5, max_fraction=2e-3):
    """Extra tolerance for end-to-end comparisons, from the factor blocks that were rounded differently.

    An FP4 code is a discontinuous function of its FP32 input (Section 2.1: round to nearest on the E2M1 grid
    after dividing by the block scale and the tensor scale amax/2688).  The library's FP32 factors agree with
    the oracle's to a few 1e-7, so once in a while an entry that sits on a rounding midpoint, or a block maximum
    on a scale boundary, lands on the other side.  In the residual that moves one entry of bulk size and is
    covered by the base tolerance; in a factor the entry is multiplied by its singular value (one re-rounded
    code of a leading vector moved a layer output by 2e-3 of its norm, k = 12 on 512 x 768).

    The allowance is computed from the blocks that differ: a block of factor vector j whose dequantized values
    differ by delta changes the operand by sigma_j * |delta| in Frobenius norm; relative to |sigma| (the energy of
    the low-rank part, a lower bound of the operand's) these are summed over blocks and operands and multiplied by
    `gain` (sampled outputs are a noisier statistic than whole ones; measured errors stayed below the base
    tolerance plus 0.4 of the un-gained sum on every case of the suite).  The number
    of differing blocks itself must stay below max_fraction of all factor blocks (at least four are allowed;
    5e-4 of the blocks differ at k = 64 on 28672 x 8192, where neighbouring singular values are 3.7 % apart and
    the vectors themselves agree to ~3e-6 only): more than that is a failure, not rounding.

    pairs: (library operand, or its (left, right) factors already read with nv_to_numpy; oracle operand with
    .raw["left"] / .raw["right"] = (codes, scales, tensor scale), .sigma and .k)."""
    extra, differing, total = 0.0, 0, 0
    for op, q in pairs:
        if q.k == 0:
            continue
        left, right = op if isinstance(op, tuple) else (nv_to_numpy(op.left_q), nv_to_numpy(op.right_q))
        sig = np.asarray(q.sigma, dtype=np.float64)
        for (c, s, ts), name in ((left, "left"), (right, "right")):
            oc, os_, ots = q.raw[name]
            n = oc.shape[0]
            diff = (c[:n] != oc).reshape(n, -1, 16).any(axis=2) | (s[:n] != os_)
            total += diff.size
            differing += int(diff.sum())
            if diff.any():
                delta = onv.dequantize(c[:n], s[:n], ts) - onv.dequantize(oc, os_, ots)       # n x len
                per_vec = np.sqrt((delta.reshape(n, -1, 16) ** 2).sum(axis=2))                 # n x blocks
                extra += float((sig[:, None] * per_vec * diff).sum() / np.linalg.norm(sig))
    assert differing <= max(4, max_fraction * total), (differing, total)
    return gain * extra

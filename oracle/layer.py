"""Split-FP4 linear layer: forward (Eq. 2), input gradient (Eq. 3), weight gradient (Section 3.2).

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

Convention: X is l x m (tokens x in-features), W_t is n x m (out x in; the paper's W is W_t^T),
D = dL/dY is l x n.  Y = X W_t^T, dX = D W_t, dW_t = D^T X.

Every operand T is represented as  Tq = Lq diag(sigma) Rq^T + Resq  where Lq, Rq, Resq are NVFP4
tensors and sigma stays in high precision (the paper quantizes every matrix of Eq. 1 except the
singular values).  Each tall-skinny factor is quantized once with blocks along its long
dimension.  Block-scaled hardware needs the 16-element blocks to lie along the contraction axis
of the product that consumes the tensor, and a quantized tensor cannot be transposed, so the
residual is quantized separately for each contraction axis it is used with:

    forward  contracts over m:  X by columns, W_t by columns
    dgrad    contracts over n:  D by columns, W_t by rows
    wgrad    contracts over l:  D by rows,    X by rows

All products are evaluated literally in float64 from the dequantized tensors.
"""
from dataclasses import dataclass

import numpy as np

from . import nvfp4, philox
from . import split as split_mod


@dataclass
class QOperand:
    """Dequantized pieces of one split + quantized operand, float64, in the operand's own orientation."""
    k: int
    left_q: np.ndarray          # rows x k
    sigma: np.ndarray           # k
    right_q: np.ndarray         # cols x k
    res_by_cols: np.ndarray     # rows x cols, blocks along columns
    res_by_rows: np.ndarray     # rows x cols, blocks along rows
    split: split_mod.Split
    raw: dict                   # codes / scales / tensor scales of every quantized piece (K-major storage)

    def dense(self, residual_axis):
        res = self.res_by_cols if residual_axis == nvfp4.AXIS_COLS else self.res_by_rows
        if self.k == 0:
            return res
        return (self.left_q * self.sigma) @ self.right_q.T + res


def quantize_operand(x, k, p, mode, seed, rounding=nvfp4.ROUND_RNE):
    """Split x (float32 array holding the bf16 input values) and quantize every piece.

    The residual's tensor scale is the *source* tensor's amax/2688 (not the residual's own), so a
    fused single pass can quantize the residual without a second reduction; factors use their own amax.
    """
    x32 = np.asarray(x, dtype=np.float32)
    sp = split_mod.split(x32.astype(np.float64), k, p, mode=mode, seed=seed)
    s_src = nvfp4.tensor_scale_from_amax(np.max(np.abs(x32)))
    res32 = sp.residual.astype(np.float32)
    raw = {}
    rc = nvfp4.quantize(res32, nvfp4.AXIS_COLS, rounding, seed, philox.STREAM_RESIDUAL, tensor_scale=s_src)
    rr = nvfp4.quantize(res32, nvfp4.AXIS_ROWS, rounding, seed, philox.STREAM_RESIDUAL, tensor_scale=s_src)
    raw["res_by_cols"], raw["res_by_rows"] = rc, rr
    res_c = nvfp4.dequantize(*rc)
    res_r = nvfp4.dequantize(*rr).T
    if k:
        # factors are held transposed (k x rows, k x cols: one factor vector per stored row), so their
        # blocks of 16 run along the long dimension and the draw of element (j, i) is keyed by j*len + i
        lq = nvfp4.quantize(np.ascontiguousarray(sp.left.T).astype(np.float32), nvfp4.AXIS_COLS, rounding, seed,
                            philox.STREAM_LEFT)
        rq = nvfp4.quantize(np.ascontiguousarray(sp.right.T).astype(np.float32), nvfp4.AXIS_COLS, rounding, seed,
                            philox.STREAM_RIGHT)
        raw["left"], raw["right"] = lq, rq
        left_q, right_q = nvfp4.dequantize(*lq).T, nvfp4.dequantize(*rq).T
    else:
        left_q = np.zeros((x32.shape[0], 0))
        right_q = np.zeros((x32.shape[1], 0))
    return QOperand(k, left_q, sp.sigma, right_q, res_c, res_r, sp, raw)


def requantize_operand(left, sigma, right, residual, rounding=nvfp4.ROUND_RNE, seed=0, residual_scale=None):
    """NVFP4 forms of an operand that is HELD as separately stored pieces (Section 3.2 keeps a weight as U, S, V and
    W_R, which training updates; per step they are only quantized again, never decomposed again).

    left (rows x k), right (cols x k), residual (rows x cols) are the stored float32 values.  Every piece is
    quantized on its own: the factors exactly as quantize_operand does it, the residual in both block orientations
    with its OWN amax/2688 as tensor scale (there is no source tensor here) unless residual_scale is given."""
    res32 = np.asarray(residual, dtype=np.float32)
    k = int(np.asarray(sigma).shape[0])
    rc = nvfp4.quantize(res32, nvfp4.AXIS_COLS, rounding, seed, philox.STREAM_RESIDUAL, tensor_scale=residual_scale)
    rr = nvfp4.quantize(res32, nvfp4.AXIS_ROWS, rounding, seed, philox.STREAM_RESIDUAL, tensor_scale=residual_scale)
    raw = {"res_by_cols": rc, "res_by_rows": rr}
    if k:
        lq = nvfp4.quantize(np.ascontiguousarray(np.asarray(left, dtype=np.float32).T), nvfp4.AXIS_COLS, rounding, seed, philox.STREAM_LEFT)
        rq = nvfp4.quantize(np.ascontiguousarray(np.asarray(right, dtype=np.float32).T), nvfp4.AXIS_COLS, rounding, seed, philox.STREAM_RIGHT)
        raw["left"], raw["right"] = lq, rq
        left_q, right_q = nvfp4.dequantize(*lq).T, nvfp4.dequantize(*rq).T
    else:
        left_q, right_q = np.zeros((res32.shape[0], 0)), np.zeros((res32.shape[1], 0))
    sp = split_mod.Split(np.asarray(left, dtype=np.float64), np.asarray(sigma, dtype=np.float64), np.asarray(right, dtype=np.float64),
                         res32.astype(np.float64))
    return QOperand(k, left_q, np.asarray(sigma, dtype=np.float64), right_q, nvfp4.dequantize(*rc), nvfp4.dequantize(*rr).T, sp, raw)


def linear_fwd(xq, wq):
    """Eq. 2: Y^ = Xq Wq^T, both residuals quantized along the in-feature axis."""
    return xq.dense(nvfp4.AXIS_COLS) @ wq.dense(nvfp4.AXIS_COLS).T


def linear_dgrad(dq, wq):
    """Eq. 3: dX^ = Dq Wq', contraction over out-features (D by columns, W_t by rows)."""
    return dq.dense(nvfp4.AXIS_COLS) @ wq.dense(nvfp4.AXIS_ROWS)


def linear_wgrad(dq, xq):
    """dW_t^ = Dq''^T Xq'', contraction over tokens (both residuals quantized by rows)."""
    return dq.dense(nvfp4.AXIS_ROWS).T @ xq.dense(nvfp4.AXIS_ROWS)


def factor_grads(dw_t, wq):
    """Gradients of the weight factors from the paper-orientation weight gradient dW = dW_t^T (m x n).

    W = U S V^T with U = wq.right_q (m x k), V = wq.left_q (n x k):
    dU = dW V S, dS = diag(U^T dW V), dV = dW^T U S.
    """
    dw = dw_t.T
    u, v, s = wq.right_q, wq.left_q, wq.sigma
    return (dw @ v) * s, np.einsum("ik,ij,jk->k", u, dw, v), (dw.T @ u) * s

"""Oracle pieces for outputs sampled from a large layer (test infrastructure).

The split of an operand is taken on the whole matrix, as the oracle defines it; only the NVFP4 encoding of the
residual - the expensive part in numpy - is restricted to the rows or columns that the sampled outputs read.
Blocks along the columns make every row independent and blocks along the rows every column, and the
stochastic-rounding draws are keyed by the element's index in the whole tensor, so the sliced encoding is
exactly the slice of the full one (pinned by a CPU test of the oracle's `index` argument)."""
import numpy as np

from oracle import nvfp4 as onv, philox, split as osp


class PartialOperand:
    def __init__(self, x, k, p, mode, seed, rounding=onv.ROUND_RNE):
        x32 = np.asarray(x, dtype=np.float32)
        self.rows, self.cols = x32.shape
        self.k, self.seed, self.rounding = k, seed, rounding
        self.s_src = onv.tensor_scale_from_amax(np.max(np.abs(x32)))
        if k:
            sp = osp.split(x32.astype(np.float64), k, p, mode=mode, seed=seed)
            self.sigma = sp.sigma
            self.right = sp.right
            self.res = sp.residual.astype(np.float32)
            lq = onv.quantize(np.ascontiguousarray(sp.left.T).astype(np.float32), onv.AXIS_COLS, rounding, seed, philox.STREAM_LEFT)
            rq = onv.quantize(np.ascontiguousarray(sp.right.T).astype(np.float32), onv.AXIS_COLS, rounding, seed, philox.STREAM_RIGHT)
            self.left_q, self.right_q = onv.dequantize(*lq).T, onv.dequantize(*rq).T
            self.raw = {"left": lq, "right": rq}
        else:
            self.sigma = np.zeros(0)
            self.res = x32
            self.left_q, self.right_q = np.zeros((self.rows, 0)), np.zeros((self.cols, 0))

    def low(self, rows=slice(None), cols=slice(None)):
        return (self.left_q[rows] * self.sigma) @ self.right_q[cols].T

    def dense_by_cols(self, rows):
        """Rows `rows` of the dequantized operand whose residual has its blocks along the columns."""
        rows = np.asarray(rows)
        idx = rows[:, None].astype(np.uint64) * np.uint64(self.cols) + np.arange(self.cols, dtype=np.uint64)[None, :]
        q = onv.quantize(self.res[rows], onv.AXIS_COLS, self.rounding, self.seed, philox.STREAM_RESIDUAL,
                         tensor_scale=self.s_src, index=idx)
        return self.low(rows) + onv.dequantize(*q)

    def dense_by_rows(self, cols):
        """Columns `cols` of the dequantized operand whose residual has its blocks along the rows."""
        cols = np.asarray(cols)
        idx = np.arange(self.rows, dtype=np.uint64)[:, None] * np.uint64(self.cols) + cols[None, :].astype(np.uint64)
        q = onv.quantize(self.res[:, cols], onv.AXIS_ROWS, self.rounding, self.seed, philox.STREAM_RESIDUAL,
                         tensor_scale=self.s_src, index=idx)
        return self.low(slice(None), cols) + onv.dequantize(*q).T

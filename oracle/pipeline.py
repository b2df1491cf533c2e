"""The hot path end to end, step by step (Algorithm 2 RTN case + Eq. 7).

Test infrastructure (see the package docstring).  Layout bridge: the paper uses
column vectors, X in R^{d_in x d_batch}, W in R^{d_in x d_out}, output W^T X.
Here arrays are row-major X[M, K], W[N, K], Y[M, N] = X W^T with M = d_batch,
K = d_in, N = d_out, g = d, C = K / g.  The paper's T_(i) x on a column block is
x_row_block @ T_(i)^T:  v[m, c*g + j] = sum_k T[c, j, k] * x[m, c*g + k].
"""
import numpy as np

from . import formats as F
from . import quantizers as Q
from . import wush_transform as WT

F32 = np.float32


def second_moment_sums(Xv, g):
    """Unnormalised per-block second moments  S_c = sum_t x_{t,c}^T x_{t,c}  ([C, g, g]).

    Algorithm 2 divides by the number of rows (d_batch or d_out) afterwards.
    """
    Xv = np.asarray(Xv, dtype=np.float64)
    B, K = Xv.shape
    xb = Xv.reshape(B, K // g, g)
    # batched matrix product over blocks: S_c = X_c^T X_c with X_c = Xv[:, c*g:(c+1)*g]
    return np.matmul(xb.transpose(1, 2, 0), xb.transpose(1, 0, 2))


def transform_blocks(Xv, T):
    """v = x_blk @ T_c^T for every row and block, in fp64.  Xv [M, K], T [C, g, g]."""
    Xv = np.asarray(Xv, dtype=np.float64)
    C, g, _ = T.shape
    xb = Xv.reshape(Xv.shape[0], C, g)
    # per block c: V_c = X_c @ T_c^T   (V_c[m, j] = sum_k T[c, j, k] X_c[m, k])
    vb = np.matmul(xb.transpose(1, 0, 2), np.asarray(T, dtype=np.float64).transpose(0, 2, 1))
    return np.ascontiguousarray(vb.transpose(1, 0, 2)).reshape(Xv.shape)


def quantize_transformed(Xv, T, fmt, ts=None):
    """q(T x): transform in fp64, round once to fp32, quantise.  Returns (v32, codes, scales)."""
    v32 = transform_blocks(Xv, T).astype(F32)
    codes, scales = Q.quantize(v32, fmt, ts)
    return v32, codes, scales


def dequantized_product(xd, wd):
    """Y[m, n] = sum_k xd[m, k] * wd[n, k] in fp64 (Eq. 7 on dequantised values)."""
    return np.asarray(xd, dtype=np.float64) @ np.asarray(wd, dtype=np.float64).T


class PreparedLayer:
    """Everything Algorithm 2 (RTN case) produces offline for one linear layer."""

    def __init__(self, W_bits, Xc_bits, fmt, lam=0.01):
        self.fmt = fmt
        self.g = g = Q.GROUP[fmt]
        Wv = F.bf16_bits_to_f64(W_bits)
        Xc = F.bf16_bits_to_f64(Xc_bits)
        self.N, self.K = Wv.shape
        self.mom_W = second_moment_sums(Wv, g) / Wv.shape[0]
        self.mom_X = second_moment_sums(Xc, g) / Xc.shape[0]
        self.T_bits, self.T_hat, T_xvsh = WT.build_transforms(self.mom_W, self.mom_X, lam)
        # the GPU library receives the weight-side transform as fp32
        self.T_xvsh32 = np.ascontiguousarray(T_xvsh, dtype=F32)
        wbar = transform_blocks(Wv, self.T_xvsh32.astype(np.float64))
        self.wbar32 = wbar.astype(F32)
        if fmt == "nvfp4":
            self.ts_w = Q.nvfp4_tensor_scale(self.wbar32)
            vcal = transform_blocks(Xc, self.T_hat).astype(F32)
            self.ts_x = Q.nvfp4_tensor_scale(vcal)      # static, from calibration tokens
        else:
            self.ts_w = None
            self.ts_x = None
        self.w_codes, self.w_scales = Q.quantize(self.wbar32, fmt, self.ts_w)
        self.w_deq = Q.dequantize(self.w_codes, self.w_scales, fmt, self.ts_w)

    def dynamic_ts_x(self, X_bits):
        """NVFP4 tensor scale of THIS batch of activations (instead of the static calibration one):
        AbsMax over all transformed tokens / (6 * 448)."""
        v32 = transform_blocks(F.bf16_bits_to_f64(X_bits), self.T_hat).astype(F32)
        return Q.nvfp4_tensor_scale(v32)

    def quantize_act(self, X_bits, ts_x=None):
        """(v32, codes, scales) of q(T x); ``ts_x`` overrides the static NVFP4 tensor scale."""
        Xv = F.bf16_bits_to_f64(X_bits)
        return quantize_transformed(Xv, self.T_hat, self.fmt, self.ts_x if ts_x is None else ts_x)

    def forward(self, X_bits, rows=None, dynamic=False):
        """Eq. 7.  ``rows`` optionally restricts the output to a subset of tokens; ``dynamic``
        takes the NVFP4 activation tensor scale from the whole batch X_bits."""
        ts_x = self.dynamic_ts_x(X_bits) if dynamic else self.ts_x
        if rows is not None:
            X_bits = np.asarray(X_bits)[rows]
        _, codes, scales = self.quantize_act(X_bits, ts_x)
        xd = Q.dequantize(codes, scales, self.fmt, ts_x)
        return dequantized_product(xd, self.w_deq)

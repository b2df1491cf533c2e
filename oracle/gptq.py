"""Algorithm 2, GPTQ case: WUSH transforms interleaved with GPTQ error propagation.

Test infrastructure (see the package docstring).  The steps below are the steps of the
"GPTQ case" of Algorithm 2 ("Compute WUSH and Pre-Quantize Weights") in the paper's order
and, inside ``wush_gptq_layer``, in the paper's own orientation: column vectors,
W in R^{d_in x d_out} (row k = input channel k), X in R^{d_in x d_batch}; block (i) is rows
i*d .. (i+1)*d - 1.  The repository's row-major arrays W[N, K] = W_paper^T are transposed
on the way in and out.

Readings where the paper is silent (all of them conventions of this build, "parity
unpinned" as far as the authors' own choice goes):
  * "standard GPTQ subroutine (intra-block error propagation)": the quantisation group of
    the formats here is exactly one block (d consecutive input channels of one output
    channel), so the subroutine fixes the group's scale from the block's CURRENT values when
    it reaches the block (GPTQ's usual non-static groups), then walks the d transformed
    coordinates in order: round coordinate q to the E2M1 grid under that scale, spread the
    error over coordinates q+1.. of the same block through the lower Cholesky factor of the
    inverse of the block's (transformed) Hessian.
  * the quantiser q is the one of ``quantizers.py`` (fp32 inputs): the block is rounded to
    fp32 before its AbsMax is taken, and each coordinate is rounded to fp32 before it is
    converted, so the same definition serves the RTN and the GPTQ case.
  * NVFP4 needs the tensor scale before the first block is quantised, while the weights
    still change: it is an input (default: the RTN case's value for the same layer).
  * storage: as in the RTN case the activation-side transform is rounded to bf16 and every
    later step (T_xvsh, the transformed weights, the transformed Hessian, the error in the
    original space) uses the ROUNDED values, because those are what runs online; T_xvsh is
    the inverse-transpose of the rounded transform, kept as fp32 like in the RTN case, and the
    error in the original space uses T_wush^T for T_xvsh^-1 (Eq. 6).
  * damping: the same ratio lambda in the Hessian's damping and in Algorithm 1.
"""
import numpy as np

from . import formats as F
from . import quantizers as Q
from . import wush_transform as WT

F32 = np.float32


def hessian(Xc):
    """GPTQ's Hessian  d_batch^-1 X X^T  (d_in x d_in) from calibration rows Xc[B, K] (= X^T)."""
    Xc = np.asarray(Xc, dtype=np.float64)
    return Xc.T @ Xc / Xc.shape[0]


def inverse_hessian_cholesky(H, lam):
    """L lower triangular with  L L^T = (H + lam * d_in^-1 tr(H) I)^-1."""
    d_in = H.shape[0]
    Hd = H + lam * np.trace(H) / d_in * np.eye(d_in)
    return np.linalg.cholesky(np.linalg.inv(Hd))


def block_scale(wbar_block, fmt, ts=None):
    """Scale of one quantisation group per output channel, from the block's current values.

    wbar_block: [d, d_out] (transformed coordinates x output channels).  Returns
    (scale bytes uint8 [d_out], multiplier fp64 [d_out], dequantisation scale fp64 [d_out]):
    code = E2M1(value * multiplier), value_hat = grid[code] * scale.
    """
    a = np.max(np.abs(wbar_block.astype(F32)), axis=0).astype(np.float64)
    if fmt in ("mxfp4", "mxfp4_ceil"):
        e = Q.mx_shared_exponent(a, "floor" if fmt == "mxfp4" else "ceil")
        return (e + 127).astype(np.uint8), np.ldexp(1.0, -e), np.ldexp(1.0, e)
    if fmt == "nvfp4":
        ts = F32(ts)
        with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
            r = ((a.astype(F32) / F32(6.0)).astype(F32) / ts).astype(F32)
            sb = F.e4m3_encode_satfinite(r.astype(np.float64))
            d32 = (F.e4m3_decode(sb).astype(F32) * ts).astype(F32)      # the quantiser's divisor: one fp32 rounding
            inv = np.where(d32 == 0, F32(0), F32(1.0) / d32).astype(F32)
        # what a code stands for is grid * scale byte * tensor scale without that rounding (the GEMM's arithmetic)
        return sb, inv.astype(np.float64), F.e4m3_decode(sb) * float(ts)
    raise ValueError(fmt)


def gptq_block(wbar, Hbar, fmt, ts=None, propagate=True):
    """The GPTQ subroutine on one transformed block.

    wbar [d, d_out]: transformed weights (row q = transformed coordinate q); Hbar [d, d]: the
    block's Hessian in the transformed basis.  Returns (codes uint8 [d, d_out],
    scale bytes uint8 [d_out], dequantised values fp64 [d, d_out]).

    With Lb the lower Cholesky factor of Hbar^-1, coordinate q is rounded and its error,
    divided by Lb[q, q], is subtracted from the later coordinates r > q with weight Lb[r, q].
    propagate=False skips the spreading (plain RTN under the same scale) - used only to pin
    the reduction to the RTN case.
    """
    wcur = np.array(wbar, dtype=np.float64)
    d = wcur.shape[0]
    Lb = np.linalg.cholesky(np.linalg.inv(Hbar))
    sbytes, mult, dq = block_scale(wcur, fmt, ts)
    codes = np.zeros(wcur.shape, dtype=np.uint8)
    what = np.zeros_like(wcur)
    for q in range(d):
        w32 = wcur[q].astype(F32)
        if fmt == "nvfp4":                               # one fp32 multiplication, as in the quantiser
            u = (w32 * mult.astype(F32)).astype(F32).astype(np.float64)
            u = np.where(dq == 0, np.copysign(0.0, w32), u)
        else:
            u = w32.astype(np.float64) * mult            # exact power-of-two scaling
        codes[q] = F.e2m1_encode(u)
        what[q] = F.e2m1_decode(codes[q]) * dq
        if propagate and q + 1 < d:
            err = (wcur[q] - what[q]) / Lb[q, q]
            wcur[q + 1:] -= np.outer(Lb[q + 1:, q], err)
    return codes, sbytes, what


def propagate_error(Wp, L, i, d, E):
    """Inter-block step of Algorithm 2:  W_(j) <- W_(j) + L_(j,i) L_(i,i)^-1 E_(i)  for j = i .. d_in/d.

    Wp [d_in, d_out] is updated in place; L [d_in, d_in] lower; E [d, d_out] is the error of
    block i in the original space (dequantised minus current).  The paper's loop includes
    j = i, which turns block i itself into its dequantised value.
    """
    Lii = L[i * d:(i + 1) * d, i * d:(i + 1) * d]
    Z = np.linalg.solve(Lii, E)                          # L_(i,i)^-1 E_(i)
    Wp[i * d:] += L[i * d:, i * d:(i + 1) * d] @ Z
    return Wp


def wush_gptq_layer(W_bits, Xc_bits, fmt, lam=0.01, ts_w=None, intra=True, stored_T=None):
    """Algorithm 2, GPTQ case, for one layer.  W_bits [N, K], Xc_bits [B, K] as bf16 bit patterns.

    Returns a dict: T_bits uint16 [C,d,d] (bf16 storage of T_wush), T_hat fp64 [C,d,d],
    T_xvsh fp64 [C,d,d], codes uint8 [N, K] (unpacked), scales uint8 [N, C], w_deq fp64 [N, K]
    (dequantised transformed weights, the GEMM operand), W_hat fp64 [N, K] (the quantised layer
    back in the original space: block i is T_xvsh(i)^-1 W~(i)), ts_w, T_wush fp64 [C,d,d] (Algorithm 1's result
    before the 16-bit rounding).

    stored_T: optional {block index: uint16 [d,d]} - use these stored transforms for the listed blocks instead
    of rounding Algorithm 1's result (which is still computed and returned in T_wush).  An entry of T_wush that
    sits on a bf16 rounding boundary can legitimately be stored either way, and every later block depends on the
    choice; a comparison with another implementation fixes the choice this way and checks everything else.
    """
    d = Q.GROUP[fmt]
    Wp = F.bf16_bits_to_f64(W_bits).T.copy()             # paper orientation [d_in, d_out]
    Xc = F.bf16_bits_to_f64(Xc_bits)
    d_in, d_out = Wp.shape
    C = d_in // d
    if fmt == "nvfp4" and ts_w is None:
        raise ValueError("NVFP4 needs the weight tensor scale up front")
    Hs = hessian(Xc)                                     # GPTQ's Hessian
    M_X = [Hs[i * d:(i + 1) * d, i * d:(i + 1) * d] for i in range(C)]     # its diagonal blocks
    L = inverse_hessian_cholesky(Hs, lam)                # Cholesky of the damped Hessian's inverse
    T_bits = np.zeros((C, d, d), dtype=np.uint16)
    T_hat = np.zeros((C, d, d))
    T_wush = np.zeros((C, d, d))
    T_xvsh = np.zeros((C, d, d))
    codes = np.zeros((d_in, d_out), dtype=np.uint8)
    scales = np.zeros((C, d_out), dtype=np.uint8)
    w_deq = np.zeros((d_in, d_out))
    W_hat = np.zeros((d_in, d_out))
    for i in range(C):
        blk = slice(i * d, (i + 1) * d)
        Wi = Wp[blk]                                     # current (updated) weight block
        M_W = Wi @ Wi.T / d_out                          # second moment of the updated block
        T_wush[i] = WT.wush_block(M_W, M_X[i], lam)      # Algorithm 1
        T_bits[i] = F.f64_to_bf16_bits(T_wush[i])        # stored in 16 bits
        if stored_T is not None and i in stored_T:
            T_bits[i] = np.asarray(stored_T[i], dtype=np.uint16)
        T_hat[i] = F.bf16_bits_to_f64(T_bits[i])
        T_xvsh[i] = WT.xvsh_from_wush(T_hat[i]).astype(F32)                # Eq. 6; handed on as fp32, as in the RTN case
        wbar = T_xvsh[i] @ Wi                            # transformed weights
        Lii = L[blk, blk]
        Hbar = T_hat[i] @ np.linalg.inv(Lii @ Lii.T) @ T_hat[i].T          # transformed Hessian
        c, sb, wq = gptq_block(wbar, Hbar, fmt, ts_w, propagate=intra)     # intra-block error propagation
        codes[blk], scales[i], w_deq[blk] = c, sb, wq
        W_hat[blk] = T_hat[i].T @ wq                     # T_xvsh^-1 = T_wush^T: the weights the online layer realises
        E = W_hat[blk] - Wi                              # error in the original space
        propagate_error(Wp, L, i, d, E)                  # inter-block error propagation
    return dict(T_bits=T_bits, T_hat=T_hat, T_xvsh=T_xvsh, codes=codes.T.copy(), scales=scales.T.copy(),
                w_deq=w_deq.T.copy(), W_hat=W_hat.T.copy(), ts_w=ts_w, T_wush=T_wush)


def proxy_loss(W_hat, W, Hs):
    """Layer-wise output error  tr((W_hat - W) H (W_hat - W)^T)  for row-major [N, K] weights."""
    D = np.asarray(W_hat, dtype=np.float64) - np.asarray(W, dtype=np.float64)
    return float(np.sum((D @ Hs) * D))

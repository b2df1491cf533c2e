"""Pins for the oracle's GPTQ case of Algorithm 2 (CPU only).

Nothing here re-types the oracle's formulas.  The pins are:
  * the Cholesky factor against its defining identity;
  * one inter-block propagation step in exact rational arithmetic;
  * the intra-block subroutine against the greedy optimal-brain-quantisation rule it is a fast form
    of: the value a coordinate has when its turn comes is the exact minimiser of the quadratic loss
    over the still-free coordinates, computed here from the Hessian itself by a linear solve (no
    inverse, no Cholesky factor, no triangular indexing);
  * the whole layer against the same closed form across blocks (what block i looks like when its
    turn comes follows from the damped Hessian and the already-quantised blocks alone);
  * reduction to the RTN case (already pinned) when the Hessian is block diagonal and the
    intra-block spreading is off;
  * the proxy loss against the RTN case on seeded correlated activations.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import formats as F
from oracle import gptq as G
from oracle import pipeline as P
from oracle import quantizers as Q
from oracle import wush_transform as WT
from paper_2512_00956_b200 import synth


def _correlated_layer(seed, N, K, B):
    return synth.correlated_layer(seed, N, K, B)


def test_inverse_hessian_cholesky_identity():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((200, 24))
    H = G.hessian(X)
    assert np.allclose(H, sum(np.outer(x, x) for x in X) / 200, rtol=1e-12)
    lam = 0.01
    L = G.inverse_hessian_cholesky(H, lam)
    assert np.allclose(L, np.tril(L)) and np.all(np.diag(L) > 0)
    Hd = H + lam * np.trace(H) / 24 * np.eye(24)
    assert np.allclose(L @ L.T @ Hd, np.eye(24), atol=1e-10)


def test_propagate_error_exact_rational():
    """W_(j) <- W_(j) + L_(j,i) L_(i,i)^-1 E_(i) for j >= i, with small integers so that fractions are exact."""
    d, C, d_out, i = 2, 3, 2, 1
    rng = np.random.default_rng(3)
    Lr = [[Fraction(int(rng.integers(-3, 4))) if c < r else (Fraction(int(rng.integers(1, 4))) if c == r else Fraction(0))
           for c in range(d * C)] for r in range(d * C)]
    Wr = [[Fraction(int(rng.integers(-8, 9)), 4) for _ in range(d_out)] for _ in range(d * C)]
    Er = [[Fraction(int(rng.integers(-8, 9)), 8) for _ in range(d_out)] for _ in range(d)]
    # L_(i,i)^-1 E by forward substitution in rationals
    Z = [[Fraction(0)] * d_out for _ in range(d)]
    for r in range(d):
        for n in range(d_out):
            acc = Er[r][n] - sum(Lr[i * d + r][i * d + c] * Z[c][n] for c in range(r))
            Z[r][n] = acc / Lr[i * d + r][i * d + r]
    want = [row[:] for row in Wr]
    for r in range(i * d, d * C):                          # every row of blocks j >= i
        for n in range(d_out):
            want[r][n] += sum(Lr[r][i * d + c] * Z[c][n] for c in range(d))
    Wf = np.array([[float(v) for v in row] for row in Wr])
    got = G.propagate_error(Wf.copy(), np.array([[float(v) for v in row] for row in Lr]), i, d,
                            np.array([[float(v) for v in row] for row in Er]))
    assert np.allclose(got, np.array([[float(v) for v in row] for row in want]), rtol=0, atol=1e-13)
    assert np.array_equal(got[:i * d], Wf[:i * d])         # earlier blocks are never touched
    # j = i: the block itself becomes current + E (its dequantised value)
    assert np.allclose(got[i * d:(i + 1) * d], Wf[i * d:(i + 1) * d] + np.array([[float(v) for v in row] for row in Er]), atol=1e-13)


def _greedy_obq_reference(wbar, Hbar, fmt, ts):
    """Coordinate q's value when its turn comes = argmin over the free coordinates of the quadratic loss with
    the already-rounded ones fixed: v = w_free - H_ff^-1 H_fq_done (what_done - w_done); then round v[0]."""
    d, n = wbar.shape
    sb, mult, dq = G.block_scale(wbar, fmt, ts)
    what = np.zeros_like(wbar)
    codes = np.zeros(wbar.shape, dtype=np.uint8)
    seen = np.zeros_like(wbar)
    for q in range(d):
        if q == 0:
            v = wbar[0]
        else:
            delta = what[:q] - wbar[:q]                                           # [q, n]
            v = (wbar[q:] - np.linalg.solve(Hbar[q:, q:], Hbar[q:, :q] @ delta))[0]
        seen[q] = v
        codes[q], _ = _rtn_row(v, mult, dq, fmt)
        what[q] = F.e2m1_decode(codes[q]) * dq
    return codes, what, seen


def _rtn_row(v, mult, dq, fmt):
    v32 = v.astype(np.float32)
    if fmt == "nvfp4":
        u = (v32 * mult.astype(np.float32)).astype(np.float32).astype(np.float64)
    else:
        u = v32.astype(np.float64) * mult
    return F.e2m1_encode(u), u


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_gptq_block_is_greedy_optimal_brain_quantisation(fmt):
    d = Q.GROUP[fmt]
    rng = np.random.default_rng(10 + d)
    A = rng.standard_normal((3 * d, d)) @ np.diag(np.exp(rng.standard_normal(d))) @ rng.standard_normal((d, d))
    Hbar = A.T @ A / (3 * d) + 0.05 * np.eye(d)
    wbar = rng.standard_normal((d, 300)) * np.exp(rng.standard_normal((1, 300)))
    ts = np.float32(np.max(np.abs(wbar)) / 2688.0) if fmt == "nvfp4" else None
    codes, sb, what = G.gptq_block(wbar, Hbar, fmt, ts)
    rcodes, rwhat, _ = _greedy_obq_reference(wbar, Hbar, fmt, ts)
    # two mathematically equal routes: codes may differ only where a value sits on a rounding boundary to ~1e-12,
    # and such a flip would change everything after it in that column - so compare column by column
    same_cols = np.all(codes == rcodes, axis=0)
    assert same_cols.mean() >= 0.99
    assert np.allclose(what[:, same_cols], rwhat[:, same_cols], rtol=0, atol=1e-12 * np.max(np.abs(wbar)))
    # and the spreading does what it is for: lower quadratic loss than plain rounding under the same scales
    _, _, w_rtn = G.gptq_block(wbar, Hbar, fmt, ts, propagate=False)
    loss = lambda wh: float(np.sum((wh - wbar) * (Hbar @ (wh - wbar))))
    assert loss(what) < 0.9 * loss(w_rtn)
    # first coordinate: nothing has been spread yet, so it is plain RTN of the input
    assert np.array_equal(codes[0], Q.quantize(wbar.T.astype(np.float32), fmt, ts)[0][:, 0])


def test_gptq_block_without_spreading_is_the_block_quantiser():
    """propagate=False must be q(.) of quantizers.py bit for bit (same scale rule, same rounding)."""
    rng = np.random.default_rng(5)
    for fmt in ("mxfp4", "mxfp4_ceil", "nvfp4"):
        d = Q.GROUP[fmt]
        wbar = (rng.standard_normal((d, 257)) * np.exp(3 * rng.standard_normal((1, 257)))).astype(np.float32).astype(np.float64)
        ts = Q.nvfp4_tensor_scale(wbar.astype(np.float32)) if fmt == "nvfp4" else None
        codes, sb, what = G.gptq_block(wbar, np.eye(d), fmt, ts, propagate=False)
        c0, s0 = Q.quantize(wbar.T.astype(np.float32), fmt, ts)                   # rows = output channels, one group each
        assert np.array_equal(codes.T, c0) and np.array_equal(sb, s0[:, 0])
        assert np.array_equal(what.T, Q.dequantize(c0, s0, fmt, ts))
        # identity Hessian: the Cholesky factor is diagonal, so spreading changes nothing either
        codes2, _, _ = G.gptq_block(wbar, np.eye(d), fmt, ts, propagate=True)
        assert np.array_equal(codes2, codes)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_layer_matches_closed_form_compensation_across_blocks(fmt):
    """When block i's turn comes, the current weights of blocks >= i are the original ones plus the optimal
    continuous compensation for the error committed in blocks < i under the damped Hessian.  Rebuild every
    block's input that way (linear solve with the Hessian itself), redo its transform and its subroutine, and
    compare with what the layer routine produced."""
    d = Q.GROUP[fmt]
    N, K, B, lam = 48, 4 * d, 400, 0.01
    W_bits, Xc_bits = _correlated_layer(21, N, K, B)
    Wv = F.bf16_bits_to_f64(W_bits)
    ts_w = np.float32(0.001) if fmt == "nvfp4" else None
    out = G.wush_gptq_layer(W_bits, Xc_bits, fmt, lam, ts_w)
    Hs = G.hessian(F.bf16_bits_to_f64(Xc_bits))
    Hd = Hs + lam * np.trace(Hs) / K * np.eye(K)
    W_hat = out["W_hat"]                                    # [N, K], original space
    for i in range(K // d):
        lo = i * d
        if i == 0:
            cur = Wv[:, lo:]
        else:
            delta = (W_hat[:, :lo] - Wv[:, :lo]).T          # [lo, N] error of the finished blocks
            cur = Wv[:, lo:] - np.linalg.solve(Hd[lo:, lo:], Hd[lo:, :lo] @ delta).T
        Wi = cur[:, :d].T                                   # [d, N] paper orientation
        T = WT.wush_block(Wi @ Wi.T / N, Hs[lo:lo + d, lo:lo + d], lam)
        bits = F.f64_to_bf16_bits(T)
        # the transform depends continuously on the block: same bf16 bits up to isolated last-place flips
        assert np.mean(bits == out["T_bits"][i]) >= 0.98
        That = out["T_hat"][i]
        wbar = out["T_xvsh"][i] @ Wi
        # conditional Hessian of block i given the finished blocks, later blocks free: Schur complement of Hd
        if lo + d < K:
            Hc = Hd[lo:lo + d, lo:lo + d] - Hd[lo:lo + d, lo + d:] @ np.linalg.solve(Hd[lo + d:, lo + d:], Hd[lo + d:, lo:lo + d])
        else:
            Hc = Hd[lo:lo + d, lo:lo + d]
        codes, sb, wq = G.gptq_block(wbar, That @ Hc @ That.T, fmt, ts_w)
        same = np.all(codes.T == out["codes"][:, lo:lo + d], axis=1)
        assert same.mean() >= 0.97, (i, same.mean())
        assert np.array_equal(sb[same], out["scales"][same, i])


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_reduces_to_rtn_case_for_block_diagonal_hessian(fmt):
    """Calibration tokens that are non-zero in one block only make the Hessian block diagonal: nothing crosses
    blocks, every transform is the RTN case's, and with the intra-block spreading off the codes are too."""
    d = Q.GROUP[fmt]
    C, N, B = 3, 40, 96
    cfg = synth.CONFIGS[1]
    W_bits = synth.weights(cfg, N=N, K=C * d)
    Xc_bits = synth.calibration(cfg, B=C * B, K=C * d).copy()
    for c in range(C):                                      # token t belongs to block t // B
        keep = np.zeros(C * d, dtype=bool); keep[c * d:(c + 1) * d] = True
        Xc_bits[c * B:(c + 1) * B, ~keep] = 0
    L = P.PreparedLayer(W_bits, Xc_bits, fmt)
    out = G.wush_gptq_layer(W_bits, Xc_bits, fmt, 0.01, L.ts_w, intra=False)
    assert np.array_equal(out["T_bits"], L.T_bits)
    assert np.array_equal(out["scales"], L.w_scales)
    assert np.array_equal(out["codes"], L.w_codes)
    assert np.allclose(out["w_deq"], L.w_deq, rtol=0, atol=0)
    # with the spreading on, the scales (taken before any spreading) are still the RTN case's
    out2 = G.wush_gptq_layer(W_bits, Xc_bits, fmt, 0.01, L.ts_w)
    assert np.array_equal(out2["scales"], L.w_scales) and np.array_equal(out2["T_bits"], L.T_bits)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_proxy_loss_not_above_rtn_case(fmt):
    d = Q.GROUP[fmt]
    for seed in (1, 2, 3):
        W_bits, Xc_bits = _correlated_layer(seed, 64, 4 * d, 512)
        Wv = F.bf16_bits_to_f64(W_bits)
        Hs = G.hessian(F.bf16_bits_to_f64(Xc_bits))
        L = P.PreparedLayer(W_bits, Xc_bits, fmt)
        W_rtn = np.concatenate([L.w_deq[:, c * d:(c + 1) * d] @ L.T_hat[c] for c in range(4)], axis=1)
        out = G.wush_gptq_layer(W_bits, Xc_bits, fmt, 0.01, L.ts_w)
        assert G.proxy_loss(out["W_hat"], Wv, Hs) < G.proxy_loss(W_rtn, Wv, Hs)
        # the GEMM operand and the original-space view describe the same weights
        back = np.concatenate([out["w_deq"][:, c * d:(c + 1) * d] @ out["T_hat"][c] for c in range(4)], axis=1)
        assert np.allclose(back, out["W_hat"], rtol=0, atol=1e-12)

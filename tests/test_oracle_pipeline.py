"""Pins for the oracle's end-to-end path (CPU only): invariance before quantisation,
exact-rational dequantised products, moments, and the qualitative ordering of Table 1."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from oracle import wush_transform as WT
from paper_2512_00956_b200 import synth


def _small_layer(fmt, M=24, N=40, K=128, B=256, cfg_idx=1):
    cfg = synth.CONFIGS[cfg_idx]
    d = synth.layer_inputs(cfg, M=M, N=N, K=K, B=B)
    return d, P.PreparedLayer(d["W"], d["Xc"], fmt)


def test_second_moment_sums_brute_force():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((5, 32))
    S = P.second_moment_sums(X, 16)
    for c in range(2):
        ref = np.zeros((16, 16))
        for t in range(5):
            x = X[t, c * 16:(c + 1) * 16]
            ref += np.outer(x, x)
        assert np.allclose(S[c], ref, rtol=1e-13)


def test_transform_blocks_brute_force_orientation():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((3, 32)); T = rng.standard_normal((2, 16, 16))
    v = P.transform_blocks(X, T)
    for m in range(3):
        for c in range(2):
            ref = T[c] @ X[m, c * 16:(c + 1) * 16]            # the paper's T_(i) x on a column block
            assert np.allclose(v[m, c * 16:(c + 1) * 16], ref, rtol=1e-13)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_prequantisation_invariance(fmt):
    """W x = (W T^-1)(T x): with the fp64 inverse-transpose of the rounded transform, to 1e-10."""
    d, L = _small_layer(fmt, M=16, N=32, K=256)
    Xv, Wv = F.bf16_bits_to_f64(d["X"]), F.bf16_bits_to_f64(d["W"])
    Tx = np.stack([WT.xvsh_from_wush(L.T_hat[c]) for c in range(L.T_hat.shape[0])])
    y0 = Xv @ Wv.T
    y1 = P.transform_blocks(Xv, L.T_hat) @ P.transform_blocks(Wv, Tx).T
    assert np.linalg.norm(y1 - y0) / np.linalg.norm(y0) < 1e-10
    # the fp32 copy handed to the GPU library costs about one fp32 rounding
    y2 = P.transform_blocks(Xv, L.T_hat) @ P.transform_blocks(Wv, L.T_xvsh32.astype(np.float64)).T
    assert np.linalg.norm(y2 - y0) / np.linalg.norm(y0) < 1e-6


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_dequantised_product_exact_rational(fmt):
    g = Q.GROUP[fmt]
    d, L = _small_layer(fmt, M=3, N=4, K=2 * g, B=64)
    _, codes, scales = L.quantize_act(d["X"])
    Y = L.forward(d["X"])
    grid = [Fraction(x) for x in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]

    def deq(c, sbyte, ts):
        mag = grid[int(c) & 7] * (-1 if int(c) & 8 else 1)
        if fmt == "mxfp4":
            s = Fraction(2) ** (int(sbyte) - 127)
        else:
            s = Fraction(float(F.e4m3_decode(np.uint8(sbyte)))) * Fraction(float(ts))
        return mag * s

    for m in range(3):
        for n in range(4):
            acc = Fraction(0)
            for k in range(2 * g):
                acc += deq(codes[m, k], scales[m, k // g], L.ts_x) * deq(L.w_codes[n, k], L.w_scales[n, k // g], L.ts_w)
            assert Y[m, n] == pytest.approx(float(acc), rel=1e-13, abs=0)
            if fmt == "mxfp4":
                assert Y[m, n] == float(acc)               # dyadic rationals: fp64 sum is exact


@pytest.mark.parametrize("fmt,level", [("mxfp4", 0.2), ("nvfp4", 0.2)])
def test_forward_close_to_unquantised(fmt, level):
    d, L = _small_layer(fmt, M=64, N=96, K=512, B=512)
    Y = L.forward(d["X"])
    Yref = F.bf16_bits_to_f64(d["X"]) @ F.bf16_bits_to_f64(d["W"]).T
    rel = np.linalg.norm(Y - Yref) / np.linalg.norm(Yref)
    assert 0.005 < rel < level
    rows = np.array([3, 17, 40])
    assert np.allclose(L.forward(d["X"], rows=rows), Y[rows], rtol=1e-12, atol=1e-12)


def test_switches_ceil_rule_and_dynamic_tensor_scale():
    """The two optional rules run through the same pipeline.  Ceil rule: no transformed activation or weight
    saturates.  Per-batch NVFP4 scale: the block that holds the batch's AbsMax uses the top E4M3 scale (448),
    a batch 100x larger than the calibration data still quantises without clipping (the static scale clips it),
    and restricting the output rows does not change the scale."""
    d, L = _small_layer("mxfp4_ceil", M=64, N=96, K=512, B=512)
    v32, codes, scales = L.quantize_act(d["X"])
    assert np.abs(v32.reshape(64, 16, 32) / F.e8m0_decode(scales)[:, :, None]).max() <= 6.0
    assert np.abs(L.wbar32.reshape(96, 16, 32) / F.e8m0_decode(L.w_scales)[:, :, None]).max() <= 6.0
    Yref = F.bf16_bits_to_f64(d["X"]) @ F.bf16_bits_to_f64(d["W"]).T
    rel = np.linalg.norm(L.forward(d["X"]) - Yref) / np.linalg.norm(Yref)
    assert 0.005 < rel < 0.2

    d, L = _small_layer("nvfp4", M=64, N=96, K=512, B=512)
    ts = L.dynamic_ts_x(d["X"])
    _, _, sb = L.quantize_act(d["X"], ts)
    assert sb.max() == 0x7E
    Y = L.forward(d["X"], dynamic=True)
    rows = np.array([3, 17, 40])
    assert np.allclose(L.forward(d["X"], rows=rows, dynamic=True), Y[rows], rtol=1e-12, atol=1e-12)
    big = F.f64_to_bf16_bits(F.bf16_bits_to_f64(d["X"]) * 128.0)          # exact in bf16: a power of two
    Yb_ref = 128.0 * Yref_nv(d)
    e_dyn = np.linalg.norm(L.forward(big, dynamic=True) - Yb_ref) / np.linalg.norm(Yb_ref)
    e_sta = np.linalg.norm(L.forward(big) - Yb_ref) / np.linalg.norm(Yb_ref)
    assert e_dyn < 0.2 and e_sta > 2 * e_dyn


def Yref_nv(d):
    return F.bf16_bits_to_f64(d["X"]) @ F.bf16_bits_to_f64(d["W"]).T


def _layer_loss(kind, fmt, d, rng):
    g = Q.GROUP[fmt]
    Xv, Wv, Xc = (F.bf16_bits_to_f64(d[k]) for k in ("X", "W", "Xc"))
    C = Xv.shape[1] // g
    mW = P.second_moment_sums(Wv, g) / Wv.shape[0]
    mX = P.second_moment_sums(Xc, g) / Xc.shape[0]
    T = np.stack([WT.variant_transform(kind, mW[c], mX[c], rng=rng) for c in range(C)])
    Tx = np.stack([WT.xvsh_from_wush(T[c]) for c in range(C)])
    v = P.transform_blocks(Xv, T).astype(np.float32)
    w = P.transform_blocks(Wv, Tx).astype(np.float32)
    tsx = Q.nvfp4_tensor_scale(P.transform_blocks(Xc, T).astype(np.float32)) if fmt == "nvfp4" else None
    tsw = Q.nvfp4_tensor_scale(w) if fmt == "nvfp4" else None
    xd = Q.dequantize(*Q.quantize(v, fmt, tsx), fmt, tsx)
    wd = Q.dequantize(*Q.quantize(w, fmt, tsw), fmt, tsw)
    Y0 = Xv @ Wv.T
    return np.linalg.norm(xd @ wd.T - Y0) / np.linalg.norm(Y0)


def test_table1_ordering_on_synthetic_layer():
    """Table 1's qualitative ordering: for MXFP4, WUSH < H < I; WUSH beats every variant."""
    cfg = synth.CONFIGS[1]
    d = synth.layer_inputs(cfg, M=128, N=256, K=512, B=512)
    rng = np.random.default_rng(7)
    mx = {k: _layer_loss(k, "mxfp4", d, rng) for k in ("I", "R", "H", "WUS", "WUSH")}
    assert mx["WUSH"] < mx["H"] < mx["I"]
    assert mx["WUSH"] < mx["R"] and mx["WUSH"] < mx["WUS"]
    nv = {k: _layer_loss(k, "nvfp4", d, rng) for k in ("I", "H", "WUSH")}
    assert nv["WUSH"] < nv["I"] and nv["WUSH"] < nv["H"]


def test_synth_generators_are_seeded_and_shaped():
    cfg = synth.CONFIGS[2]
    a = synth.activations(cfg, M=8, K=256); b = synth.activations(cfg, M=8, K=256)
    assert a.dtype == np.uint16 and a.shape == (8, 256) and np.array_equal(a, b)
    s = synth.channel_scales(cfg, K=4096)
    assert int(round(0.01 * 4096)) == np.sum(s > 12)          # 41 outlier channels x50 stand out
    assert not np.array_equal(synth.calibration(cfg, B=8, K=256), a)
    for i, c in synth.CONFIGS.items():
        for f in c.formats:
            assert c.K % synth.GROUP[f] == 0

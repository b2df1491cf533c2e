"""Parity at the benchmark's full sizes (configs 3-5), in the launch configuration bench.py uses
(`wush_linear`, TILED scales, persistent kernels).  Activations are checked in full (codes and
scale bytes, guard-band rule; at M = 16384 on 256 sampled token rows); Y is checked on sampled
token rows, and for the 28672-wide layer also on sampled output channels, because the fp64 oracle
cannot afford the full product."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import synth, wush
from parity_util import compare_quantized, dev, dev_bf16, rel_fro, untile

pytestmark = pytest.mark.gpu
G = Q.GROUP


def _check_layer(cfg, fmt, M, W_bits, Xc_bits, seed=0, rows=64, check_codes=True, dynamic=False):
    g = G[fmt]
    X_bits = synth.activations(cfg, M=M)
    L = P.PreparedLayer(W_bits, Xc_bits, fmt)
    K, N = cfg.K, W_bits.shape[0]
    X, W = dev_bf16(X_bits), dev_bf16(W_bits)
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if (fmt == "nvfp4" and not dynamic) else None
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, fmt, tsx, tsw)      # NVFP4 without tsx: per-batch scale
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, K, g) == 0
    ts_x = L.dynamic_ts_x(X_bits) if dynamic else L.ts_x
    if dynamic:
        assert abs(wush.linear_dynamic_scale(wsp, M, K, g)[0] - float(ts_x)) <= 2e-7 * float(ts_x)
    if check_codes:                                    # the activation codes wush_linear left in its workspace
        codes = wsp[: M * K // 2].view(M, K // 2).cpu().numpy()
        off = (M * K // 2 + 15) // 16 * 16
        sc = untile(wsp[off: off + wush.scale_bytes(M, K, g, wush.SF_TILED)].cpu().numpy(), M, K // g)
        v32, _, _ = L.quantize_act(X_bits, ts_x)
        compare_quantized(codes, sc, v32, fmt, ts_x)
    rng = np.random.default_rng(seed)
    pick = np.sort(rng.choice(M, size=min(rows, M), replace=False))
    if not check_codes:                                # too many rows for the oracle: codes and scales of sampled rows
        sel = np.sort(rng.choice(M, size=256, replace=False))
        codes = wsp[: M * K // 2].view(M, K // 2)[torch.from_numpy(sel).cuda()].cpu().numpy()
        off = (M * K // 2 + 15) // 16 * 16
        sc = untile(wsp[off: off + wush.scale_bytes(M, K, g, wush.SF_TILED)].cpu().numpy(), M, K // g)[sel]
        v32, _, _ = L.quantize_act(X_bits[sel], ts_x)
        compare_quantized(codes, sc, v32, fmt, ts_x)
    Yo = L.forward(X_bits, rows=pick, dynamic=dynamic)
    assert rel_fro(Y[torch.from_numpy(pick).cuda()].cpu().numpy(), Yo) <= 1e-3
    return L


def test_config3_mxfp4_full():
    cfg = synth.CONFIGS[3]
    _check_layer(cfg, "mxfp4", cfg.M, synth.weights(cfg), synth.calibration(cfg))


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4", "mxfp4_ceil"])
def test_config4_full(fmt):
    cfg = synth.CONFIGS[4]
    _check_layer(cfg, fmt, cfg.M, synth.weights(cfg), synth.calibration(cfg))


def test_config2_per_batch_tensor_scale_full():
    cfg = synth.CONFIGS[2]
    _check_layer(cfg, "nvfp4", cfg.M, synth.weights(cfg), synth.calibration(cfg), dynamic=True)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_config5_token_sweep(fmt):
    """M in {1, 16, 128, 1024, 4096, 16384} at K = 8192 against the first 4096 output channels of the
    28672-wide layer (weight rows are independent; the subset keeps the fp64 oracle affordable)."""
    cfg = synth.CONFIGS[5]
    W_bits = synth.weights(cfg, N=4096)
    Xc_bits = synth.calibration(cfg)
    for M in cfg.m_sweep:
        _check_layer(cfg, fmt, M, W_bits, Xc_bits, seed=M, rows=32, check_codes=(M <= 4096))


@pytest.mark.parametrize("fmt,M", [("mxfp4", 4096), ("nvfp4", 4096), ("nvfp4", 16384)])
def test_config5_full_width_sampled_channels(fmt, M):
    """All 28672 output channels on the GPU; the oracle prepares 512 sampled channels (and, for NVFP4, the
    tensor scale of the whole transformed weight matrix, which needs the transform but not the quantiser)."""
    cfg = synth.CONFIGS[5]
    g = G[fmt]
    W_bits = synth.weights(cfg)
    Xc_bits = synth.calibration(cfg)
    X_bits = synth.activations(cfg, M=M)
    rng = np.random.default_rng(5 + M)
    cols = np.sort(rng.choice(cfg.N, size=512, replace=False))
    rows = np.sort(rng.choice(M, size=64, replace=False))
    # transforms depend on the weight moments of ALL channels: take them from the full matrix
    Wv = F.bf16_bits_to_f64(W_bits)
    Xcv = F.bf16_bits_to_f64(Xc_bits)
    momW = P.second_moment_sums(Wv, g) / Wv.shape[0]
    momX = P.second_moment_sums(Xcv, g) / Xcv.shape[0]
    from oracle import wush_transform as WT
    T_bits, T_hat, T_xvsh = WT.build_transforms(momW, momX, 0.01)
    Tx32 = np.ascontiguousarray(T_xvsh, dtype=np.float32)
    ts_w = ts_x = None
    if fmt == "nvfp4":
        amax_w = 0.0
        for r0 in range(0, cfg.N, 4096):          # AbsMax of the whole transformed tensor, in slices
            amax_w = max(amax_w, float(np.max(np.abs(P.transform_blocks(Wv[r0:r0 + 4096], Tx32.astype(np.float64)).astype(np.float32)))))
        ts_w = np.float32(np.float32(amax_w) / np.float32(2688.0))
        ts_x = Q.nvfp4_tensor_scale(P.transform_blocks(Xcv, T_hat).astype(np.float32))
    wbar = P.transform_blocks(Wv[cols], Tx32.astype(np.float64)).astype(np.float32)
    del Wv
    wc, wsb = Q.quantize(wbar, fmt, ts_w)
    wdeq = Q.dequantize(wc, wsb, fmt, ts_w)
    v32, xc, xs = P.quantize_transformed(F.bf16_bits_to_f64(X_bits[rows]), T_hat, fmt, ts_x)
    Yo = P.dequantized_product(Q.dequantize(xc, xs, fmt, ts_x), wdeq)
    X, W = dev_bf16(X_bits), dev_bf16(W_bits)
    wq, ws, tsw_g = wush.quantize_weight(W, dev(Tx32), fmt, sf=wush.SF_TILED)
    tsx_g = dev(np.full(4, ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, wsp = wush.linear(X, dev_bf16(T_bits), wq, ws, fmt, tsx_g, tsw_g)
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, cfg.K, g) == 0
    if fmt == "nvfp4":
        assert abs(float(tsw_g[0].item()) - float(ts_w)) <= 2e-7 * float(ts_w)
    Yg = Y[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].cpu().numpy()
    assert rel_fro(Yg, Yo) <= 1e-3

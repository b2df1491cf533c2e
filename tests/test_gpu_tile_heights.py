"""GPU parity of the streaming quantiser's two tile heights (64 and 128 token rows) on RAGGED problems.

The library picks 128-row tiles once every SM gets at least five 128 x 128 work items, so the predicated copy
of the 128-row item body (last row block with M % 128 != 0, last channel panel with K % 128 != 0) only runs on
large ragged inputs, and the 64-row one only on small ones.  Two routes reach both here:
  * inputs large enough to select 128-row tiles by themselves (M = 4099 / K = 4096: 33 x 32 = 1056 items;
    M = 3000 / K = 4160: 24 x 33 = 792 items, K tail of 64 channels), static and per-batch tensor scale;
  * the test hook `wush_debug_quantiser_rows`, which forces either height on the small ragged shapes of a
    seeded sweep, all three quantiser rules, both scale layouts, and through `wush_linear`.
Oracle side: transform in fp64, one rounding to fp32, the quantiser definition.  Tolerances: guard-band rule
for codes and scale bytes (identical outside the 1e-4 bands), 1e-3 relative Frobenius for Y.
"""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import synth, wush
from parity_util import compare_quantized, dev, dev_bf16, rel_fro, untile

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _automatic_height_afterwards():
    yield
    wush.debug_quantiser_rows(0)


def _random_problem(rng, M, K, fmt):
    g = Q.GROUP[fmt]
    X_bits = F.f64_to_bf16_bits(rng.standard_normal((M, K)) * np.exp(rng.uniform(-2, 2, (1, K))))
    T_bits = F.f64_to_bf16_bits(rng.standard_normal((K // g, g, g)) / np.sqrt(g))
    v32 = P.transform_blocks(F.bf16_bits_to_f64(X_bits), F.bf16_bits_to_f64(T_bits)).astype(np.float32)
    return X_bits, T_bits, v32


def _check_act(X_bits, T_bits, v32, fmt, sf, dynamic=False):
    M, K = X_bits.shape
    g = Q.GROUP[fmt]
    ts = Q.nvfp4_tensor_scale(v32) if fmt == "nvfp4" else None
    if dynamic:
        codes, scales, ts_g = wush.quantize_act_dynamic(dev_bf16(X_bits), dev_bf16(T_bits), sf)
        torch.cuda.synchronize()
        # the device finds AbsMax over its own fp32-accumulated products: equal to the oracle's up to that rounding;
        # the scale it derived must be exactly AbsMax / 2688 in fp32, and the codes are checked under that scale
        amax_g = np.float32(ts_g[1].item())
        assert abs(float(amax_g) - float(np.max(np.abs(v32)))) <= 1e-6 * float(np.max(np.abs(v32)))
        assert np.float32(ts_g[0].item()) == np.float32(amax_g / np.float32(2688.0))
        ts = np.float32(ts_g[0].item())
    else:
        ts_d = dev(np.full(4, ts, dtype=np.float32)) if ts is not None else None
        codes, scales = wush.quantize_act(dev_bf16(X_bits), dev_bf16(T_bits), fmt, ts_d, sf)
        torch.cuda.synchronize()
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, M, K // g)
    stats = compare_quantized(codes.cpu().numpy(), sc, v32, fmt, ts)
    assert stats["flipped_codes"] <= stats["guarded_elems"], (fmt, M, K, sf)
    return stats


# ------------------------------------------------------------------ sizes that select 128-row tiles by themselves
@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
@pytest.mark.parametrize("M,K", [(4099, 4096), (3000, 4160)])
@pytest.mark.parametrize("sf", [wush.SF_LINEAR, wush.SF_TILED])
def test_large_ragged_selects_128_row_tiles(fmt, M, K, sf):
    assert wush.debug_quantiser_rows(0) == 0
    assert ((K // 32 + 3) // 4) * ((M + 127) // 128) >= 5 * 148      # the library's own rule for 128-row tiles
    rng = np.random.default_rng(M + K)
    _check_act(*_random_problem(rng, M, K, fmt), fmt, sf)


@pytest.mark.parametrize("M,K", [(4099, 4096), (3000, 4160)])
def test_large_ragged_per_batch_scale_128_row_tiles(M, K):
    """The AbsMax instantiation on 128-row tiles, then the quantising pass that reads its result."""
    rng = np.random.default_rng(7 * M + K)
    _check_act(*_random_problem(rng, M, K, "nvfp4"), "nvfp4", wush.SF_TILED, dynamic=True)


# ------------------------------------------------------------------ both heights forced on small ragged shapes
@pytest.mark.parametrize("rows", [64, 128])
def test_forced_height_random_shapes(rows):
    wush.debug_quantiser_rows(rows)
    assert wush.debug_quantiser_rows(rows) == rows
    rng = np.random.default_rng(100 + rows)
    for i in range(24):
        fmt = ("mxfp4", "nvfp4", "mxfp4_ceil")[i % 3]
        K = int(rng.choice([64, 128, 192, 256, 320, 576, 1024, 2112]))
        M = int(rng.integers(1, 900))
        sf = int(rng.integers(0, 2))
        if sf == wush.SF_LINEAR and (K // Q.GROUP[fmt]) % 4 != 0:
            sf = wush.SF_TILED                    # the streaming kernel declines such LINEAR rows: keep it in play
        _check_act(*_random_problem(rng, M, K, fmt), fmt, sf)


@pytest.mark.parametrize("rows", [64, 128])
def test_forced_height_per_batch_scale(rows):
    wush.debug_quantiser_rows(rows)
    rng = np.random.default_rng(200 + rows)
    for M, K in ((1, 64), (129, 320), (531, 1024), (77, 2112)):
        _check_act(*_random_problem(rng, M, K, "nvfp4"), "nvfp4", wush.SF_TILED, dynamic=True)


def test_hook_rejects_other_heights():
    with pytest.raises(wush.WushError):
        wush.debug_quantiser_rows(96)
    assert wush.debug_quantiser_rows(0) == 0


@pytest.mark.parametrize("rows", [64, 128])
@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_forced_height_whole_layer(rows, fmt):
    """wush_linear on a ragged layer with either height: same codes in the workspace, Y within tolerance, and
    bit-identical Y for the two heights (the quantiser's output does not depend on its tiling)."""
    g = Q.GROUP[fmt]
    M, N, K = 389, 264, 832
    d = synth.layer_inputs(synth.CONFIGS[2], M=M, N=N, K=K, B=256)
    L = P.PreparedLayer(d["W"], d["Xc"], fmt)
    X, W = dev_bf16(d["X"]), dev_bf16(d["W"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    wush.debug_quantiser_rows(rows)
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, fmt, tsx, tsw)
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, K, g) == 0
    codes = wsp[: M * K // 2].view(M, K // 2).cpu().numpy()
    off = (M * K // 2 + 15) // 16 * 16
    sc = untile(wsp[off: off + wush.scale_bytes(M, K, g, wush.SF_TILED)].cpu().numpy(), M, K // g)
    v32, _, _ = L.quantize_act(d["X"])
    compare_quantized(codes, sc, v32, fmt, L.ts_x)
    assert rel_fro(Y.cpu().numpy(), L.forward(d["X"])) <= 1e-3
    wush.debug_quantiser_rows(192 - rows)
    Y2, wsp2 = wush.linear(X, dev_bf16(L.T_bits), wq, ws, fmt, tsx, tsw)
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2) and torch.equal(wsp[: M * K // 2], wsp2[: M * K // 2])


@pytest.mark.parametrize("rows", [0, 64])
@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4", "mxfp4_ceil"])
def test_weight_quantiser_on_both_kernels(rows, fmt):
    """wush_quantize_weight (fp32 transforms, exact three-way bf16 split) through the tcgen05 kernel (hook 0, the
    default for more than 256 rows) and through the warp-level kernel (hook 64), ragged row count and a channel tail:
    both against the oracle, and bit-identical scale bytes between the two."""
    g = Q.GROUP[fmt]
    rng = np.random.default_rng(31)
    N, K = 1237, 1088
    W_bits = F.f64_to_bf16_bits(0.02 * rng.standard_normal((N, K)) * np.exp(rng.uniform(-1, 1, (1, K))))
    Tinv = (rng.standard_normal((K // g, g, g)) / np.sqrt(g)).astype(np.float32)
    wbar = P.transform_blocks(F.bf16_bits_to_f64(W_bits), Tinv.astype(np.float64)).astype(np.float32)
    ts = Q.nvfp4_tensor_scale(wbar) if fmt == "nvfp4" else None
    wush.debug_quantiser_rows(rows)
    for sf in (wush.SF_LINEAR, wush.SF_TILED):
        codes, scales, ts_g = wush.quantize_weight(dev_bf16(W_bits), dev(Tinv), fmt, sf=sf)
        torch.cuda.synchronize()
        sc = scales.cpu().numpy()
        if sf == wush.SF_TILED:
            sc = untile(sc, N, K // g)
        if fmt == "nvfp4":
            assert abs(float(ts_g[0].item()) - float(ts)) <= 2e-7 * float(ts)
        stats = compare_quantized(codes.cpu().numpy(), sc, wbar, fmt, ts)
        assert stats["flipped_codes"] <= stats["guarded_elems"]

"""GPU parity tests: every entry point of libwush against the CPU oracle on the same
seeded inputs, called through the C ABI (ctypes binding).  Sizes span several tiles and
ragged tails; tolerances are the build target's:
  - stand-alone quantiser on fp32 input: codes and scale bytes bit-exact;
  - transform: |v_gpu - v_oracle| <= 1e-5 * AbsMax(block);
  - transform + quantise: bit-exact outside the 1e-4 guard bands, one step inside;
  - Y: relative Frobenius error <= 1e-3 (fp32 output);  moments: <= 1e-5.
"""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import synth, wush
from parity_util import (compare_quantized, dev, dev_bf16, rel_fro, tile, untile)

pytestmark = pytest.mark.gpu
G = Q.GROUP


def _sync():
    torch.cuda.synchronize()


# ------------------------------------------------------------------ stand-alone quantiser
def _quantizer_inputs(fmt, R, K, seed):
    rng = np.random.default_rng(seed)
    g = G[fmt]
    spread = 20 if fmt == "mxfp4" else 3
    v = (rng.standard_normal((R, K)) * np.exp(rng.uniform(-spread, spread, (R, K // g, 1)).repeat(g, 2).reshape(R, K)))
    v = v.astype(np.float32)
    v[0, :g] = 0.0                                            # all-zero block
    v[1, :g] = -0.0
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 4.0, -0.25, -5.0], dtype=np.float32)
    v[2, :g] = 0; v[2, :len(mids)] = mids                     # exact ties, block AbsMax 6 -> scale 1
    v[3, :g] = np.float32(2.0 ** 5) * (1 - 2.0 ** -24)        # just under a power of two
    v[4, :g] = 1e-38 if fmt == "mxfp4" else 1e-6              # tiny / subnormal scale region
    v[5, :g] = 3e38 if fmt == "mxfp4" else 1e4                # huge (NVFP4: saturating scale)
    return v


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
@pytest.mark.parametrize("sf", [wush.SF_LINEAR, wush.SF_TILED])
def test_quantize_f32_bit_exact(fmt, sf):
    R, K = 333, 512
    v = _quantizer_inputs(fmt, R, K, 11)
    ts = np.float32(0.0371) if fmt == "nvfp4" else None
    ts_d = dev(np.full(4, ts, dtype=np.float32)) if ts is not None else None
    codes, scales = wush.quantize_f32(dev(v), fmt, ts_d, sf)
    _sync()
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, R, K // G[fmt])
    compare_quantized(codes.cpu().numpy(), sc, v, fmt, ts, strict=True)


# ------------------------------------------------------------------ transform alone
def _layer(idx, fmt, M=None, N=None, K=None, B=None):
    cfg = synth.CONFIGS[idx]
    d = synth.layer_inputs(cfg, M=M, N=N, K=K, B=B)
    return d, P.PreparedLayer(d["W"], d["Xc"], fmt)


@pytest.mark.parametrize("fmt,M,K", [("mxfp4", 128, 2048), ("nvfp4", 77, 320), ("mxfp4", 1, 64), ("nvfp4", 300, 1024)])
def test_transform_act_f32(fmt, M, K):
    d, L = _layer(1, fmt, M=M, N=64, K=K, B=256)
    g = G[fmt]
    V = wush.transform_act_f32(dev_bf16(d["X"]), dev_bf16(L.T_bits), g)
    _sync()
    v_o = P.transform_blocks(F.bf16_bits_to_f64(d["X"]), L.T_hat)
    amax = np.abs(v_o.reshape(M, K // g, g)).max(axis=2).repeat(g, axis=1)
    err = np.abs(V.cpu().numpy().astype(np.float64) - v_o)
    assert np.all(err <= 1e-5 * amax + 1e-300), float((err / np.maximum(amax, 1e-300)).max())


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_transform_weight_f32(fmt):
    d, L = _layer(1, fmt, M=16, N=200, K=384, B=256)
    g = G[fmt]
    V = wush.transform_weight_f32(dev_bf16(d["W"]), dev(L.T_xvsh32), g)
    _sync()
    w_o = P.transform_blocks(F.bf16_bits_to_f64(d["W"]), L.T_xvsh32.astype(np.float64))
    amax = np.abs(w_o.reshape(200, 384 // g, g)).max(axis=2).repeat(g, axis=1)
    err = np.abs(V.cpu().numpy().astype(np.float64) - w_o)
    assert np.all(err <= 1e-5 * amax), float((err / amax).max())


# ------------------------------------------------------------------ transform + quantise
@pytest.mark.parametrize("fmt,M,K,sf", [
    ("mxfp4", 128, 2048, wush.SF_LINEAR), ("mxfp4", 77, 192, wush.SF_LINEAR), ("mxfp4", 1, 64, wush.SF_TILED),
    ("mxfp4", 300, 1024, wush.SF_TILED), ("nvfp4", 128, 2048, wush.SF_LINEAR), ("nvfp4", 77, 320, wush.SF_TILED),
    ("nvfp4", 16, 64, wush.SF_LINEAR), ("nvfp4", 531, 1024, wush.SF_TILED)])
def test_quantize_act_parity(fmt, M, K, sf):
    d, L = _layer(1 if fmt == "mxfp4" else 2, fmt, M=M, N=64, K=K, B=256)
    ts_d = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    codes, scales = wush.quantize_act(dev_bf16(d["X"]), dev_bf16(L.T_bits), fmt, ts_d, sf)
    _sync()
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, M, K // G[fmt])
    v32, _, _ = L.quantize_act(d["X"])
    stats = compare_quantized(codes.cpu().numpy(), sc, v32, fmt, L.ts_x)
    assert stats["flipped_codes"] <= stats["guarded_elems"]


def test_quantize_act_deterministic_and_in_bounds():
    d, L = _layer(1, "mxfp4", M=200, N=64, K=512, B=256)
    X, T = dev_bf16(d["X"]), dev_bf16(L.T_bits)
    pad = 4096
    codes = torch.full((200 * 256 + 2 * pad,), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.full((200 * 16 + 2 * pad,), 0xCD, dtype=torch.uint8, device="cuda")
    out = (codes[pad:pad + 200 * 256].view(200, 256), scales[pad:pad + 200 * 16].view(200, 16))
    wush.quantize_act(X, T, "mxfp4", None, wush.SF_LINEAR, out=out)
    c1, s1 = out[0].clone(), out[1].clone()
    wush.quantize_act(X, T, "mxfp4", None, wush.SF_LINEAR, out=out)
    _sync()
    assert torch.equal(c1, out[0]) and torch.equal(s1, out[1])
    for buf, val, n in ((codes, 0xAB, 200 * 256), (scales, 0xCD, 200 * 16)):     # canaries untouched
        assert bool((buf[:pad] == val).all()) and bool((buf[pad + n:] == val).all())


# ------------------------------------------------------------------ weight side
@pytest.mark.parametrize("fmt,N,K", [("mxfp4", 200, 384), ("nvfp4", 200, 384), ("mxfp4", 2048, 2048), ("nvfp4", 1000, 1024)])
def test_quantize_weight_parity(fmt, N, K):
    d, L = _layer(1, fmt, M=16, N=N, K=K, B=256)
    codes, scales, ts = wush.quantize_weight(dev_bf16(d["W"]), dev(L.T_xvsh32), fmt, sf=wush.SF_LINEAR)
    _sync()
    if fmt == "nvfp4":
        ts_g = float(ts.cpu().numpy()[0])
        assert abs(ts_g - float(L.ts_w)) <= 2e-7 * float(L.ts_w)
    compare_quantized(codes.cpu().numpy(), scales.cpu().numpy(), L.wbar32, fmt, L.ts_w)


# ------------------------------------------------------------------ moments
@pytest.mark.parametrize("g,B,K", [(32, 512, 2048), (16, 333, 320), (32, 1, 64), (16, 1024, 4096)])
def test_calib_moments(g, B, K):
    cfg = synth.CONFIGS[1]
    Xc = synth.calibration(cfg, B=B, K=K)
    mom, cnt = wush.calib_moments(dev_bf16(Xc), g)
    _sync()
    S = P.second_moment_sums(F.bf16_bits_to_f64(Xc), g)
    assert rel_fro(mom.cpu().numpy(), S) <= 1e-5
    assert int(cnt[0].item()) == B
    # accumulate in place: a second chunk adds on top, bit-identically from run to run
    mom2, cnt2 = wush.calib_moments(dev_bf16(Xc), g, mom.clone(), cnt.clone())
    mom3, _ = wush.calib_moments(dev_bf16(Xc), g, mom.clone(), cnt.clone())
    _sync()
    assert int(cnt2[0].item()) == 2 * B and torch.equal(mom2, mom3)
    assert rel_fro(mom2.cpu().numpy(), 2 * S) <= 1e-5


# ------------------------------------------------------------------ GEMM alone (oracle's codes in)
@pytest.mark.parametrize("fmt,M,N,K", [
    ("mxfp4", 128, 256, 256), ("mxfp4", 3, 8, 64), ("mxfp4", 200, 264, 448), ("mxfp4", 128, 2048, 2048),
    ("nvfp4", 128, 256, 256), ("nvfp4", 5, 16, 64), ("nvfp4", 131, 392, 320), ("nvfp4", 300, 1024, 1536),
    # every activation-slot height of the M <= 128 kernel (16, 32, 64 rows), K long enough for its ring to wrap
    ("mxfp4", 9, 264, 2560), ("nvfp4", 16, 128, 2304), ("mxfp4", 24, 136, 2048), ("nvfp4", 32, 264, 2048),
    ("mxfp4", 50, 128, 1792), ("nvfp4", 64, 136, 2048), ("nvfp4", 33, 8, 1536), ("mxfp4", 100, 72, 1600)])
def test_gemm_fp4_against_oracle_product(fmt, M, N, K):
    d, L = _layer(1, fmt, M=M, N=N, K=K, B=256)
    g = G[fmt]
    _, xc, xs = L.quantize_act(d["X"])
    Y_o = P.dequantized_product(Q.dequantize(xc, xs, fmt, L.ts_x), L.w_deq)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    tsw = dev(np.full(4, L.ts_w, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, status = wush.gemm_fp4(dev(F.pack_e2m1(xc)), dev(tile(xs)), dev(F.pack_e2m1(L.w_codes)), dev(tile(L.w_scales)),
                              K, fmt, tsx, tsw)
    _sync()
    assert int(status[0].item()) == 0, hex(int(status[0].item()))
    assert rel_fro(Y.cpu().numpy(), Y_o) <= 1e-5                      # same codes in: only fp32 accumulation differs
    Yb, _ = wush.gemm_fp4(dev(F.pack_e2m1(xc)), dev(tile(xs)), dev(F.pack_e2m1(L.w_codes)), dev(tile(L.w_scales)),
                          K, fmt, tsx, tsw, out_dtype=torch.bfloat16)
    _sync()
    Y_ob = F.round_to_bf16(Y_o)
    assert rel_fro(Yb.float().cpu().numpy(), Y_ob) <= 4e-3            # bf16 output vs bf16-rounded oracle


# ------------------------------------------------------------------ the whole layer
def _run_linear(idx, fmt, M=None, N=None, K=None, B=None, rows=None):
    d, L = _layer(idx, fmt, M=M, N=N, K=K, B=B)
    g = G[fmt]
    W, X = dev_bf16(d["W"]), dev_bf16(d["X"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, fmt, tsx, tsw)
    _sync()
    assert wush.linear_status(wsp, X.shape[0], X.shape[1], g) == 0
    Yg = Y.cpu().numpy()
    Y_o = L.forward(d["X"], rows=rows)
    return rel_fro(Yg if rows is None else Yg[rows], Y_o)


@pytest.mark.parametrize("fmt,M,N,K", [("mxfp4", 77, 136, 320), ("nvfp4", 77, 136, 320), ("mxfp4", 260, 520, 1024)])
def test_linear_small(fmt, M, N, K):
    assert _run_linear(1, fmt, M=M, N=N, K=K, B=256) <= 1e-3


def test_linear_config1_full():
    assert _run_linear(1, "mxfp4") <= 1e-3


def test_linear_config2_full():
    assert _run_linear(2, "nvfp4") <= 1e-3


# ------------------------------------------------------------------ GPU-side layer preparation
@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_prepare_layer_invariants_and_loss_level(fmt):
    """The product-side transform builder is checked by invariants (several T are equally valid),
    and the layer it prepares must reach the oracle's quantisation-error level."""
    from paper_2512_00956_b200 import prepare
    cfg = synth.CONFIGS[1]
    d = synth.layer_inputs(cfg, M=128, N=256, K=512, B=512)
    g = G[fmt]
    W, Xc, X = dev_bf16(d["W"]), dev_bf16(d["Xc"]), dev_bf16(d["X"])
    layer = prepare.QuantizedLinear(W, Xc, fmt)
    _sync()
    T = layer.T.double().cpu().numpy(); Tinv = layer.Tinv.double().cpu().numpy()
    for c in range(T.shape[0]):
        assert np.allclose(Tinv[c] @ T[c].T, np.eye(g), atol=1e-5)                 # Eq. 6 on the stored values
    Xcv = F.bf16_bits_to_f64(d["Xc"])
    mX = P.second_moment_sums(Xcv, g) / Xcv.shape[0]
    for c in range(0, T.shape[0], 5):                                              # equalised diagonal (appendix)
        A = T[c] @ (mX[c] + 0.01 * np.trace(mX[c]) / g * np.eye(g)) @ T[c].T
        assert np.ptp(np.diag(A)) <= 0.05 * np.diag(A).mean()
    Y = layer(X).cpu().numpy()
    Xv, Wv = F.bf16_bits_to_f64(d["X"]), F.bf16_bits_to_f64(d["W"])
    Y0 = Xv @ Wv.T
    L = P.PreparedLayer(d["W"], d["Xc"], fmt)
    loss_gpu = rel_fro(Y, Y0); loss_oracle = rel_fro(L.forward(d["X"]), Y0)
    assert abs(loss_gpu - loss_oracle) <= 0.1 * loss_oracle, (loss_gpu, loss_oracle)
    # the oracle's transforms and the GPU-built ones agree closely (same conventions)
    assert np.abs(T - L.T_hat).max() <= 0.02 * np.abs(L.T_hat).max()


def test_linear_bf16_output_config2_bench_configuration():
    """The configuration bench.py times by default: config 2, NVFP4, bf16 output."""
    d, L = _layer(2, "nvfp4")
    W, X = dev_bf16(d["W"]), dev_bf16(d["X"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), "nvfp4", sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32))
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, "nvfp4", tsx, tsw, out_dtype=torch.bfloat16)
    _sync()
    assert wush.linear_status(wsp, X.shape[0], X.shape[1], 16) == 0
    Yo = F.round_to_bf16(L.forward(d["X"]))
    assert rel_fro(Y.float().cpu().numpy(), Yo) <= 1e-3


@pytest.mark.parametrize("kind", ["hadamard", "identity", "wus"])
def test_fixed_transform_variants_run_through_the_same_kernels(kind):
    """H + Quant, None + Quant (Sec. 5) and WUS (Table 1) are the WUSH kernels with another T; on a layer
    with outlier channels the ordering of Table 1 must show: WUSH below each of them (MXFP4)."""
    from paper_2512_00956_b200 import prepare
    cfg = synth.CONFIGS[1]
    d = synth.layer_inputs(cfg, M=128, N=256, K=512, B=512)
    W, Xc, X = dev_bf16(d["W"]), dev_bf16(d["Xc"]), dev_bf16(d["X"])
    Y0 = F.bf16_bits_to_f64(d["X"]) @ F.bf16_bits_to_f64(d["W"]).T
    loss = {}
    for k in ("wush", kind):
        layer = prepare.QuantizedLinear(W, Xc, "mxfp4", transform=k)
        loss[k] = rel_fro(layer(X).cpu().numpy(), Y0)
    assert loss["wush"] < loss[kind]
    # and the fixed transform agrees with the oracle run on the same transform bytes
    layer = prepare.QuantizedLinear(W, Xc, "mxfp4", transform=kind)
    T = layer.T.double().cpu().numpy()
    Tx = layer.Tinv.double().cpu().numpy()
    v32 = P.transform_blocks(F.bf16_bits_to_f64(d["X"]), T).astype(np.float32)
    w32 = P.transform_blocks(F.bf16_bits_to_f64(d["W"]), Tx).astype(np.float32)
    Yo = P.dequantized_product(Q.dequantize(*Q.quantize(v32, "mxfp4"), "mxfp4"), Q.dequantize(*Q.quantize(w32, "mxfp4"), "mxfp4"))
    assert rel_fro(layer(X).cpu().numpy(), Yo) <= 1e-3


@pytest.mark.parametrize("g", [16, 32])
def test_library_fixed_transforms_match_the_oracle(g):
    """WUSH_KIND_HADAMARD / WUSH_KIND_IDENTITY: the stored bf16 matrix is the oracle's Sylvester-Hadamard matrix
    (or I) rounded to bf16, the same in every block, and Tinv is the inverse-transpose of the STORED values."""
    from oracle import wush_transform as WT
    C = 5
    for kind, ref in (("hadamard", WT.hadamard(g)), ("identity", np.eye(g))):
        T, Tinv, info = wush.fixed_transforms(kind, C, g, torch.device("cuda"))
        torch.cuda.synchronize()
        assert int(info.abs().max().item()) == 0
        bits = T.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(bits, np.broadcast_to(F.f64_to_bf16_bits(ref), (C, g, g)))
        That = F.bf16_bits_to_f64(bits)
        want = np.stack([WT.xvsh_from_wush(That[c]) for c in range(C)])
        assert np.max(np.abs(Tinv.double().cpu().numpy() - want)) <= 1e-6 * np.max(np.abs(want))


# ------------------------------------------------------------------ Algorithm 1 on the device
@pytest.mark.parametrize("fmt,K", [("mxfp4", 1024), ("nvfp4", 512)])
def test_build_transforms_kernel_against_oracle_and_identities(fmt, K):
    """wush_build_transforms: same conventions as the oracle, so the stored bf16 transforms agree to about
    one bf16 step; and the identities of Eq. 6 / the equalisation appendix hold on what it returns."""
    from oracle import wush_transform as WT
    g = G[fmt]
    cfg = synth.CONFIGS[1]
    d = synth.layer_inputs(cfg, M=16, N=768, K=K, B=640)
    Wv, Xcv = F.bf16_bits_to_f64(d["W"]), F.bf16_bits_to_f64(d["Xc"])
    sW, sX = P.second_moment_sums(Wv, g), P.second_moment_sums(Xcv, g)
    T, Tinv, info = wush.build_transforms(dev(sW.astype(np.float32)), Wv.shape[0], dev(sX.astype(np.float32)),
                                          Xcv.shape[0], g, 0.01)
    _sync()
    assert int(info.abs().max().item()) == 0
    Tg = T.double().cpu().numpy(); Tig = Tinv.double().cpu().numpy()
    bits, That, Tx = WT.build_transforms(sW / Wv.shape[0], sX / Xcv.shape[0], 0.01)
    scale = np.abs(That).max(axis=(1, 2), keepdims=True)
    assert np.all(np.abs(Tg - That) <= 2.0 ** -7 * np.abs(That) + 2e-3 * scale)
    assert np.mean(Tg == That) > 0.9                                   # most entries round to the same bf16 value
    C = K // g
    for c in range(C):
        assert np.allclose(Tig[c] @ Tg[c].T, np.eye(g), atol=1e-5)      # Eq. 6 on the stored values
    mX = sX / Xcv.shape[0]
    for c in range(0, C, 3):                                            # equalised diagonal, up to bf16 rounding of T
        A = Tg[c] @ WT.damped(mX[c], 0.01) @ Tg[c].T
        assert np.ptp(np.diag(A)) <= 0.05 * np.diag(A).mean()
    # and the layer prepared from it reaches the oracle's quantisation-error level
    L = P.PreparedLayer(d["W"], d["Xc"], fmt)
    X, W = dev_bf16(d["X"]), dev_bf16(d["W"])
    wq, ws, tsw = wush.quantize_weight(W, Tinv, fmt, sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, _ = wush.linear(X, T, wq, ws, fmt, tsx, tsw)
    _sync()
    Y0 = F.bf16_bits_to_f64(d["X"]) @ Wv.T
    lg, lo = rel_fro(Y.cpu().numpy(), Y0), rel_fro(L.forward(d["X"]), Y0)
    assert abs(lg - lo) <= 0.15 * lo, (lg, lo)


@pytest.mark.parametrize("g,K", [(32, 512), (16, 256)])
def test_wus_kind_and_invert_transforms(g, K):
    """WUSH_KIND_WUS is WUSH without its Hadamard factor (Table 1's "WUS"): H T_wus reproduces the WUSH transform
    of the same moments, and the kernel agrees with the oracle's WUS; wush_invert_transforms returns the
    inverse-transpose of any stored transforms (Eq. 6)."""
    from oracle import wush_transform as WT
    cfg = synth.CONFIGS[1]
    d = synth.layer_inputs(cfg, M=16, N=512, K=K, B=512)
    Wv, Xcv = F.bf16_bits_to_f64(d["W"]), F.bf16_bits_to_f64(d["Xc"])
    sW, sX = P.second_moment_sums(Wv, g), P.second_moment_sums(Xcv, g)
    args = (dev(sW.astype(np.float32)), Wv.shape[0], dev(sX.astype(np.float32)), Xcv.shape[0], g, 0.01)
    Tw, _, info_w = wush.build_transforms(*args)
    Ts, Tsinv, info_s = wush.build_transforms(*args, kind="wus")
    _sync()
    assert int(info_w.abs().max().item()) == 0 and int(info_s.abs().max().item()) == 0
    Tw, Ts, Tsinv = Tw.double().cpu().numpy(), Ts.double().cpu().numpy(), Tsinv.double().cpu().numpy()
    H = WT.hadamard(g)
    C = K // g
    for c in range(C):
        scale = np.abs(Tw[c]).max()
        assert np.allclose(H @ Ts[c], Tw[c], atol=2.0 ** -6 * scale * np.sqrt(g))     # two bf16 roundings apart
        assert np.allclose(Tsinv[c] @ Ts[c].T, np.eye(g), atol=1e-5)                  # Eq. 6 on the stored values
        To = WT.variant_transform("WUS", sW[c] / Wv.shape[0], sX[c] / Xcv.shape[0], 0.01)
        assert np.allclose(Ts[c], To, atol=2.0 ** -7 * np.abs(To).max() + 1e-12, rtol=2.0 ** -7)
    # inverse-transpose of arbitrary (here: random, well conditioned) bf16 transforms
    rng = np.random.default_rng(g)
    A = np.eye(g)[None] + 0.2 * rng.standard_normal((C, g, g))
    Ab = F.f64_to_bf16_bits(A)
    Tinv, info = wush.invert_transforms(dev_bf16(Ab), g)
    _sync()
    assert int(info.abs().max().item()) == 0
    Av = F.bf16_bits_to_f64(Ab)
    ref = np.stack([np.linalg.inv(Av[c]).T for c in range(C)])
    assert np.allclose(Tinv.double().cpu().numpy(), ref, rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_linear_captured_in_a_cuda_graph_matches_the_eager_call(fmt):
    """The whole layer (two kernels chained by programmatic dependent launch) is capturable: three steps
    captured in one graph and replayed twice give bit-identical outputs to the eager call."""
    d, L = _layer(1, fmt, M=300, N=520, K=1024, B=256)
    W, X = dev_bf16(d["W"]), dev_bf16(d["X"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED)
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    T = dev_bf16(L.T_bits)
    Y0, wsp0 = wush.linear(X, T, wq, ws, fmt, tsx, tsw)
    _sync()
    outs = [torch.zeros_like(Y0) for _ in range(3)]
    wsps = [torch.empty_like(wsp0) for _ in range(3)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(3):
                wush.linear(X, T, wq, ws, fmt, tsx, tsw, out=outs[i], workspace=wsps[i])
        for _ in range(2):
            graph.replay()
        side.synchronize()
    for i in range(3):
        assert wush.linear_status(wsps[i], 300, 1024, G[fmt]) == 0
        assert torch.equal(outs[i], Y0)

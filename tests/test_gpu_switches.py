"""GPU parity of the two optional quantiser rules against the oracle, through the C ABI:
the MXFP4 ceil rule ("mxfp4_ceil") and the per-batch NVFP4 activation tensor scale.
Same tolerances as the main parity tests.  Also here: the exhaustive check of the branch-free
division and the error path of a bounded wait that runs out."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import synth, wush
from parity_util import compare_quantized, dev, dev_bf16, rel_fro, untile

pytestmark = pytest.mark.gpu


def _layer(idx, fmt, M=None, N=None, K=None, B=None):
    d = synth.layer_inputs(synth.CONFIGS[idx], M=M, N=N, K=K, B=B)
    return d, P.PreparedLayer(d["W"], d["Xc"], fmt)


# ------------------------------------------------------------------ MXFP4, ceil rule
@pytest.mark.parametrize("sf", [wush.SF_LINEAR, wush.SF_TILED])
def test_ceil_rule_quantize_f32_bit_exact(sf):
    rng = np.random.default_rng(21)
    R, K = 333, 512
    v = (rng.standard_normal((R, K)) * np.exp(rng.uniform(-20, 20, (R, K // 32, 1)).repeat(32, 2).reshape(R, K))).astype(np.float32)
    v[0, :32] = 0.0
    v[1, :32] = 0; v[1, 0] = 48.0                                        # AbsMax = 6 * 2^3 exactly: e = 3
    v[2, :32] = 0; v[2, 5] = -np.nextafter(np.float32(48.0), np.float32(np.inf))   # one ulp above: e = 4
    v[3, :32] = np.float32(2.0 ** 5) * (1 - 2.0 ** -24)
    v[4, :32] = 1e-38
    v[5, :32] = 3e38
    v[6, :32] = 0; v[6, :7] = [6, 5, 3.5, 2.5, 1.75, 0.75, 0.25]         # exact ties at scale 1
    codes, scales = wush.quantize_f32(dev(v), "mxfp4_ceil", None, sf)
    torch.cuda.synchronize()
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, R, K // 32)
    compare_quantized(codes.cpu().numpy(), sc, v, "mxfp4_ceil", None, strict=True)
    # and it differs from the floor rule where it should
    _, sc_floor = Q.quantize(v, "mxfp4")
    assert 0.2 < np.mean(sc != sc_floor) < 0.8


@pytest.mark.parametrize("M,K,sf", [(128, 2048, wush.SF_TILED), (77, 192, wush.SF_LINEAR), (300, 1024, wush.SF_LINEAR), (1, 64, wush.SF_TILED)])
def test_ceil_rule_quantize_act_parity(M, K, sf):
    d, L = _layer(1, "mxfp4_ceil", M=M, N=64, K=K, B=256)
    codes, scales = wush.quantize_act(dev_bf16(d["X"]), dev_bf16(L.T_bits), "mxfp4_ceil", None, sf)
    torch.cuda.synchronize()
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, M, K // 32)
    v32, _, _ = L.quantize_act(d["X"])
    stats = compare_quantized(codes.cpu().numpy(), sc, v32, "mxfp4_ceil")
    assert stats["flipped_codes"] <= stats["guarded_elems"]


def test_ceil_rule_weights_and_whole_layer():
    d, L = _layer(1, "mxfp4_ceil", M=260, N=520, K=1024, B=256)
    W, X = dev_bf16(d["W"]), dev_bf16(d["X"])
    wq, ws, _ = wush.quantize_weight(W, dev(L.T_xvsh32), "mxfp4_ceil", sf=wush.SF_LINEAR)
    torch.cuda.synchronize()
    compare_quantized(wq.cpu().numpy(), ws.cpu().numpy(), L.wbar32, "mxfp4_ceil")
    wq, ws, _ = wush.quantize_weight(W, dev(L.T_xvsh32), "mxfp4_ceil", sf=wush.SF_TILED)
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, "mxfp4_ceil")
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, 260, 1024, 32) == 0
    assert rel_fro(Y.cpu().numpy(), L.forward(d["X"])) <= 1e-3
    # the GEMM does not care which rule produced its operands
    xq, xs = wush.quantize_act(X, dev_bf16(L.T_bits), "mxfp4_ceil", None, wush.SF_TILED)
    Y2, st = wush.gemm_fp4(xq, xs, wq, ws, 1024, "mxfp4")
    torch.cuda.synchronize()
    assert int(st[0].item()) == 0 and torch.equal(Y, Y2)


# ------------------------------------------------------------------ NVFP4, per-batch tensor scale
@pytest.mark.parametrize("M,K,sf", [(128, 2048, wush.SF_TILED), (77, 320, wush.SF_LINEAR), (531, 1024, wush.SF_TILED), (16, 64, wush.SF_LINEAR)])
def test_dynamic_scale_quantize_act_parity(M, K, sf):
    d, L = _layer(2, "nvfp4", M=M, N=64, K=K, B=256)
    codes, scales, ts = wush.quantize_act_dynamic(dev_bf16(d["X"]), dev_bf16(L.T_bits), sf)
    torch.cuda.synchronize()
    ts_o = L.dynamic_ts_x(d["X"])
    ts_g, amax_g = (float(x) for x in ts.cpu().numpy()[:2])
    assert abs(ts_g - float(ts_o)) <= 2e-7 * float(ts_o)
    assert np.float32(ts_g) == np.float32(np.float32(amax_g) / np.float32(2688.0))
    sc = scales.cpu().numpy()
    if sf == wush.SF_TILED:
        sc = untile(sc, M, K // 16)
    v32, _, _ = L.quantize_act(d["X"], ts_o)
    compare_quantized(codes.cpu().numpy(), sc, v32, "nvfp4", ts_o)
    assert sc.max() == 0x7E                                   # the AbsMax block uses the top E4M3 scale


@pytest.mark.parametrize("M,N,K", [(77, 136, 320), (300, 520, 1024), (1, 64, 64)])
def test_dynamic_scale_whole_layer(M, N, K):
    d, L = _layer(2, "nvfp4", M=M, N=N, K=K, B=256)
    W, X = dev_bf16(d["W"]), dev_bf16(d["X"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), "nvfp4", sf=wush.SF_TILED)
    Y, wsp = wush.linear(X, dev_bf16(L.T_bits), wq, ws, "nvfp4", None, tsw)          # no x_tensor_scale: per batch
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, K, 16) == 0
    ts_g, _ = wush.linear_dynamic_scale(wsp, M, K, 16)
    ts_o = float(L.dynamic_ts_x(d["X"]))
    assert abs(ts_g - ts_o) <= 2e-7 * ts_o
    assert rel_fro(Y.cpu().numpy(), L.forward(d["X"], dynamic=True)) <= 1e-3
    # a batch far outside the calibration range: the static scale clips, the per-batch one does not
    big = F.f64_to_bf16_bits(F.bf16_bits_to_f64(d["X"]) * 128.0)
    Yb, wsp = wush.linear(dev_bf16(big), dev_bf16(L.T_bits), wq, ws, "nvfp4", None, tsw, workspace=wsp)
    torch.cuda.synchronize()
    assert rel_fro(Yb.cpu().numpy(), L.forward(big, dynamic=True)) <= 1e-3
    # second call on the same workspace, same input: identical (nothing is left over between calls)
    Yb2, _ = wush.linear(dev_bf16(big), dev_bf16(L.T_bits), wq, ws, "nvfp4", None, tsw, workspace=wsp)
    torch.cuda.synchronize()
    assert torch.equal(Yb, Yb2)


def test_dynamic_scale_all_zero_batch():
    d, L = _layer(2, "nvfp4", M=40, N=64, K=128, B=256)
    X = torch.zeros(40, 128, dtype=torch.bfloat16, device="cuda")
    codes, scales, ts = wush.quantize_act_dynamic(X, dev_bf16(L.T_bits), wush.SF_LINEAR)
    torch.cuda.synchronize()
    assert float(ts[0].item()) == 1.0 and float(ts[1].item()) == 0.0
    assert int(codes.max().item()) == 0 and int(scales.max().item()) == 0


# ------------------------------------------------------------------ the NVFP4 scale path's division
def test_branch_free_division_equals_ieee_division_for_every_x():
    """The scale byte must come from correctly rounded divisions.  The kernels' branch-free form is compared
    on the device with the IEEE division for every fp32 x in [2^-60, 2^60] and for: 6, the tensor scales of
    the synthetic layers, significands of all ones / one ulp above a power of two, and seeded random divisors
    across the guarded exponent range."""
    rng = np.random.default_rng(3)
    divs = [6.0, 1.0, 0.0371, 2688.0]
    for idx in (2, 4, 5):
        d = synth.layer_inputs(synth.CONFIGS[idx], M=64, N=64)
        L = P.PreparedLayer(d["W"], d["Xc"], "nvfp4")
        divs += [float(L.ts_x), float(L.ts_w), float(L.dynamic_ts_x(d["X"]))]
    bits = []
    for e in (-40, -17, -1, 0, 1, 23, 40):
        for m in (0x7FFFFF, 0x7FFFFE, 0x000001, 0x400000, 0x3FFFFF, 0x2AAAAB):
            bits.append(((127 + e) << 23) | m)
    bits += [int(((127 + int(rng.integers(-40, 41))) << 23) | int(rng.integers(0, 1 << 23))) for _ in range(64)]
    divs = np.concatenate([np.array(divs, dtype=np.float32), np.array(bits, dtype=np.uint32).view(np.float32)])
    bad = wush.check_division(dev(divs))
    torch.cuda.synchronize()
    assert int(bad.abs().max().item()) == 0, [(float(divs[i]), int(b)) for i, b in enumerate(bad.cpu().tolist()) if b]


def test_static_tensor_scale_of_calibration_tokens():
    """wush_act_tensor_scale: AbsMax of the transformed calibration tokens within the transform's tolerance of
    the oracle's, and the scale is exactly that AbsMax / 2688 in fp32 - the oracle's static ts_x."""
    d, L = _layer(1, "nvfp4", M=16, N=256, K=1024, B=700)
    out = wush.act_tensor_scale(dev_bf16(d["Xc"]), dev_bf16(L.T_bits), 16).cpu().numpy()
    amax_o = np.float32(L.ts_x) * np.float32(2688.0)
    assert abs(out[1] - amax_o) <= 1e-5 * amax_o
    assert out[0] == np.float32(out[1]) / np.float32(2688.0)
    assert abs(out[0] - L.ts_x) <= 1e-5 * L.ts_x


# ------------------------------------------------------------------ error path: a bounded wait that runs out
def test_expired_wait_is_reported_and_the_next_call_works():
    """The test hook leaves one tile of the quantiser unrequested: the consumers' bounded wait for it
    (about a second) expires, the status word names the quantiser's consumer role, both kernels of the call
    still complete, nothing faults, and the same call repeated without the hook gives the oracle's result."""
    fmt, M, N, K = "mxfp4", 300, 520, 1024
    d, L = _layer(1, fmt, M=M, N=N, K=K, B=256)
    X, W = dev_bf16(d["X"]), dev_bf16(d["W"])
    wq, ws, tsw = wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED)
    T = dev_bf16(L.T_bits)
    wush.debug_drop_tile(0)
    Y, wsp = wush.linear(X, T, wq, ws, fmt, None, tsw)
    torch.cuda.synchronize()
    word = wush.linear_status(wsp, M, K, 32)
    assert word != 0 and (word >> 16) in (0x04, 0x05, 0x06, 0x07, 0x08), hex(word)     # a role of the quantiser
    assert wush.decode_status(word) == wush.lib().wush_decode_status(1) != 0      # WUSH_ERR_TIMEOUT
    assert wush.decode_status(0) == 0
    Y, wsp = wush.linear(X, T, wq, ws, fmt, None, tsw)                           # the hook was for one call
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, K, 32) == 0
    assert rel_fro(Y.cpu().numpy(), L.forward(d["X"])) <= 1e-3


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_one_workspace_serves_every_call(fmt):
    """wush_workspace_bytes(M, N, K, fmt, g): a single buffer of that size is enough for the moments of W and of the
    calibration tokens, the weight quantiser and the online layer, and the layer's result is the oracle's."""
    g = 32 if fmt == "mxfp4" else 16
    M, N, K, B = 300, 520, 1024, 512
    d, L = _layer(2, fmt, M=M, N=N, K=K, B=B)
    need = wush.workspace_bytes(M, N, K, fmt)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    W, Xc, X = dev_bf16(d["W"]), dev_bf16(d["Xc"]), dev_bf16(d["X"])
    mom_w, cnt_w = wush.calib_moments(W, g, workspace=ws)
    mom_x, cnt_x = wush.calib_moments(Xc, g, workspace=ws)
    torch.cuda.synchronize()
    S = P.second_moment_sums(F.bf16_bits_to_f64(d["W"]), g)
    assert rel_fro(mom_w.cpu().numpy(), S) <= 1e-5 and int(cnt_w[0].item()) == N and int(cnt_x[0].item()) == B
    codes, scales = wush._alloc_q(N, K, g, wush.SF_TILED, W.device)
    tsw = torch.zeros(4, dtype=torch.float32, device="cuda") if fmt == "nvfp4" else None
    wush.quantize_weight(W, dev(L.T_xvsh32), fmt, sf=wush.SF_TILED, out=(codes, scales, tsw, ws))
    tsx = dev(np.full(4, L.ts_x, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, _ = wush.linear(X, dev_bf16(L.T_bits), codes, scales, fmt, tsx, tsw, workspace=ws)
    torch.cuda.synchronize()
    assert wush.linear_status(ws, M, K, g) == 0
    assert rel_fro(Y.cpu().numpy(), L.forward(d["X"])) <= 1e-3

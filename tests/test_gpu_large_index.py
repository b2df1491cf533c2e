"""Sizes beyond 2^31 elements: every kernel of the online path and the moments kernel address their operands with
64-bit offsets.  X has 262344 x 8192 = 2.15e9 entries (4.3 GB of bf16), so element offsets pass 2^31 at row 262144
and the packed codes pass 2^30 bytes at the same row; 262344 is not a multiple of 128, so the last row block of
both the quantiser and the GEMM is ragged.

The oracle cannot afford the whole matrix.  Token rows are independent (Eq. 7), so sampled rows - the first ones,
the rows on either side of the 2^30 / 2^31 element boundaries and the last ones - are checked in full: codes and
scale bytes against the oracle's quantiser (guard-band rule), Y against the fp64 product of the dequantised
operands.  For the moments (Algorithm 2, first step) the property that holds at any size is additivity over row
ranges: the sum over all rows equals the sum of two halves that are each below 2^31 elements, a size at which the
kernel is compared with the oracle elsewhere.
"""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import pipeline as P
from oracle import quantizers as Q
from paper_2512_00956_b200 import wush
from parity_util import compare_quantized, dev, dev_bf16, rel_fro, tile, untile

pytestmark = pytest.mark.gpu
G = Q.GROUP
M, K, N = 262344, 8192, 256


def _big_x():
    gen = torch.Generator(device="cuda")
    gen.manual_seed(20251201)
    X = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, M, 32768):                     # in slices: the fp32 draw of the whole matrix would be 8.6 GB
        r1 = min(M, r0 + 32768)
        X[r0:r1] = (torch.randn((r1 - r0, K), generator=gen, device="cuda") * 0.8).to(torch.bfloat16)
    return X


def _rows():
    rng = np.random.default_rng(3)
    fixed = [0, 1, 127, 128, 131071, 131072, 131073, 262143, 262144, 262145, 262271, 262272, M - 2, M - 1]
    return np.unique(np.concatenate([np.array(fixed), rng.choice(M, size=34, replace=False)]))


@pytest.mark.parametrize("fmt", ["mxfp4", "nvfp4"])
def test_online_layer_beyond_2_31_elements(fmt):
    g = G[fmt]
    rng = np.random.default_rng(11)
    X = _big_x()
    T_bits = F.f64_to_bf16_bits(rng.standard_normal((K // g, g, g)) / np.sqrt(g))
    wc = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    if fmt == "mxfp4":
        wsb = rng.integers(121, 132, size=(N, K // g), dtype=np.uint8)
    else:
        wsb = rng.integers(0x28, 0x50, size=(N, K // g), dtype=np.uint8)
    ts = 0.0123 if fmt == "nvfp4" else None
    tsd = dev(np.full(4, ts, dtype=np.float32)) if fmt == "nvfp4" else None
    Y, wsp = wush.linear(X, dev_bf16(T_bits), dev(F.pack_e2m1(wc)), dev(tile(wsb)), fmt, tsd, tsd)
    torch.cuda.synchronize()
    assert wush.linear_status(wsp, M, K, g) == 0
    rows = _rows()
    sel = torch.from_numpy(rows).cuda()
    X_bits = X[sel].view(torch.int16).cpu().numpy().view(np.uint16)
    codes = wsp[: M * K // 2].view(M, K // 2)[sel].cpu().numpy()
    off = (M * K // 2 + 15) // 16 * 16
    nsb = wush.scale_bytes(M, K, g, wush.SF_TILED)
    sc = untile(wsp[off: off + nsb].cpu().numpy(), rows, K // g)
    v32, _, _ = P.quantize_transformed(F.bf16_bits_to_f64(X_bits), F.bf16_bits_to_f64(T_bits), fmt, ts)
    compare_quantized(codes, sc, v32, fmt, ts)
    # the GEMM on what the quantiser wrote: exact operands, so the product is compared tightly
    xd = Q.dequantize(F.unpack_e2m1(codes), sc, fmt, ts)
    Yo = P.dequantized_product(xd, Q.dequantize(wc, wsb, fmt, ts))
    assert rel_fro(Y[sel].cpu().numpy(), Yo) <= 1e-5
    del Y, wsp, X
    torch.cuda.empty_cache()


def test_moments_are_additive_beyond_2_31_elements():
    g = 32
    X = _big_x()
    half = 131072                                      # 2^30 elements: each part is addressed with small offsets too
    full, cnt = wush.calib_moments(X, g)
    a, ca = wush.calib_moments(X[:half], g)
    b, cb = wush.calib_moments(X[half:], g)
    torch.cuda.synchronize()
    assert int(cnt[0].item()) == M and int(ca[0].item()) + int(cb[0].item()) == M
    want = a.double() + b.double()
    err = (full.double() - want).abs().max().item()
    assert err <= 1e-5 * want.abs().max().item()
    # and the second half alone against the oracle on a block it can afford: 64 channels of the last 4096 rows
    rows = X[M - 4096:, :64].contiguous()
    part, _ = wush.calib_moments(X[M - 4096:], g)
    torch.cuda.synchronize()
    ref = P.second_moment_sums(F.bf16_bits_to_f64(rows.view(torch.int16).cpu().numpy().view(np.uint16)), g)
    assert np.max(np.abs(part[:2].double().cpu().numpy() - ref)) <= 1e-5 * np.max(np.abs(ref))
    del X
    torch.cuda.empty_cache()

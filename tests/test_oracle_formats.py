"""Pins for the oracle's number formats and block quantisers (CPU only).

Each codec is compared with something that is not itself: the ml_dtypes library's
independent implementations, brute-force nearest-neighbour search over the grid,
the format definitions' worked values, and the stored E2M1 grid.
"""
import os
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest

from oracle import formats as F
from oracle import quantizers as Q

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _grid_from_file():
    rows = [l.split() for l in open(os.path.join(GOLD, "e2m1_grid.txt")) if l.strip() and l[0] != "#"]
    return np.array([float(v) for _, v in rows])


def test_e2m1_grid_matches_golden_and_ml_dtypes():
    grid = _grid_from_file()
    assert np.array_equal(F.E2M1_GRID, grid)
    all_codes = np.arange(16, dtype=np.uint8)
    lib = all_codes.view(ml_dtypes.float4_e2m1fn).astype(np.float64)
    assert np.array_equal(F.e2m1_decode(all_codes), lib)
    assert np.array_equal(F.e2m1_decode(all_codes)[8:], -grid)


def test_e2m1_roundtrip_all_codes():
    c = np.arange(16, dtype=np.uint8)
    assert np.array_equal(F.e2m1_encode(F.e2m1_decode(c)), c)       # incl. -0 -> 0x8


def _brute_force_e2m1(u):
    grid = _grid_from_file()
    out = np.empty(u.shape, dtype=np.uint8)
    for i, x in enumerate(u):
        mag = min(abs(float(x)), 6.0)
        dist = [abs(Fraction(mag) - Fraction(gv)) for gv in grid]
        best = min(dist)
        cands = [k for k, dv in enumerate(dist) if dv == best]
        k = cands[0] if len(cands) == 1 else [k for k in cands if k % 2 == 0][0]
        out[i] = k | (8 if np.signbit(x) else 0)
    return out


def test_e2m1_encode_brute_force_and_midpoints():
    rng = np.random.default_rng(0)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32)
    near = np.concatenate([mids, np.nextafter(mids, np.float32(10)), np.nextafter(mids, np.float32(-10))])
    u = np.concatenate([near, -near, rng.uniform(-8, 8, 4000).astype(np.float32),
                        np.float32([0.0, -0.0, 6.0, 6.5, 1e30, -1e30, 1e-30, -1e-30])])
    assert np.array_equal(F.e2m1_encode(u), _brute_force_e2m1(u))
    # ties go to the even code: values 0, 1, 1, 2, 2, 4, 4
    assert np.array_equal(F.e2m1_decode(F.e2m1_encode(mids)), [0, 1, 1, 2, 2, 4, 4])


def test_e2m1_encode_matches_ml_dtypes_cast():
    rng = np.random.default_rng(1)
    u = rng.uniform(-6, 6, 20000).astype(np.float32)
    lib = u.astype(ml_dtypes.float4_e2m1fn).view(np.uint8) & 0xF
    assert np.array_equal(F.e2m1_encode(u), lib)
    assert F.e2m1_encode(np.float32([np.nan]))[0] == 7


def test_pack_order_low_nibble_first():
    codes = np.array([[1, 2, 0xF, 0]], dtype=np.uint8)
    p = F.pack_e2m1(codes)
    assert p.tolist() == [[0x21, 0x0F]]
    assert np.array_equal(F.unpack_e2m1(p), codes)


def test_e8m0_decode():
    b = np.arange(0, 255, dtype=np.uint8)
    lib = b.view(ml_dtypes.float8_e8m0fnu).astype(np.float64)
    assert np.array_equal(F.e8m0_decode(b), lib)
    assert F.e8m0_decode(127) == 1.0 and F.e8m0_decode(0) == 2.0 ** -127


def test_e4m3_decode_table_matches_ml_dtypes():
    b = np.arange(256, dtype=np.uint8)
    lib = b.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    mine = F.e4m3_decode(b)
    assert np.array_equal(np.isnan(mine), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(mine[ok], lib[ok])
    assert F.e4m3_decode(0x7E) == 448.0 and F.e4m3_decode(0x38) == 1.0 and F.e4m3_decode(0x01) == 2.0 ** -9


def test_e4m3_encode_roundtrip_and_ml_dtypes():
    b = np.arange(0, 0x7F, dtype=np.uint8)
    assert np.array_equal(F.e4m3_encode_satfinite(F.e4m3_decode(b)), b)
    rng = np.random.default_rng(2)
    r = np.concatenate([np.exp(rng.uniform(np.log(2.0 ** -12), np.log(448.0), 50000)),
                        np.float64([0.0, 2.0 ** -10, 2.0 ** -9, 1.5 * 2.0 ** -9, 2.0 ** -6, 448.0])]).astype(np.float32)
    lib = r.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(F.e4m3_encode_satfinite(r), lib)
    # exact midpoints between neighbouring codes go to the even code
    vals = F.e4m3_decode(b)
    mid = (vals[:-1] + vals[1:]) / 2
    enc = F.e4m3_encode_satfinite(mid)
    assert np.all(enc % 2 == 0) and np.all((enc == b[:-1]) | (enc == b[1:]))
    # saturation: above 448 -> 448, never NaN
    assert F.e4m3_encode_satfinite(np.float64([449.0, 464.0, 480.0, 1e9, np.inf])).tolist() == [0x7E] * 5


def test_bf16_rounding_matches_ml_dtypes_and_is_single_rounding():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(50000) * np.exp(rng.uniform(-30, 30, 50000)), [0.0, -0.0, 1.0, 1e-40]])
    lib = x.astype(ml_dtypes.bfloat16).view(np.uint16)      # direct fp64 -> bf16 cast
    assert np.array_equal(F.f64_to_bf16_bits(x), lib)
    # a value that double rounding (fp64 -> fp32 -> bf16) would get wrong
    y = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert F.round_to_bf16(y) == 1.0 + 2.0 ** -7
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    assert np.array_equal(F.f64_to_bf16_bits(F.bf16_bits_to_f64(bits)), bits)


# ------------------------------------------------------------------ block quantisers
def test_mxfp4_worked_blocks():
    blk = np.zeros((1, 32), dtype=np.float32)
    blk[0, :4] = [6, 3, 1, 0.5]
    codes, sc = Q.quantize_mxfp4(blk)
    assert sc[0, 0] == 127 + 0 and np.array_equal(Q.dequantize_mxfp4(codes, sc), blk)      # floor(log2 6)-2 = 0
    ones = np.ones((1, 32), dtype=np.float32)
    codes, sc = Q.quantize_mxfp4(ones)
    assert sc[0, 0] == 127 - 2 and np.all(codes == 6)                                        # u = 4 -> code 6
    assert np.array_equal(Q.dequantize_mxfp4(codes, sc), ones)
    k = 5
    blk = np.full((1, 32), np.nextafter(np.float32(2.0 ** k), np.float32(0)), dtype=np.float32)
    codes, sc = Q.quantize_mxfp4(blk)
    assert sc[0, 0] == 127 + k - 3 and np.all(codes == 7)                                    # just under 2^k: saturates
    z = np.zeros((1, 32), dtype=np.float32)
    codes, sc = Q.quantize_mxfp4(z)
    assert sc[0, 0] == 0 and np.all(codes == 0)


def test_mxfp4_scale_rule_properties():
    rng = np.random.default_rng(4)
    v = (rng.standard_normal((64, 256)) * np.exp(rng.uniform(-20, 20, (64, 1)))).astype(np.float32)
    codes, sc = Q.quantize_mxfp4(v)
    amax = np.abs(v.reshape(64, 8, 32)).max(axis=2).astype(np.float64)
    ratio = amax / F.e8m0_decode(sc)
    assert np.all((ratio >= 4) & (ratio < 8))
    deq = Q.dequantize_mxfp4(codes, sc)
    assert np.all(np.abs(deq).reshape(64, 8, 32).max(axis=2) <= 6 * F.e8m0_decode(sc))
    # elementwise error: half a grid step (<= 1 * scale above 4, 0.5 below ...) unless clamped
    u = v.reshape(64, 8, 32) / F.e8m0_decode(sc)[:, :, None]
    err = np.abs(deq.reshape(64, 8, 32) / F.e8m0_decode(sc)[:, :, None] - u)
    assert np.all(err[np.abs(u) <= 6] <= 1.0 + 1e-12)
    assert np.all(err[np.abs(u) <= 2] <= 0.25 + 1e-12)


def test_mxfp4_ceil_rule_is_the_smallest_non_saturating_exponent():
    """Exact rationals: e is the least integer with AbsMax <= 6 * 2^e (nothing clamps, nothing is wasted),
    it is the floor-rule exponent or one more, and the two rules agree exactly when AbsMax / 2^e_floor <= 6."""
    rng = np.random.default_rng(14)
    a = np.abs(rng.standard_normal(4000) * np.exp(rng.uniform(-30, 30, 4000))).astype(np.float32)
    edge = np.float32([6.0, 3.0, 1.5, 0.75, 4.0, 8.0, 12.0, 96.0])           # on and around the decision boundaries
    edge = np.concatenate([edge, np.nextafter(edge, np.float32(0)), np.nextafter(edge, np.float32(np.inf))])
    a = np.concatenate([a, edge]).astype(np.float32)
    e_c = Q.mx_shared_exponent(a, "ceil")
    e_f = Q.mx_shared_exponent(a, "floor")
    for x, ec, ef in zip(a, e_c, e_f):
        fx = Fraction(float(x))
        assert fx <= 6 * Fraction(2) ** int(ec) and fx > 6 * Fraction(2) ** (int(ec) - 1)
        assert ec - ef == (1 if fx > 6 * Fraction(2) ** int(ef) else 0)
    # whole quantiser: no element saturates, so every element is within half a grid step of its value
    v = (rng.standard_normal((32, 128)) * np.exp(rng.uniform(-10, 10, (32, 1)))).astype(np.float32)
    codes, sc = Q.quantize(v, "mxfp4_ceil")
    u = v.reshape(32, 4, 32) / F.e8m0_decode(sc)[:, :, None]
    assert np.abs(u).max() <= 6.0 and np.all(np.abs(u).max(axis=2) > 3.0)
    deq_u = Q.dequantize(codes, sc, "mxfp4_ceil").reshape(32, 4, 32) / F.e8m0_decode(sc)[:, :, None]
    assert np.all(np.abs(deq_u - u) <= 1.0 + 1e-12) and np.all(np.abs(deq_u - u)[np.abs(u) <= 2] <= 0.25 + 1e-12)
    # worked blocks: AbsMax 6 -> e = 0 under both rules; AbsMax 7 -> floor keeps e = 0 and clamps, ceil takes e = 1
    blk = np.zeros((1, 32), dtype=np.float32); blk[0, 0] = 7.0; blk[0, 1] = 1.0
    cf, sf = Q.quantize(blk, "mxfp4"); cc, sc2 = Q.quantize(blk, "mxfp4_ceil")
    assert sf[0, 0] == 127 and Q.dequantize(cf, sf, "mxfp4")[0, 0] == 6.0
    assert sc2[0, 0] == 128 and Q.dequantize(cc, sc2, "mxfp4_ceil")[0, 0] == 8.0 and Q.dequantize(cc, sc2, "mxfp4_ceil")[0, 1] == 1.0
    z = np.zeros((1, 32), dtype=np.float32)
    assert Q.quantize(z, "mxfp4_ceil")[1][0, 0] == 0


def test_nvfp4_worked_block_and_tensor_scale():
    blk = np.zeros((1, 16), dtype=np.float32)
    blk[0, :4] = [6, -3, 1, 0.5]
    big = np.concatenate([blk, np.full((1, 16), 2688.0, dtype=np.float32)])
    ts = Q.nvfp4_tensor_scale(big)
    assert ts == np.float32(1.0)                                   # 2688 / (6*448)
    codes, sb = Q.quantize_nvfp4(big, ts)
    assert sb[0, 0] == 0x38 and sb[1, 0] == 0x7E                   # 1.0 and 448
    assert np.array_equal(Q.dequantize_nvfp4(codes, sb, ts), big)  # both blocks lossless
    z = np.zeros((1, 16), dtype=np.float32); z[0, 3] = -0.0
    codes, sb = Q.quantize_nvfp4(z, ts)
    assert sb[0, 0] == 0 and np.all((codes & 7) == 0) and codes[0, 3] == 8
    assert Q.nvfp4_tensor_scale(np.zeros((4, 16), dtype=np.float32)) == np.float32(1.0)   # all-zero tensor: any positive scale


def test_nvfp4_matches_exact_rational_definition():
    """Recompute the fp32 step sequence with exact rationals + explicit fp32 rounding."""
    rng = np.random.default_rng(5)
    v = (rng.standard_normal((40, 16)) * np.exp(rng.uniform(-3, 3, (40, 1)))).astype(np.float32)
    ts = np.float32(0.0123)
    codes, sb = Q.quantize_nvfp4(v, ts)

    def rn32(fr):           # exact Fraction -> nearest fp32 (Python float division is correctly rounded)
        return np.float32(fr.numerator / fr.denominator) if fr.denominator != 1 else np.float32(int(fr))

    for r in range(v.shape[0]):
        a = max(abs(Fraction(float(x))) for x in v[r])
        q1 = Fraction(float(rn32(a / 6)))
        rr = Fraction(float(rn32(q1 / Fraction(float(ts)))))
        grid = [Fraction(float(x)) for x in F.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))]
        dist = [abs(rr - gq) for gq in grid]
        best = min(dist)
        cand = [k for k, dd in enumerate(dist) if dd == best]
        k = cand[0] if len(cand) == 1 else [c for c in cand if c % 2 == 0][0]
        assert sb[r, 0] == k
        d = Fraction(float(rn32(grid[k] * Fraction(float(ts)))))
        inv = Fraction(float(rn32(1 / d)))
        for j in range(16):
            u = float(rn32(Fraction(float(v[r, j])) * inv))
            assert codes[r, j] == _brute_force_e2m1(np.float32([u]))[0]


def test_nvfp4_properties():
    rng = np.random.default_rng(6)
    v = (rng.standard_normal((128, 256)) * np.exp(rng.uniform(-2, 2, (128, 1)))).astype(np.float32)
    ts = Q.nvfp4_tensor_scale(v)
    codes, sb = Q.quantize_nvfp4(v, ts)
    assert sb.max() == 0x7E                       # the block holding the tensor AbsMax uses scale 448
    deq = Q.dequantize_nvfp4(codes, sb, ts)
    rel = np.linalg.norm(deq - v) / np.linalg.norm(v)
    assert 0.02 < rel < 0.15                      # 4-bit RTN error level for Gaussian data
    # AbsMax element of each block is reproduced to within the scale's own rounding (E4M3: 2^-4 relative)
    vb, db = v.reshape(128, 16, 16), deq.reshape(128, 16, 16)
    i = np.abs(vb).argmax(axis=2)
    top_v = np.take_along_axis(vb, i[:, :, None], 2)[:, :, 0]
    top_d = np.take_along_axis(db, i[:, :, None], 2)[:, :, 0]
    assert np.all(np.abs(top_d - top_v) <= np.abs(top_v) * (2.0 ** -4 + 1e-6))


def test_table7_storage_reading():
    """One 16-bit d x d matrix per block per linear layer reproduces Table 7's overhead."""
    rows = [l.split() for l in open(os.path.join(GOLD, "table7_storage.txt")) if l.strip() and l[0] != "#"]
    want = {fmt: float(p) for _, fmt, p in rows}
    hidden, inter, layers, vocab, kv = 4096, 14336, 32, 128256, 1024
    sum_K = 4 * hidden + 2 * hidden + inter          # q,k,v,o read 4096; gate,up read 4096; down reads 14336
    lin_params = layers * (hidden * hidden * 2 + 2 * hidden * kv + 3 * hidden * inter)
    for fmt, d in (("mxfp4", 32), ("nvfp4", 16)):
        transform_bytes = layers * sum_K * d * 2
        bits_per_w = 4 + 8.0 / d
        ckpt = lin_params * bits_per_w / 8 + 2 * vocab * hidden * 2
        pct = 100 * transform_bytes / ckpt
        assert abs(pct - want[fmt]) < 0.15, (fmt, pct)

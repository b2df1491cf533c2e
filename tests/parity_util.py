"""Helpers of the GPU parity tests: device upload, the TILED scale permutation written
out independently of the library, and the guard-band comparison of codes and scales.

Guard bands (tolerance of the build target): an element is "guarded" when the oracle's
scaled value u lies within 1e-4 relative of an E2M1 rounding midpoint; a whole block is
guarded when the quantity that decides its scale byte lies within 1e-4 relative of a
decision boundary (a power of two for MXFP4, 6 times a power of two under its ceil rule; an E4M3
rounding midpoint for NVFP4).
Outside the guards codes and scale bytes must be identical; inside, one step apart at most.
"""
import numpy as np
import torch

from oracle import formats as F
from oracle import quantizers as Q

MIDS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
GUARD = 1e-4


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def tiled_offsets(rows, KB):
    """Byte offset of scale (r, kb) in the GEMM-native layout, for all kb and all r < rows (or the rows listed)."""
    r = (np.arange(rows) if np.isscalar(rows) else np.asarray(rows, dtype=np.int64))[:, None]
    kb = np.arange(KB)[None, :]
    ktiles = (KB + 3) // 4
    return ((r // 128) * ktiles + kb // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + kb % 4


def untile(buf, rows, KB):
    return np.asarray(buf)[tiled_offsets(rows, KB)]


def tile(scales):
    rows, KB = scales.shape
    out = np.zeros(((rows + 127) // 128) * ((KB + 3) // 4) * 512, dtype=np.uint8)
    out[tiled_offsets(rows, KB)] = scales
    return out


def canon(codes):
    """-0 and +0 dequantise identically: map code 0x8 to 0x0."""
    codes = np.asarray(codes).copy()
    codes[codes == 8] = 0
    return codes


def guards(v32, fmt, ts):
    """(block_guard [R,KB], elem_guard [R,K]) from the oracle's own intermediate values."""
    g = Q.GROUP[fmt]
    R, K = v32.shape
    vb = v32.reshape(R, K // g, g)
    amax = np.abs(vb).max(axis=2).astype(np.float64)
    if fmt in ("mxfp4", "mxfp4_ceil"):
        m, _ = np.frexp(np.where(amax == 0, 1.0, amax))              # m in [0.5, 1)
        if fmt == "mxfp4":
            block_guard = (m - 0.5 <= 0.5 * GUARD) | (1.0 - m <= GUARD)
        else:                                                        # the exponent steps where AbsMax = 6 * 2^k
            block_guard = np.abs(m - 0.75) <= 0.75 * GUARD
        e = Q.mx_shared_exponent(amax, "floor" if fmt == "mxfp4" else "ceil")
        u = np.ldexp(vb.astype(np.float64), (-e)[:, :, None])
    else:
        f32 = np.float32
        with np.errstate(all="ignore"):
            r = ((amax.astype(f32) / f32(6.0)).astype(f32) / f32(ts)).astype(f32).astype(np.float64)
            vals = F.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))
            mids = (vals[:-1] + vals[1:]) / 2
            idx = np.clip(np.searchsorted(mids, r), 1, len(mids) - 1)
            near = np.minimum(np.abs(r - mids[idx - 1]) / mids[idx - 1], np.abs(r - mids[idx]) / mids[idx])
            block_guard = near <= GUARD
            sb = F.e4m3_encode_satfinite(r)
            d = (F.e4m3_decode(sb).astype(f32) * f32(ts)).astype(f32)
            inv = np.where(d == 0, f32(0), f32(1.0) / d).astype(f32)
            u = (vb * inv[:, :, None]).astype(f32).astype(np.float64)
    au = np.abs(u)[..., None]
    elem_guard = np.any(np.abs(au - MIDS) <= GUARD * MIDS, axis=-1)
    return block_guard, elem_guard.reshape(R, K)


def compare_quantized(codes_gpu_packed, scales_gpu, v32_oracle, fmt, ts=None, strict=False):
    """Returns a dict of statistics and raises AssertionError on a parity violation."""
    g = Q.GROUP[fmt]
    codes_o, sc_o = Q.quantize(v32_oracle, fmt, ts)
    codes_g = F.unpack_e2m1(np.asarray(codes_gpu_packed))
    sc_g = np.asarray(scales_gpu)
    assert codes_g.shape == codes_o.shape and sc_g.shape == sc_o.shape
    cg, co = canon(codes_g), canon(codes_o)
    if strict:
        assert np.array_equal(sc_g, sc_o), f"scale mismatches: {np.count_nonzero(sc_g != sc_o)}"
        assert np.array_equal(cg, co), f"code mismatches: {np.count_nonzero(cg != co)}"
        return dict(elems=cg.size, guarded_elems=0, guarded_blocks=0)
    bguard, eguard = guards(v32_oracle, fmt, ts)
    bad_scale = (sc_g != sc_o) & ~bguard
    assert not bad_scale.any(), f"{np.count_nonzero(bad_scale)} scale bytes differ outside the guard band"
    step = np.abs(sc_g.astype(int) - sc_o.astype(int))
    assert step.max() <= 1, "scale byte more than one step away"
    block_ok = np.repeat(sc_g == sc_o, g, axis=1)                      # blocks whose scales agree
    diff = cg != co
    bad = diff & block_ok & ~eguard
    assert not bad.any(), f"{np.count_nonzero(bad)} codes differ outside the guard band"
    near = diff & block_ok & eguard
    if near.any():
        mg = (cg[near] & 7).astype(int); mo = (co[near] & 7).astype(int)
        assert np.all(np.abs(mg - mo) <= 1), "guarded code more than one step away"
    stats = dict(elems=cg.size, guarded_elems=int(eguard.sum()), guarded_blocks=int(bguard.sum()),
                 flipped_codes=int(near.sum()), flipped_scales=int((sc_g != sc_o).sum()))
    # the guard bands must stay a small exception, or the test would be vacuous
    assert stats["guarded_elems"] <= 0.01 * cg.size + 16
    assert stats["guarded_blocks"] <= 0.01 * sc_g.size + 4
    return stats


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)

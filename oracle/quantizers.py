"""Round-to-nearest AbsMax block quantisers q(.) of the problem statement.

Test infrastructure (see the package docstring).  Sec. 3 ("Block-independent
constraint") fixes q as round-to-nearest with one AbsMax scale per group of d
consecutive input channels, and Sec. 6 names the two instances measured on the
GPU path: MXFP4 (d = 32, E2M1 elements, E8M0 scale) and NVFP4 (d = 16, E2M1
elements, E4M3 scale, one fp32 scale per tensor).  The paper does not spell the
quantisers out; the step order below is this build's reading and is what the
CUDA kernels are compared against.

Both quantisers are defined on fp32 inputs (the transform result is rounded to
fp32 first) so that "bit-exact" has a meaning.
"""
import numpy as np

from . import formats as F

F32 = np.float32


def _blocks(v, g):
    v = np.asarray(v)
    if v.ndim != 2 or v.shape[1] % g != 0:
        raise ValueError("expected [rows, K] with K a multiple of the group size")
    return v.reshape(v.shape[0], v.shape[1] // g, g)


# ----------------------------------------------------------------------------- MXFP4
def mx_shared_exponent(amax, rule="floor"):
    """E8M0 exponent e of a block with AbsMax ``amax``.

    rule "floor" (the default of this build): e = floor(log2 amax) - 2.  2 is the
    exponent of the largest power of two E2M1 represents (4 = 2^2), so amax / 2^e
    lies in [4, 8); values in (6, 8) saturate to 6.
    rule "ceil": e = ceil(log2(amax / 6)), the smallest exponent for which no element
    of the block saturates (amax / 2^e in (3, 6]).  With amax = m * 2^ex, m in
    [0.5, 1), amax / 6 = (m / 0.75) * 2^(ex - 3) and m / 0.75 lies in [2/3, 4/3): the
    ceiling is ex - 3 when m <= 0.75 and ex - 2 otherwise - no logarithm is evaluated.
    Either way the exponent is clamped to [-127, 127]; an all-zero block gets -127.
    """
    amax = np.asarray(amax, dtype=np.float64)
    m, ex = np.frexp(amax)                   # amax = m * 2^ex, m in [0.5,1): floor(log2) = ex-1
    if rule == "floor":
        e = ex - 1 - 2
    elif rule == "ceil":
        e = ex - 3 + (m > 0.75)
    else:
        raise ValueError(rule)
    e = np.clip(e, -127, 127)
    return np.where(amax == 0, -127, e).astype(np.int64)


def quantize_mxfp4(v32, rule="floor"):
    """fp32 [R, K] -> (codes uint8 [R, K] unpacked, scale bytes uint8 [R, K/32])."""
    v32 = np.asarray(v32, dtype=F32)
    vb = _blocks(v32, 32).astype(np.float64)
    amax = np.max(np.abs(vb), axis=2)
    e = mx_shared_exponent(amax, rule)
    u = np.ldexp(vb, (-e)[:, :, None])       # exact power-of-two scaling
    codes = F.e2m1_encode(u).reshape(v32.shape)
    return codes, (e + 127).astype(np.uint8)


def dequantize_mxfp4(codes, scale_bytes):
    c = _blocks(codes, 32)
    return (F.e2m1_decode(c) * F.e8m0_decode(scale_bytes)[:, :, None]).reshape(np.shape(codes))


# ----------------------------------------------------------------------------- NVFP4
def nvfp4_tensor_scale(v32):
    """fp32 tensor scale: AbsMax / (6 * 448), one fp32 division; 1 for an all-zero tensor
    (every positive value then gives the same all-zero codes)."""
    amax = F32(np.max(np.abs(np.asarray(v32, dtype=F32)))) if np.size(v32) else F32(0)
    return F32(1.0) if amax == 0 else F32(amax / F32(2688.0))


def quantize_nvfp4(v32, ts):
    """fp32 [R, K], fp32 tensor scale ts > 0 -> (codes [R, K], E4M3 scale bytes [R, K/16]).

    Every operation is a single IEEE fp32 operation, round to nearest, in this
    order:  a = max|v| ; r = (a / 6) / ts ; sb = E4M3(r) ; d = float(sb) * ts ;
    inv = 1 / d ; u = v * inv ; code = E2M1(u).  A block whose d is zero gets all
    zero magnitudes (signs kept).
    """
    v32 = np.asarray(v32, dtype=F32)
    ts = F32(ts)
    vb = _blocks(v32, 16)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        a = np.max(np.abs(vb), axis=2).astype(F32)
        r = ((a / F32(6.0)).astype(F32) / ts).astype(F32)
        sb = F.e4m3_encode_satfinite(r.astype(np.float64))
        d = (F.e4m3_decode(sb).astype(F32) * ts).astype(F32)
        inv = (F32(1.0) / d).astype(F32)
        u = (vb * inv[:, :, None]).astype(F32)
    zero = (d == 0)[:, :, None]
    u = np.where(zero, np.copysign(F32(0), vb), u)
    codes = F.e2m1_encode(u.astype(np.float64)).reshape(v32.shape)
    return codes, sb


def dequantize_nvfp4(codes, scale_bytes, ts):
    c = _blocks(codes, 16)
    s = F.e4m3_decode(scale_bytes) * float(F32(ts))
    return (F.e2m1_decode(c) * s[:, :, None]).reshape(np.shape(codes))


# ----------------------------------------------------------------------------- dispatch
# "mxfp4_ceil" is MXFP4 with the non-saturating scale rule; it dequantises like "mxfp4"
GROUP = {"mxfp4": 32, "nvfp4": 16, "mxfp4_ceil": 32}


def quantize(v32, fmt, ts=None):
    if fmt == "mxfp4":
        return quantize_mxfp4(v32)
    if fmt == "mxfp4_ceil":
        return quantize_mxfp4(v32, rule="ceil")
    if fmt == "nvfp4":
        return quantize_nvfp4(v32, ts)
    raise ValueError(fmt)


def dequantize(codes, scale_bytes, fmt, ts=None):
    if fmt in ("mxfp4", "mxfp4_ceil"):
        return dequantize_mxfp4(codes, scale_bytes)
    if fmt == "nvfp4":
        return dequantize_nvfp4(codes, scale_bytes, ts)
    raise ValueError(fmt)

"""Number formats used by the W4A4 path: bf16, E2M1, E8M0, E4M3.

Test infrastructure (see the package docstring).  The paper names the block
formats (Sec. 1 and Sec. 6: MXFP4 with group 32, NVFP4 with group 16) and refers
to the OCP Microscaling and Blackwell specifications for their definition; the
encodings below follow those public format definitions:

  E2M1  sign | 2-bit exponent | 1-bit mantissa; magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6
  E8M0  unsigned power of two, value 2^(byte-127); 0xFF is NaN and never produced
  E4M3  "FN" flavour: bias 7, subnormals m*2^-9, largest finite 448, 0x7F/0xFF NaN

Everything here is exact arithmetic on fp64 numpy arrays (np.rint rounds half to
even), so each function can be checked by eye against the format definition.
"""
import numpy as np

E2M1_GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)
# Midpoint i lies between magnitude code i and i+1.
E2M1_MIDPOINTS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float64)


# ----------------------------------------------------------------------------- bf16
def bf16_bits_to_f64(bits):
    """Decode bf16 bit patterns (uint16) exactly into fp64."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round fp64 to bf16 (8 significant bits, round-half-even) in ONE rounding.

    The "16-bit transforms" of Sec. 3 ("Costs for online inference") are stored
    this way.  Going through fp32 first could round twice, so the rounding is
    done on the fp64 value directly: quantum = 2^(exponent-7), with the fp32
    subnormal floor 2^-133, then np.rint (ties to even).
    """
    x = np.asarray(x, dtype=np.float64)
    _, ex = np.frexp(x)                       # |x| = m * 2^ex, m in [0.5, 1)
    qexp = np.maximum(ex - 8, -133)           # exponent of one unit in the last place
    with np.errstate(invalid="ignore"):
        q = np.ldexp(np.rint(np.ldexp(x, -qexp)), qexp)
        q = np.where(np.abs(q) >= 2.0 ** 128, np.copysign(np.inf, x), q)
        q = np.where(np.isfinite(x), q, x)
    f32 = q.astype(np.float32)                # exact: q has 8 significant bits
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_to_bf16(x):
    """fp64 -> nearest bf16 value, returned as fp64."""
    return bf16_bits_to_f64(f64_to_bf16_bits(x))


# ----------------------------------------------------------------------------- E2M1
def e2m1_encode(u):
    """Round-to-nearest E2M1 code (0..15) of each element of ``u``.

    Nearest grid magnitude; an exact midpoint goes to the neighbour with the even
    code (mantissa bit 0); magnitudes above 6 saturate to 6; the sign bit is copied
    from ``u`` (so -0 and negatives that round to zero give 0x8); NaN gives +6
    (code 7), which is what the Blackwell conversion instruction returns.
    """
    u = np.asarray(u, dtype=np.float64)
    mag = np.abs(u)
    code = np.zeros(u.shape, dtype=np.uint8)
    for i, mid in enumerate(E2M1_MIDPOINTS):
        upper_is_even = ((i + 1) % 2 == 0)
        step = (mag > mid) | ((mag == mid) & upper_is_even)
        code += step.astype(np.uint8)
    sign = np.signbit(u).astype(np.uint8) << np.uint8(3)
    out = code | sign
    return np.where(np.isnan(u), np.uint8(7), out).astype(np.uint8)


def e2m1_decode(code):
    """E2M1 code (0..15) -> fp64 value."""
    code = np.asarray(code, dtype=np.uint8)
    mag = E2M1_GRID[code & np.uint8(7)]
    return np.where((code & np.uint8(8)) != 0, -mag, mag)


def pack_e2m1(codes):
    """[..., K] codes -> [..., K/2] bytes; element 2t in the LOW nibble of byte t."""
    codes = np.asarray(codes, dtype=np.uint8)
    return (codes[..., 0::2] | (codes[..., 1::2] << np.uint8(4))).astype(np.uint8)


def unpack_e2m1(packed):
    packed = np.asarray(packed, dtype=np.uint8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = packed & np.uint8(0x0F)
    out[..., 1::2] = packed >> np.uint8(4)
    return out


# ----------------------------------------------------------------------------- E8M0
def e8m0_decode(byte):
    """E8M0 scale byte -> 2^(byte-127) as fp64 (0xFF, NaN, is never produced here)."""
    return np.ldexp(1.0, np.asarray(byte, dtype=np.int64) - 127)


# ----------------------------------------------------------------------------- E4M3
def e4m3_decode(byte):
    """E4M3-FN byte -> fp64.  0x7F and 0xFF are NaN."""
    b = np.asarray(byte, dtype=np.uint8).astype(np.int64)
    s = (b >> 7) & 1
    e = (b >> 3) & 15
    m = b & 7
    val = np.where(e == 0, np.ldexp(m.astype(np.float64), -9),
                   np.ldexp(1.0 + m / 8.0, e - 7))
    val = np.where((b & 0x7F) == 0x7F, np.nan, val)
    return np.where(s == 1, -val, val)


def e4m3_encode_satfinite(r):
    """Non-negative fp value -> E4M3-FN byte, round-half-even, saturating at 448.

    Below the smallest normal (2^-6) the quantum is 2^-9; above, 4 significant
    bits.  A result above 448 becomes 0x7E (448); NaN becomes 0x7F.
    """
    r = np.asarray(r, dtype=np.float64)
    if np.any(r < 0):
        raise ValueError("scale codes are unsigned")
    out = np.zeros(r.shape, dtype=np.int64)
    sub = r < 2.0 ** -6
    q_sub = np.rint(np.ldexp(r, 9))                 # 0..8 ; 8 is the code of 2^-6
    m, ex = np.frexp(np.where(sub | ~np.isfinite(r), 1.0, r))
    q = np.rint(m * 16.0)                           # significand*8 in [8, 16]
    E = ex - 1
    carry = q == 16
    q = np.where(carry, 8, q)
    E = np.where(carry, E + 1, E)
    norm_code = ((E + 7).astype(np.int64) << 3) | (q.astype(np.int64) - 8)
    too_big = np.ldexp(q / 8.0, E) > 448.0
    norm_code = np.where(too_big, 0x7E, norm_code)
    q_sub = np.where(np.isfinite(q_sub), q_sub, 0)
    out = np.where(sub, q_sub.astype(np.int64), norm_code)
    out = np.where(np.isinf(r), 0x7E, out)
    out = np.where(np.isnan(r), 0x7F, out)
    return out.astype(np.uint8)

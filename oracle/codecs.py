"""Number formats and the ExpCast-FP8 map -- oracle side (test infrastructure only).

Everything here is written from the format definitions:

* E4M3 ("fn" flavour: no infinities, 0x7F/0xFF are NaN): a byte with exponent field e and
  mantissa field m decodes to 2^(e-7) (1 + m/8) for e > 0 (Sec. 3.3, the sentence before
  Eq. 7) and to (m/8) 2^-6 for e = 0 (subnormals); largest finite value 448.
* E2M1: 1 sign, 2 exponent (bias 1), 1 mantissa bit: {0, .5, 1, 1.5, 2, 3, 4, 6}.
* NVFP4 = E2M1 elements under one unsigned E4M3 microscale per 16 elements
  (App. A "Scope of ExpCast-FP8").
* bf16 = the upper 16 bits of an IEEE fp32.
* ExpCast-FP8 (Eq. 7): code(u) = clip_[0,120](Round(8 (u + 8) + 56 + beta)), Round =
  round-to-nearest-even, the byte then *viewed* as E4M3.

All encoders round to nearest, ties to even, and saturate to the largest finite value
(the behaviour of a saturating hardware convert).  Encoders never search the decode table:
they compute the binade and the step from the definition, so the exhaustive
decode -> encode identity test is a real check.
"""
import numpy as np

E4M3_MAX = 448.0
E2M1_MAX = 6.0
EXPCAST_BETA = -0.35          # Eq. 7
EXPCAST_SHIFT = 8.0           # the row maximum lands at 2^8 = 256 (Sec. 3.3)
EXPCAST_TOP_CODE = 120        # 8 * (8 + 7): byte of the value 256


# ----------------------------------------------------------------------------- bf16
def bf16_round(x):
    """Round fp32 values to the nearest bf16 (ties to even); result is fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x):
    """bf16 bit patterns (uint16) of values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)


# ----------------------------------------------------------------------------- E4M3
def e4m3_decode(code):
    """uint8 -> float64 by the format definition (NaN for 0x7F / 0xFF)."""
    code = np.asarray(code, dtype=np.uint8).astype(np.int64)
    s = (code >> 7) & 1
    e = (code >> 3) & 0xF
    m = code & 0x7
    normal = np.exp2(e.astype(np.float64) - 7.0) * (1.0 + m / 8.0)
    subnormal = (m / 8.0) * 2.0 ** -6
    mag = np.where(e == 0, subnormal, normal)
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return np.where(s == 1, -mag, mag)


def _round_to_grid(a, emin, mant_bits, amax):
    """|x| -> nearest representable magnitude of a small float format (RNE, saturating).

    emin: exponent of the lowest normal binade (its step also serves the subnormals);
    mant_bits: explicit mantissa bits.  Returns (value, q, e): value = q * 2^(e-mant_bits).
    """
    a = np.minimum(np.asarray(a, dtype=np.float64), amax)
    _, ex = np.frexp(a)                         # a = f * 2^ex with f in [0.5, 1)
    e = np.maximum(ex.astype(np.int64) - 1, emin)  # binade: 2^e <= a < 2^(e+1)
    step = np.exp2((e - mant_bits).astype(np.float64))
    q = np.rint(a / step)                       # division by a power of two is exact
    return q * step, q, e


def e4m3_encode(x):
    """float -> uint8 E4M3 code: round-to-nearest-even, saturate to +-448, keep the sign."""
    x = np.asarray(x)
    v, _, _ = _round_to_grid(np.abs(x), emin=-6, mant_bits=3, amax=E4M3_MAX)
    f, ex = np.frexp(v)                         # re-derive the fields from the rounded value
    e = ex.astype(np.int64) - 1
    mant = np.rint((f * 2.0 - 1.0) * 8.0).astype(np.int64)
    normal_code = ((e + 7) << 3) | mant
    sub_code = np.rint(v * 2.0 ** 9).astype(np.int64)   # multiples of 2^-9 below 2^-6
    code = np.where(v >= 2.0 ** -6, normal_code, sub_code)
    code = code | (np.signbit(x).astype(np.int64) << 7)
    return code.astype(np.uint8)


# ----------------------------------------------------------------------------- E2M1
def e2m1_decode(code):
    """4-bit code (bit 3 = sign) -> float64."""
    code = np.asarray(code).astype(np.int64)
    s = (code >> 3) & 1
    e = (code >> 1) & 0x3
    m = code & 0x1
    mag = np.where(e == 0, 0.5 * m, np.exp2(e.astype(np.float64) - 1.0) * (1.0 + 0.5 * m))
    return np.where(s == 1, -mag, mag)


def e2m1_encode(x):
    """float -> 4-bit E2M1 code (uint8 holding 0..15): RNE, saturate to +-6."""
    x = np.asarray(x)
    v, _, _ = _round_to_grid(np.abs(x), emin=0, mant_bits=1, amax=E2M1_MAX)
    f, ex = np.frexp(v)
    e = ex.astype(np.int64) - 1
    mant = np.rint((f * 2.0 - 1.0) * 2.0).astype(np.int64)
    normal_code = ((e + 1) << 1) | mant
    sub_code = np.rint(v * 2.0).astype(np.int64)         # 0 or 0.5
    code = np.where(v >= 1.0, normal_code, sub_code)
    code = code | (np.signbit(x).astype(np.int64) << 3)
    return code.astype(np.uint8)


# ----------------------------------------------------------------------------- ExpCast-FP8
def expcast_code(u, beta=EXPCAST_BETA):
    """Eq. 7.  u = log2-domain score minus the running row maximum (u <= 0), fp32.

    c = 8 u + (120 + beta) is one fused multiply-add in fp32 (8 u is exact), clipped to
    [0, 120], then rounded to the nearest integer, ties to even.  Clipping before or
    after the rounding gives the same byte because both bounds are integers.
    """
    u = np.asarray(u, dtype=np.float32)
    k = np.float32(8.0 * EXPCAST_SHIFT + 56.0 + beta)
    c = (np.float32(8.0) * u + k).astype(np.float32)
    c = np.clip(c, np.float32(0.0), np.float32(EXPCAST_TOP_CODE))
    return np.rint(c).astype(np.uint8)


def exp_then_cast_code(u):
    """The conventional path (Fig. 4a, upper box): p = 2^(u+8) in fp32, then cast to E4M3."""
    u = np.asarray(u, dtype=np.float32)
    p = np.exp2(u.astype(np.float64) + EXPCAST_SHIFT).astype(np.float32)
    return e4m3_encode(p)


# ----------------------------------------------------------------------------- NVFP4 groups
def nvfp4_quantize_groups(x, outer_scale=np.float32(1.0)):
    """Quantize the LAST axis of x (fp32, length divisible by 16) in groups of 16.

    Per group: sb = E4M3(max|x| * (1/(6 * outer))) is the unsigned microscale code,
    element = E2M1(x * rcp) with rcp = 1 / (outer * dec(sb)), every step one IEEE fp32
    operation.  sb = 0 zeroes the group.  Returns (codes uint8 0..15, micro uint8, deq fp64)
    where deq = dec(code) * dec(sb) (without the outer scale).
    """
    x = np.asarray(x, dtype=np.float32)
    g = x.reshape(x.shape[:-1] + (x.shape[-1] // 16, 16))
    outer = np.float32(outer_scale)
    inv6 = (np.float32(1.0) / (np.float32(6.0) * outer)).astype(np.float32)
    amax = np.max(np.abs(g), axis=-1)
    micro = e4m3_encode((amax * inv6).astype(np.float32))
    sdec = e4m3_decode(micro).astype(np.float32)
    denom = (outer * sdec).astype(np.float32)
    with np.errstate(divide="ignore"):
        rcp = np.where(sdec > 0, (np.float32(1.0) / denom).astype(np.float32), np.float32(0.0))
    y = (g * rcp[..., None]).astype(np.float32)
    codes = e2m1_encode(y)
    codes = np.where(sdec[..., None] > 0, codes, np.uint8(0)).astype(np.uint8)
    deq = e2m1_decode(codes) * sdec[..., None].astype(np.float64)
    return codes.reshape(x.shape), micro, deq.reshape(x.shape)


# ----------------------------------------------------------------------------- E2M1 under UE8M0 (MXFP4)
def ue8m0_decode(code):
    """Unsigned 8-bit exponent code -> 2^(code - 127) as float64 (code 255 is not produced here)."""
    return np.exp2(np.asarray(code).astype(np.float64) - 127.0)


def mxfp4_quantize_groups(x):
    """Quantize the LAST axis of x (fp32, length divisible by 32) in groups of 32: E2M1
    elements under a power-of-two scale per group (the format of the FP8 x FP4 block-scaled
    product, used by the hybrid 4-bit arrangement: ExpCast-FP8 P times 4-bit values).

    The paper gives no rule for the exponent; taken here: the smallest power of two that maps
    the group maximum into the E2M1 range without clipping.  y = max|x| / 6 as ONE IEEE fp32
    division; e = exponent(y), plus one unless y is a power of two; scale = 2^e (stored as
    e + 127, clamped to [0, 254]); element = E2M1(x / 2^e), exact scaling, one rounding.  A
    group of zeros stores code 0 and zero elements.  Returns (codes uint8 0..15, scale codes
    uint8, deq fp64 = dec(code) * 2^e).
    """
    x = np.asarray(x, dtype=np.float32)
    g = x.reshape(x.shape[:-1] + (x.shape[-1] // 32, 32))
    amax = np.max(np.abs(g), axis=-1).astype(np.float32)
    y = (amax / np.float32(6.0)).astype(np.float32)
    bits = y.view(np.uint32).astype(np.int64)
    e = ((bits >> 23) & 0xFF) - 127 + ((bits & 0x7FFFFF) != 0).astype(np.int64)
    code = np.clip(e + 127, 0, 254)
    code = np.where(amax > 0, code, 0).astype(np.uint8)
    scale = ue8m0_decode(code)
    yv = (g.astype(np.float64) / scale[..., None]).astype(np.float32)       # exact: power of two
    codes = e2m1_encode(yv)
    codes = np.where(amax[..., None] > 0, codes, np.uint8(0)).astype(np.uint8)
    deq = e2m1_decode(codes) * scale[..., None]
    return codes.reshape(x.shape), code, deq.reshape(x.shape)

"""Number formats of the NVFP4 path: E2M1 elements, E4M3 block scales, bf16.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain CPU oracle that the
CUDA library is checked against.  Only the tests, the smoke check and the CPU
baseline leg of the benchmark may import it; the product never does.

Every value table here is generated from the paper's unified mini-float
formula (Eq. "quant-unified", Section "Low-Precision Inference"):

    Q = alpha * (-1)^sign * 2^d * (1 + sum_i m_i / 2^i)

with b=4, e=2 (one mantissa bit) for the E2M1 element and b=8, e=4 (three
mantissa bits) for the E4M3 scale, plus the usual IEEE-style conventions the
formula leaves implicit: exponent bias 2^(e-1)-1, and exponent field 0 meaning
a subnormal (no implicit leading one, exponent of field 1).  The paper fixes the
E2M1 magnitude set {0, 0.5, 1, 1.5, 2, 3, 4, 6} and the E4M3 maximum 448
(Section "Low-Precision Inference", paragraphs FP8 and FP4); the tests pin the
generated tables to both.

Rounding is round-to-nearest, ties to the code with an even mantissa bit,
saturating at the largest finite magnitude.  The paper only says "discrete
rounding operator"; round-to-nearest-even is the reading adopted everywhere in
this repository.

Parity pins: every function in this file is pinned (exhaustive tables against
the paper's value set and against torch's float8_e4m3fn / bfloat16 conversions).
The sign given to values that round to zero (the sign bit is kept) is a
convention with nothing to pin it: "parity unpinned" for that bit only.
"""
import numpy as np

E2M1_EXP_BITS, E2M1_MAN_BITS, E2M1_BIAS = 2, 1, 1
E4M3_EXP_BITS, E4M3_MAN_BITS, E4M3_BIAS = 4, 3, 7


def minifloat_magnitudes(exp_bits, man_bits, bias):
    """All magnitudes of a sign/exponent/mantissa mini-float, indexed by the
    code without its sign bit (Eq. quant-unified with alpha = 1)."""
    out = np.zeros(1 << (exp_bits + man_bits), dtype=np.float64)
    for code in range(out.size):
        exp_field = code >> man_bits
        frac = (code & ((1 << man_bits) - 1)) / float(1 << man_bits)
        if exp_field == 0:                       # subnormal: no implicit one
            out[code] = frac * 2.0 ** (1 - bias)
        else:
            out[code] = (1.0 + frac) * 2.0 ** (exp_field - bias)
    return out


# E2M1: codes 0..7 -> 0, 0.5, 1, 1.5, 2, 3, 4, 6.  Bit 3 of the nibble is the sign.
E2M1_MAGNITUDES = minifloat_magnitudes(E2M1_EXP_BITS, E2M1_MAN_BITS, E2M1_BIAS)

# E4M3 (finite-only variant): exponent field 15 with mantissa 7 is NaN, so the
# largest finite magnitude is code 0x7E = 1.75 * 2^8 = 448.
_E4M3_ALL = minifloat_magnitudes(E4M3_EXP_BITS, E4M3_MAN_BITS, E4M3_BIAS)
E4M3_NAN_CODE = 0x7F
E4M3_MAGNITUDES = _E4M3_ALL[:E4M3_NAN_CODE]      # 127 finite magnitudes, codes 0x00..0x7E
E4M3_MAX = float(E4M3_MAGNITUDES[-1])            # 448
E2M1_MAX = float(E2M1_MAGNITUDES[-1])            # 6


def _round_to_table(mag, table):
    """Index of the table entry nearest to each magnitude; a magnitude exactly
    half way between two entries goes to the even index (the index parity is
    the parity of the mantissa's last bit); magnitudes above the last entry
    saturate to it.  `mag` is float64 >= 0, `table` ascending float64."""
    mag = np.asarray(mag, dtype=np.float64)
    hi = np.searchsorted(table, mag, side="left")          # first entry >= mag
    hi = np.minimum(hi, table.size - 1)
    lo = np.maximum(hi - 1, 0)
    mid = 0.5 * (table[lo] + table[hi])                    # exact in float64
    pick_hi = (mag > mid) | ((mag == mid) & (hi % 2 == 0))
    idx = np.where(pick_hi, hi, lo)
    idx = np.where(mag >= table[-1], table.size - 1, idx)  # saturate
    return idx.astype(np.uint8)


def e2m1_decode(code):
    """Nibble (0..15) -> value, float64 (exact)."""
    code = np.asarray(code, dtype=np.uint8)
    mag = E2M1_MAGNITUDES[code & 7]
    return np.where(code & 8, -mag, mag)


def e2m1_encode(v):
    """float32 -> nibble, round-to-nearest-even, saturating at 6; the sign bit
    is copied from the input even when the magnitude rounds to zero."""
    v = np.asarray(v, dtype=np.float32)
    idx = _round_to_table(np.abs(v).astype(np.float64), E2M1_MAGNITUDES)
    return (idx | (np.signbit(v).astype(np.uint8) << 3)).astype(np.uint8)


def e4m3_decode(code):
    """Byte -> value, float64 (exact); 0x7F / 0xFF decode to NaN."""
    code = np.asarray(code, dtype=np.uint8)
    mag = _E4M3_ALL[code & 0x7F].copy()
    mag = np.where((code & 0x7F) == E4M3_NAN_CODE, np.nan, mag)
    return np.where(code & 0x80, -mag, mag)


def e4m3_encode(v):
    """float32 -> byte, round-to-nearest-even including the subnormal range,
    saturating at 448 (never produces NaN for finite input)."""
    v = np.asarray(v, dtype=np.float32)
    idx = _round_to_table(np.abs(v).astype(np.float64), E4M3_MAGNITUDES)
    return (idx | (np.signbit(v).astype(np.uint8) << 7)).astype(np.uint8)


def bf16_round(x):
    """Round float32/float64 to the nearest bfloat16 (ties to even), returned as
    float32 whose low 16 bits are zero.  bfloat16 = the top 16 bits of an IEEE
    float32 (1 sign, 8 exponent, 7 mantissa bits)."""
    x64 = np.asarray(x, dtype=np.float64)
    x32 = x64.astype(np.float32)
    # float64 -> float32 -> bf16 could round twice; redo the decision exactly:
    # the two bf16 neighbours of x are the truncation of x32 (towards zero)
    # and the next one away from zero; pick by exact float64 comparison.
    bits = x32.view(np.uint32) if x32.ndim else np.array([x32]).view(np.uint32)
    bits = bits.reshape(x32.shape)
    # make sure `down` has magnitude <= |x| (x32 may have rounded up past x)
    down_bits = bits & np.uint32(0xFFFF0000)
    down = down_bits.view(np.float32).astype(np.float64)
    too_big = np.abs(down) > np.abs(x64)
    down_bits = np.where(too_big, down_bits - np.uint32(0x10000), down_bits).astype(np.uint32)
    down = down_bits.view(np.float32).astype(np.float64)
    up_bits = (down_bits + np.uint32(0x10000)).astype(np.uint32)
    up = up_bits.view(np.float32).astype(np.float64)
    mid = 0.5 * (down + up)
    ax = np.abs(x64)
    pick_up = (ax > np.abs(mid)) | ((ax == np.abs(mid)) & ((down_bits >> 16) & 1 == 1))
    out_bits = np.where(pick_up, up_bits, down_bits).astype(np.uint32)
    return out_bits.view(np.float32).reshape(x64.shape)


def bf16_bits(x_bf16_as_f32):
    """float32 holding a bf16 value -> its 16-bit pattern."""
    a = np.ascontiguousarray(x_bf16_as_f32, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


def bf16_from_bits(b):
    """16-bit pattern -> float32 holding that bf16 value."""
    b = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32)


def pack_nibbles(codes):
    """[..., K] nibbles -> [..., K/2] bytes; element 2i in the low nibble and
    element 2i+1 in the high nibble of byte i (a layout convention, "parity
    unpinned": the paper does not describe a byte layout)."""
    codes = np.asarray(codes, dtype=np.uint8)
    return (codes[..., 0::2] | (codes[..., 1::2] << 4)).astype(np.uint8)


def unpack_nibbles(packed):
    packed = np.asarray(packed, dtype=np.uint8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = packed & 0xF
    out[..., 1::2] = packed >> 4
    return out

"""Bit-exact FP8-E4M3 codec and block quantisation (oracle; test infrastructure only).

Section 2.1 of the paper gives symmetric quantisation as
``Q(X) = clamp(round(X / s)) * s`` with ``s = max|X| / q_max`` and names FP8-E4M3
(4 exponent bits, 3 mantissa bits) as the grid.  The paper says nothing more
about the format, so the published OCP 8-bit floating point definition is used:

* 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits;
* no infinities; the only NaN pattern is S.1111.111;
* largest finite magnitude 448 (code 0x7E), smallest normal 2^-6,
  subnormals k * 2^-9 for k = 1..7.

``round`` is round-to-nearest, ties to the code whose mantissa LSB is even;
``clamp`` saturates at +-448.  The encoder works on the IEEE-754 binary32 bit
pattern with integer arithmetic only; it does not use any float8 data type.
"""

from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0
_BIAS = 7


def _build_decode_table() -> np.ndarray:
    table = np.zeros(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            val = float("nan")
        elif e == 0:
            val = sign * m * 2.0 ** (1 - _BIAS - 3)          # subnormal: m * 2^-9
        else:
            val = sign * (1.0 + m / 8.0) * 2.0 ** (e - _BIAS)
        table[code] = val
    return table


DECODE_TABLE = _build_decode_table()


def decode(codes) -> np.ndarray:
    """E4M3 code (uint8) -> value, exactly, as float64."""
    codes = np.asarray(codes, dtype=np.uint8)
    return DECODE_TABLE[codes]


def encode(x) -> np.ndarray:
    """binary32 value -> E4M3 code with round-to-nearest-even and saturation.

    ``x`` is converted to float32 first (inputs are expected to be float32
    already).  Non-finite inputs are an error.  The sign bit is always copied,
    so -0.0 and negative values that round to zero give 0x80.
    """
    xf = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    if not np.all(np.isfinite(xf)):
        raise ValueError("e4m3.encode: non-finite input")
    bits = xf.view(np.uint32).astype(np.int64)
    sign = (bits >> 31) & 1
    efield = (bits >> 23) & 0xFF
    m23 = bits & 0x7FFFFF
    E = efield - 127                                   # unbiased binary32 exponent

    # --- normal E4M3 range: |x| >= 2^-6 -----------------------------------
    keep = m23 >> 20
    rem = m23 & 0xFFFFF
    half = 1 << 19
    up = (rem > half) | ((rem == half) & ((keep & 1) == 1))
    code_norm = (((E + _BIAS) << 3) | keep) + up.astype(np.int64)   # carry may bump the exponent
    code_norm = np.minimum(code_norm, 0x7E)

    # --- subnormal E4M3 range: |x| < 2^-6, grid step 2^-9 -----------------
    # |x| = M * 2^(E-23) with M = 2^23 + m23;  k = round(|x| / 2^-9) = round(M / 2^shift)
    M = m23 | (1 << 23)
    shift = np.clip(14 - E, 0, 40)
    keep_s = M >> shift
    rem_s = M & ((np.int64(1) << shift) - 1)
    half_s = np.int64(1) << np.maximum(shift - 1, 0)
    up_s = (rem_s > half_s) | ((rem_s == half_s) & ((keep_s & 1) == 1))
    code_sub = keep_s + up_s.astype(np.int64)          # k = 8 is the smallest normal, code 0x08
    code_sub = np.where(efield == 0, 0, code_sub)      # binary32 zero / subnormal -> 0

    mag = np.where(E >= -6, code_norm, code_sub)
    mag = np.where(E > 8, 0x7E, mag)                   # >= 512: saturate (also guards the shift above)
    return ((sign << 7) | mag).astype(np.uint8)


def quantize_blocks(x, block: int):
    """Per-block FP8 quantisation along the last axis.

    x      [R, K] array holding bf16-representable values (any float dtype)
    block  number of consecutive elements along K sharing one scale

    For each block: amax = max|x|; s = fl32(amax / 448) (one binary32 division),
    s = 1 when amax == 0; q = encode(fl32(fl32(x) / s)) (one binary32 division,
    then round-to-nearest-even onto the E4M3 grid, saturating).

    Returns (codes uint8 [R, K], scales float32 [R, K // block]).
    """
    x32 = np.asarray(x, dtype=np.float32)
    R, K = x32.shape
    if K % block:
        raise ValueError("block must divide the last dimension")
    slab = max(1, (1 << 22) // max(K, 1))
    if R > slab:
        # rows are independent: walk the matrix in row slabs only to keep the integer temporaries small
        parts = [quantize_blocks(x32[r0:r0 + slab], block) for r0 in range(0, R, slab)]
        return np.concatenate([p[0] for p in parts], axis=0), np.concatenate([p[1] for p in parts], axis=0)
    xb = x32.reshape(R, K // block, block)
    amax = np.max(np.abs(xb), axis=2).astype(np.float32)
    scales = (amax / np.float32(E4M3_MAX)).astype(np.float32)
    scales = np.where(amax == 0, np.float32(1.0), scales).astype(np.float32)
    with np.errstate(over="ignore"):
        quot = (xb / scales[:, :, None]).astype(np.float32)
    # a quotient can only overflow binary32 when the scale is subnormal; it saturates anyway
    quot = np.clip(quot, -3.0e38, 3.0e38).astype(np.float32)
    codes = encode(quot).reshape(R, K)
    return codes, scales


def quantize_tensor(x):
    """Per-tensor dynamic scaling (what the paper's own rollouts used): one scale s = fl32(max|x| / 448) for the
    whole matrix, same code rule as quantize_blocks.  Returns (codes uint8 [R, K], scale float32 scalar)."""
    x32 = np.asarray(x, dtype=np.float32)
    R, K = x32.shape
    amax = np.float32(np.max(np.abs(x32))) if x32.size else np.float32(0)
    s = np.float32(1.0) if amax == 0 else (amax / np.float32(E4M3_MAX)).astype(np.float32)
    rows = max(1, (1 << 22) // max(K, 1))
    parts = []
    for r0 in range(0, max(R, 1), rows):
        with np.errstate(over="ignore"):
            quot = (x32[r0:r0 + rows] / s).astype(np.float32)
        parts.append(encode(np.clip(quot, -3.0e38, 3.0e38).astype(np.float32)))
    codes = np.concatenate(parts, axis=0).reshape(R, K) if parts else np.zeros((R, K), np.uint8)
    return codes, np.float32(s)


def dequantize_blocks(codes, scales, block: int) -> np.ndarray:
    """codes [R, K], scales [R, K // block] -> float64 [R, K] = decode(q) * s (exact product)."""
    codes = np.asarray(codes, dtype=np.uint8)
    R, K = codes.shape
    vals = decode(codes).reshape(R, K // block, block)
    out = vals * np.asarray(scales, dtype=np.float64)[:, :, None]
    return out.reshape(R, K)


# --------------------------------------------------------------------------- microscaling (power-of-two scales)
MX_BLOCK = 32
_MX_EMAX = 8              # exponent of the largest E4M3 binade: 448 = 1.75 * 2^8


def quantize_mx(x):
    """Microscaling FP8: blocks of 32 consecutive elements along the last axis share one power-of-two scale
    stored as an 8-bit biased exponent (E8M0, bias 127) -- the format the paper's limitations section points to
    for lower-precision rollouts.  Rule of the published OCP microscaling specification: the shared exponent is
    floor(log2(max|x|)) minus the exponent of the element format's largest binade, X = floor(log2 amax) - 8, and
    the elements are x / 2^X rounded to nearest-even onto the E4M3 grid, saturating (scaled magnitudes in
    (448, 512) become 448).  The specification leaves an all-zero block open: scale code 127 (2^0) here.  Codes
    are clamped to 0..254 (255 is the format's NaN).

    Returns (codes uint8 [R, K], scale codes uint8 [R, K // 32]).
    """
    x64 = np.asarray(x, dtype=np.float64)
    R, K = x64.shape
    if K % MX_BLOCK:
        raise ValueError("the last dimension must be a multiple of 32")
    slab = max(1, (1 << 22) // max(K, 1))
    if R > slab:
        parts = [quantize_mx(x64[r0:r0 + slab]) for r0 in range(0, R, slab)]
        return np.concatenate([p[0] for p in parts], axis=0), np.concatenate([p[1] for p in parts], axis=0)
    xb = x64.reshape(R, K // MX_BLOCK, MX_BLOCK)
    amax = np.max(np.abs(xb), axis=2)
    _, e = np.frexp(amax)                                   # amax = m * 2^e, m in [0.5, 1): floor(log2 amax) = e - 1
    X = np.where(amax > 0, e - 1 - _MX_EMAX, 0)
    sc = np.clip(X + 127, 0, 254).astype(np.int64)
    sc = np.where(amax > 0, sc, 127)
    scaled = np.ldexp(xb, -(sc[:, :, None] - 127))          # exact: a power of two
    scaled = np.clip(scaled, -3.0e38, 3.0e38).astype(np.float32)   # binary32 holds every scaled bf16 value exactly or saturates
    codes = encode(scaled).reshape(R, K)
    return codes, sc.astype(np.uint8)


def dequantize_mx(codes, scale_codes) -> np.ndarray:
    """codes [R, K], E8M0 scale codes [R, K // 32] -> float64 [R, K] = decode(q) * 2^(code - 127), exactly."""
    codes = np.asarray(codes, dtype=np.uint8)
    R, K = codes.shape
    vals = decode(codes).reshape(R, K // MX_BLOCK, MX_BLOCK)
    out = np.ldexp(vals, np.asarray(scale_codes, dtype=np.int64)[:, :, None] - 127)
    return out.reshape(R, K)


# --------------------------------------------------------------------------- microscaling FP4 (E2M1 elements)
_E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
_FP4_EMAX = 2             # 6 = 1.5 * 2^2


def encode_e2m1(x) -> np.ndarray:
    """Value -> 4-bit E2M1 code (1 sign, 2 exponent, 1 mantissa bit; magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6; no
    infinities or NaNs), round to nearest with ties to the code whose mantissa bit is 0, saturating at +-6.  The
    sign bit is copied from the input.  Written as a nearest-value search: the grid has eight magnitudes."""
    v = np.asarray(x, dtype=np.float64)
    if not np.all(np.isfinite(v)):
        raise ValueError("E2M1 has no encoding for infinities or NaNs")
    mag = np.minimum(np.abs(v), 6.0)
    d = np.abs(mag[..., None] - _E2M1_VALUES)
    lo = np.argmin(d, axis=-1)                               # first (smaller) of two equally near codes
    nxt = np.minimum(lo + 1, 7)
    tie = (nxt != lo) & (np.take_along_axis(d, nxt[..., None], axis=-1)[..., 0] == np.take_along_axis(d, lo[..., None], axis=-1)[..., 0])
    code = np.where(tie & (lo % 2 == 1), lo + 1, lo)         # on a tie take the even code
    return (code | (np.signbit(v).astype(np.int64) << 3)).astype(np.uint8)


def decode_e2m1(codes) -> np.ndarray:
    c = np.asarray(codes, dtype=np.uint8)
    return np.where(c & 8, -1.0, 1.0) * _E2M1_VALUES[c & 7]


def quantize_mxfp4(x):
    """Microscaling FP4: blocks of 32 elements share 2^X, X = floor(log2 amax) - 2, stored as X + 127 (clamped to
    0..254; 127 for a zero block); elements are x / 2^X on the E2M1 grid (scaled magnitudes in (6, 8) saturate to 6).
    Same published rule as quantize_mx with the FP4 element format -- the FP4 rollouts the paper names as future work.

    Returns (codes uint8 [R, K], one 4-bit code per entry, and scale codes uint8 [R, K // 32])."""
    x64 = np.asarray(x, dtype=np.float64)
    R, K = x64.shape
    if K % MX_BLOCK:
        raise ValueError("the last dimension must be a multiple of 32")
    xb = x64.reshape(R, K // MX_BLOCK, MX_BLOCK)
    amax = np.max(np.abs(xb), axis=2)
    _, e = np.frexp(amax)
    X = np.where(amax > 0, e - 1 - _FP4_EMAX, 0)
    sc = np.clip(X + 127, 0, 254).astype(np.int64)
    sc = np.where(amax > 0, sc, 127)
    scaled = np.ldexp(xb, -(sc[:, :, None] - 127))
    codes = encode_e2m1(np.clip(scaled, -1e30, 1e30)).reshape(R, K)
    return codes, sc.astype(np.uint8)


def dequantize_mxfp4(codes, scale_codes) -> np.ndarray:
    codes = np.asarray(codes, dtype=np.uint8)
    R, K = codes.shape
    vals = decode_e2m1(codes).reshape(R, K // MX_BLOCK, MX_BLOCK)
    return np.ldexp(vals, np.asarray(scale_codes, dtype=np.int64)[:, :, None] - 127).reshape(R, K)

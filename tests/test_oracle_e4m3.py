"""Pins for the oracle's E4M3 codec and block quantiser (CPU only).

The pins are independent of the oracle's own arithmetic: the format's landmark values
(tests/golden/e4m3_landmarks.txt), exhaustive round-trips, midpoint behaviour worked out from
the grid itself, a third-party float8 implementation used as a black box, and error bounds.
"""

import os

import numpy as np
import pytest

from oracle import e4m3

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _finite_codes():
    return np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def test_landmark_values():
    for line in open(os.path.join(GOLDEN, "e4m3_landmarks.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        code, val = line.split()
        code = int(code, 16)
        got = e4m3.decode(np.array([code], dtype=np.uint8))[0]
        assert got == float(val), (hex(code), got, val)
        assert np.signbit(got) == bool(code & 0x80)
        assert e4m3.encode(np.array([float(val)], dtype=np.float32))[0] == code


def test_nan_codes_and_grid_shape():
    assert np.isnan(e4m3.decode(np.array([0x7F, 0xFF], dtype=np.uint8))).all()
    pos = e4m3.decode(np.arange(0, 0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)                       # strictly increasing in the code
    assert pos[-1] == 448.0 and pos[1] == 2.0 ** -9 and pos[8] == 2.0 ** -6
    # mantissa spacing: within one binade 8 equal steps
    for e in range(1, 15):
        seg = pos[e * 8:(e + 1) * 8]
        assert np.allclose(np.diff(seg), seg[0] / 8.0, rtol=0, atol=0)


def test_round_trip_all_codes():
    codes = _finite_codes()
    vals = e4m3.decode(codes).astype(np.float32)
    assert np.array_equal(e4m3.encode(vals), codes)


def test_midpoints_tie_to_even_and_neighbours():
    pos = e4m3.decode(np.arange(0, 0x7F, dtype=np.uint8))          # 0 .. 448
    for c in range(0, 0x7E):
        lo, hi = pos[c], pos[c + 1]
        mid = np.float32((lo + hi) / 2.0)                          # exactly representable in binary32
        assert float(mid) == (lo + hi) / 2.0
        even = c if (c & 1) == 0 else c + 1
        assert e4m3.encode(np.array([mid]))[0] == even, (c, mid)
        below = np.nextafter(mid, np.float32(0))
        above = np.nextafter(mid, np.float32(1e9))
        assert e4m3.encode(np.array([below]))[0] == c
        assert e4m3.encode(np.array([above]))[0] == c + 1
        # negative side mirrors
        assert e4m3.encode(np.array([-mid]))[0] == (0x80 | even)


def test_saturation():
    xs = np.array([448.0, 449.0, 463.9, 464.0, 465.0, 480.0, 512.0, 1e4, 3e38], dtype=np.float32)
    assert np.all(e4m3.encode(xs) == 0x7E)
    assert np.all(e4m3.encode(-xs) == 0xFE)


def test_subnormal_range():
    tiny = 2.0 ** -9
    assert e4m3.encode(np.array([tiny / 2], dtype=np.float32))[0] == 0x00          # tie -> even (zero)
    assert e4m3.encode(np.array([np.nextafter(np.float32(tiny / 2), np.float32(1))]))[0] == 0x01
    assert e4m3.encode(np.array([tiny * 0.49], dtype=np.float32))[0] == 0x00
    assert e4m3.encode(np.array([tiny * 7.5], dtype=np.float32))[0] == 0x08        # tie -> even (8 = min normal)
    assert e4m3.encode(np.array([tiny * 6.5], dtype=np.float32))[0] == 0x06
    assert e4m3.encode(np.array([-1e-30], dtype=np.float32))[0] == 0x80            # sign kept
    assert e4m3.encode(np.array([-0.0], dtype=np.float32))[0] == 0x80
    assert e4m3.encode(np.array([1e-45], dtype=np.float32))[0] == 0x00             # binary32 subnormal


def test_non_finite_rejected():
    with pytest.raises(ValueError):
        e4m3.encode(np.array([np.inf], dtype=np.float32))
    with pytest.raises(ValueError):
        e4m3.encode(np.array([np.nan], dtype=np.float32))


def test_nearest_by_brute_force():
    """Every encoded value is a nearest grid point (brute-force search over the 127 magnitudes)."""
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.uniform(-448, 448, 20000),
                        rng.normal(0, 0.01, 20000)]).astype(np.float32)
    grid = e4m3.decode(np.arange(0, 0x7F, dtype=np.uint8))
    got = np.abs(e4m3.decode(e4m3.encode(x)))
    dist = np.abs(np.abs(x.astype(np.float64))[:, None] - grid[None, :]).min(axis=1)
    assert np.array_equal(np.abs(np.abs(x.astype(np.float64)) - got), dist)


def test_against_ml_dtypes_black_box():
    ml_dtypes = pytest.importorskip("ml_dtypes")
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.uniform(-448, 448, 500000), rng.normal(0, 1, 300000),
                        rng.normal(0, 2.0 ** -7, 200000)]).astype(np.float32)
    ref = x.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(e4m3.encode(x), ref)
    # all bf16 values with |x| <= 448
    bits = np.arange(0, 1 << 16, dtype=np.uint32) << 16
    v = bits.view(np.float32)
    v = v[np.isfinite(v) & (np.abs(v) <= 448)]
    assert np.array_equal(e4m3.encode(v), v.astype(ml_dtypes.float8_e4m3fn).view(np.uint8))


# ------------------------------------------------------------------ block quantisation
def _bf16_round(x):
    import torch
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).float().numpy()


def test_block_scale_rule_and_zero_block():
    x = np.zeros((2, 256), dtype=np.float32)
    x[0, :128] = _bf16_round(np.linspace(-3, 3, 128))
    x[1, 128:] = 0.0
    x[1, :128] = _bf16_round(np.random.default_rng(0).normal(size=128))
    codes, scales = e4m3.quantize_blocks(x, 128)
    assert scales.dtype == np.float32 and codes.dtype == np.uint8
    assert scales[0, 1] == 1.0 and scales[1, 1] == 1.0                # zero block -> scale 1
    assert np.all(codes[0, 128:] == 0)
    for r in range(2):
        amax = np.abs(x[r, :128]).max()
        assert scales[r, 0] == np.float32(amax) / np.float32(448.0)
        # the largest element of a non-zero block lands on +-448
        j = np.abs(x[r, :128]).argmax()
        assert codes[r, j] & 0x7F == 0x7E


def test_power_of_two_scale_block_is_exact():
    """amax = 3.5 = 448 * 2^-7: the scale is exactly 2^-7, so grid values round-trip exactly and
    halfway values go to the even code."""
    s = 2.0 ** -7
    grid = e4m3.decode(np.arange(0, 0x7F, dtype=np.uint8))
    vals = grid[8:0x7F:3] * s                                          # all bf16-exact (4 significant bits)
    x = np.zeros((1, 128), dtype=np.float32)
    x[0, :len(vals)] = vals
    x[0, 127] = 3.5
    # halfway between codes 0x38 (1.0) and 0x39 (1.125), times s: 1.0625 * 2^-7 -> even code 0x38
    x[0, 126] = 1.0625 * s
    # halfway between 0x39 (1.125) and 0x3A (1.25): 1.1875 -> even code 0x3A
    x[0, 125] = 1.1875 * s
    codes, scales = e4m3.quantize_blocks(x, 128)
    assert scales[0, 0] == np.float32(s)
    assert np.array_equal(codes[0, :len(vals)], np.arange(8, 0x7F, 3, dtype=np.uint8))
    assert codes[0, 127] == 0x7E and codes[0, 126] == 0x38 and codes[0, 125] == 0x3A
    deq = e4m3.dequantize_blocks(codes, scales, 128)
    assert np.array_equal(deq[0, :len(vals)], vals)


@pytest.mark.parametrize("block", [32, 128])
def test_block_error_bound(block):
    rng = np.random.default_rng(3)
    x = _bf16_round(rng.normal(0, 1, size=(64, 512)) * rng.lognormal(0, 2, size=(64, 1)))
    codes, scales = e4m3.quantize_blocks(x, block)
    deq = e4m3.dequantize_blocks(codes, scales, block)
    s = np.repeat(scales.astype(np.float64), block, axis=1)
    q = np.abs(x.astype(np.float64)) / s
    # half the local grid spacing: normal codes 2^(floor(log2 q) - 4); subnormal region 2^-10
    half_step = np.where(q >= 2.0 ** -6, 2.0 ** (np.floor(np.log2(np.maximum(q, 1e-300))) - 4), 2.0 ** -10)
    err = np.abs(deq - x.astype(np.float64))
    assert np.all(err <= s * half_step * (1 + 1e-6) + s * q * 2.0 ** -23)
    # relative error at most 2^-4 for everything that maps to a normal code
    norm = q >= 2.0 ** -6
    assert np.all(err[norm] <= 2.0 ** -4 * np.abs(x.astype(np.float64))[norm] * (1 + 1e-6))
    assert np.all(np.sign(deq) * np.sign(x) >= 0)


def test_block_axis_is_last_axis_only():
    """Changing an element changes only its own block's scale."""
    rng = np.random.default_rng(5)
    x = _bf16_round(rng.normal(size=(4, 256)))
    c0, s0 = e4m3.quantize_blocks(x, 128)
    y = x.copy()
    y[2, 130] = 64.0
    c1, s1 = e4m3.quantize_blocks(y, 128)
    diff = (s0 != s1)
    assert diff.sum() == 1 and diff[2, 1]
    assert np.array_equal(c0[:, :128], c1[:, :128]) and np.array_equal(c0[[0, 1, 3]], c1[[0, 1, 3]])


def test_per_tensor_quantisation():
    """One scale for the whole matrix: equals block quantisation of the flattened matrix as a single block; the
    global maximum lands on +-448; an all-zero matrix gets scale 1."""
    rng = np.random.default_rng(9)
    x = _bf16_round(rng.normal(size=(6, 96)) * 3)
    codes, s = e4m3.quantize_tensor(x)
    c1, s1 = e4m3.quantize_blocks(x.reshape(1, -1), x.size)
    assert s == s1[0, 0] and np.array_equal(codes.reshape(1, -1), c1)
    assert s == np.float32(np.abs(x).max()) / np.float32(448)
    i = np.unravel_index(np.abs(x).argmax(), x.shape)
    assert codes[i] & 0x7F == 0x7E
    z, sz = e4m3.quantize_tensor(np.zeros((3, 8), np.float32))
    assert sz == 1.0 and not z.any()


# --------------------------------------------------------------------------- microscaling (E8M0 scale per 32 elements)
def test_mx_shared_exponent_rule_and_saturation_band():
    """Hand-worked blocks: the scale code is floor(log2 amax) - 8 + 127; a zero block gets 127; scaled magnitudes
    between 448 and 512 saturate to 448 (the known clipping band of the microscaling rule)."""
    def one(amax, fill=0.0):
        x = np.full((1, 32), fill, np.float32)
        x[0, 5] = amax
        c, s = e4m3.quantize_mx(x)
        return int(s[0, 0]), float(e4m3.dequantize_mx(c, s)[0, 5])
    assert one(1.0) == (119, 1.0)                  # 1 = 256 * 2^-8
    assert one(448.0) == (127, 448.0)
    assert one(256.0) == (127, 256.0)
    assert one(255.0) == (126, 224.0)              # floor(log2 255) = 7: 255 / 2^-1 = 510 saturates to 448, times 2^-1
    assert one(0.0) == (127, 0.0)
    assert one(-3.5) == (120, -3.5)                # 3.5 = 448 * 2^-7
    assert one(480.0) == (127, 448.0)              # inside (448, 512): saturates
    assert one(2.0 ** -140) == (0, 0.0)            # below the smallest scale: the code clamps at 0, the element underflows


def test_mx_values_on_the_scaled_grid_round_trip_exactly():
    rng = np.random.default_rng(21)
    codes = rng.integers(0, 256, size=(8, 128)).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x30
    codes[:, ::32] = 0x7E                                   # every block holds the largest magnitude 448
    k = rng.integers(-20, 20, size=(8, 4))
    x = np.ldexp(e4m3.decode(codes).reshape(8, 4, 32), k[:, :, None]).reshape(8, 128)
    c, s = e4m3.quantize_mx(x)
    assert np.array_equal(s.astype(np.int64), k + 127)
    assert np.array_equal(e4m3.dequantize_mx(c, s), x)


def test_mx_against_nearest_value_search():
    """Independent restatement: exponent from math.frexp, element by exhaustive search for the nearest grid value
    (ties to the even code), saturating."""
    import math
    rng = np.random.default_rng(22)
    x = _bf16_round(rng.normal(size=(3, 64)) * np.exp(rng.normal(size=(3, 1)) * 4))
    c, s = e4m3.quantize_mx(x)
    grid = e4m3.decode(np.arange(127, dtype=np.uint8))                  # non-negative finite values, ascending
    for r in range(3):
        for b in range(2):
            blk = x[r, 32 * b:32 * b + 32].astype(np.float64)
            amax = float(np.abs(blk).max())
            X = math.frexp(amax)[1] - 1 - 8
            assert int(s[r, b]) == X + 127
            for j, v in enumerate(blk):
                t = min(abs(float(v)) / 2.0 ** X, 448.0)
                d = np.abs(grid - t)
                best = np.flatnonzero(d == d.min())
                code = int(best[0]) if len(best) == 1 else int([q for q in best if q % 2 == 0][0])
                assert int(c[r, 32 * b + j]) & 0x7F == code, (r, b, j, v)
                assert (int(c[r, 32 * b + j]) >> 7) == int(np.signbit(v))


def test_mx_error_bound():
    rng = np.random.default_rng(23)
    x = _bf16_round(rng.normal(size=(16, 256)))
    c, s = e4m3.quantize_mx(x)
    deq = e4m3.dequantize_mx(c, s)
    scale = np.repeat(np.ldexp(1.0, s.astype(np.int64) - 127), 32, axis=1)
    q = np.abs(x.astype(np.float64)) / scale
    ok = (q >= 2.0 ** -6) & (q <= 448)
    assert np.all(np.abs(deq - x)[ok] <= 2.0 ** -4 * np.abs(x)[ok])
    assert np.all(q < 512)                                   # the shared exponent never lets an element reach 512


def test_abi_layout_reader_against_a_scalar_walk():
    """The test-side reader of the packed scale bytes (tests/abi_layout.py) against a byte-by-byte walk of the order
    the C header describes: 512-byte chunks of 128 rows x 4 blocks, inside a chunk 32 row slots of 16 bytes, each
    slot holding the four 32-row quarters of the chunk with their four block bytes; the two chunks of a 256-row
    group adjacent; chunk columns of a group one after the other; groups one after the other."""
    import abi_layout
    R, K = 300, 256                                          # two row groups (the second ragged), two chunk columns
    NB = K // 32
    sc = ((np.arange(R)[:, None] * 7 + np.arange(NB)[None, :] * 3) % 250).astype(np.uint8)
    buf = []
    for group in range((R + 255) // 256):
        for chunk_col in range(NB // 4):
            for half in range(2):
                for slot in range(32):
                    for quarter in range(4):
                        for j in range(4):
                            r = group * 256 + half * 128 + quarter * 32 + slot
                            buf.append(int(sc[r, chunk_col * 4 + j]) if r < R else 127)
    buf = np.array(buf, np.uint8)
    assert buf.size == abi_layout.mx_scale_bytes(R, K)
    assert np.array_equal(abi_layout.unpack_mx_scales(buf, R, K), sc)
    pad = abi_layout.mx_scale_padding(buf, R, K)
    assert pad.size == (512 - R) * NB and np.all(pad == 127)
    assert np.array_equal(abi_layout.unpack_fp4_pairs(np.array([[0x21, 0x0F]], np.uint8)), [[1, 2, 15, 0]])


# --------------------------------------------------------------------------- microscaling FP4 (E2M1)
def test_e2m1_grid_ties_saturation_and_black_box():
    """The eight magnitudes; every midpoint goes to the code with mantissa bit 0; beyond 6 saturates; the sign is
    copied (also for zero); a third-party 4-bit float type agrees on random in-range values."""
    assert np.array_equal(e4m3.decode_e2m1(np.arange(8, dtype=np.uint8)), [0, 0.5, 1, 1.5, 2, 3, 4, 6])
    grid = [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    mids = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}       # midpoint -> even neighbour
    for i, (m, want) in enumerate(mids.items()):
        assert e4m3.decode_e2m1(e4m3.encode_e2m1(np.array([m])))[0] == want
        assert e4m3.decode_e2m1(e4m3.encode_e2m1(np.array([np.nextafter(m, 10)])))[0] == grid[i + 1]
        assert e4m3.decode_e2m1(e4m3.encode_e2m1(np.array([np.nextafter(m, -10)])))[0] == grid[i]
        assert e4m3.decode_e2m1(e4m3.encode_e2m1(np.array([-m])))[0] == -want
    assert e4m3.decode_e2m1(e4m3.encode_e2m1(np.array([6.5, 1e9, -7.0]))).tolist() == [6, 6, -6]
    assert e4m3.encode_e2m1(np.array([-0.0, -0.1]))[0] == 8 and e4m3.encode_e2m1(np.array([-0.0, -0.1]))[1] == 8
    for c in range(16):
        assert e4m3.encode_e2m1(e4m3.decode_e2m1(np.array([c], np.uint8)))[0] == c
    ml_dtypes = pytest.importorskip("ml_dtypes")
    if not hasattr(ml_dtypes, "float4_e2m1fn"):
        pytest.skip("this ml_dtypes has no 4-bit float")
    r = np.clip(np.random.default_rng(3).normal(size=200000) * 3, -6, 6).astype(np.float32)
    ref = r.astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    assert np.array_equal(e4m3.decode_e2m1(e4m3.encode_e2m1(r)), ref)


def test_mxfp4_shared_exponent_and_round_trip():
    """X = floor(log2 amax) - 2: hand cases; values on the scaled grid round-trip; the (6, 8) band saturates."""
    def one(amax):
        x = np.zeros((1, 32))
        x[0, 3] = amax
        c, s = e4m3.quantize_mxfp4(x)
        return int(s[0, 0]), float(e4m3.dequantize_mxfp4(c, s)[0, 3])
    assert one(6.0) == (127, 6.0)
    assert one(4.0) == (127, 4.0)
    assert one(1.0) == (125, 1.0)
    assert one(7.0) == (127, 6.0)                  # floor(log2 7) = 2: 7 is in the clipping band
    assert one(3.0) == (126, 3.0)
    assert one(0.0) == (127, 0.0)
    rng = np.random.default_rng(4)
    codes = rng.integers(0, 16, size=(6, 96)).astype(np.uint8)
    codes[:, ::32] = 7                                      # every block holds the largest magnitude
    k = rng.integers(-10, 10, size=(6, 3))
    x = np.ldexp(e4m3.decode_e2m1(codes).reshape(6, 3, 32), k[:, :, None]).reshape(6, 96)
    c, s = e4m3.quantize_mxfp4(x)
    assert np.array_equal(s.astype(np.int64), k + 127) and np.array_equal(e4m3.dequantize_mxfp4(c, s), x)

// Streaming kernels of the AIS path (everything that is not a dense contraction).
#include <type_traits>

#include "stream_kernels.cuh"
#include "ptx.cuh"

#include <cuda_bf16.h>
#include <math.h>

namespace ais {

namespace {

// ------------------------------------------------------------------------------------------------
// FP8-E4M3 block quantisation.  A CTA covers 32 rows x 1024 columns; each warp walks 4 rows, a lane
// holds 8 consecutive bf16 values (16-byte load), the lanes of one block share the block's amax by
// shuffles, and the block-major scales are staged in shared memory so that they leave coalesced.
// ------------------------------------------------------------------------------------------------
constexpr int kQRows = 32;
constexpr int kQCols = 1024;
constexpr int kQThreads = 256;
constexpr int kQIters = kQCols / 256;      // 16-byte loads per lane and row

__device__ __forceinline__ uint16_t cvt_e4m3x2(float hi, float lo) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Correctly rounded x / s from the correctly rounded reciprocal y = RN(1/s): two residual corrections with
// fused multiply-adds; the first makes the quotient faithful, and a faithful quotient corrected once more with
// the exact residual is the round-to-nearest quotient (Markstein's division theorem).  |x / s| <= 448 here, so
// nothing overflows; a quotient that underflows encodes to zero either way; the sign of x is restored
// explicitly because a zero residual sum would turn -0 into +0.
__device__ __forceinline__ float exact_div(float x, float s, float y) {
    float q = x * y;
    q = __fmaf_rn(__fmaf_rn(-s, q, x), y, q);
    q = __fmaf_rn(__fmaf_rn(-s, q, x), y, q);
    return copysignf(q, x);
}

// IEEE division kept out of line: it is only reached for scales outside [2^-100, 2^100] and would otherwise
// be inlined eight times into every copy of the hot loop.
__device__ __noinline__ float slow_div(float x, float s) { return __fdiv_rn(x, s); }

// amax of the block a lane belongs to, on the bf16 bit patterns: |x| is the pattern without its sign bit, and patterns
// of non-negative values order like the values, so packed 16-bit unsigned maxima do the work of eight float compares
template <int BLOCK>
__device__ __forceinline__ uint32_t block_amax_bits(const uint4 raw) {
    constexpr int kLanesPerBlock = BLOCK / 8;
    uint32_t m = __vmaxu2(__vmaxu2(raw.x & 0x7FFF7FFFu, raw.y & 0x7FFF7FFFu), __vmaxu2(raw.z & 0x7FFF7FFFu, raw.w & 0x7FFF7FFFu));
    m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
    for (int off = 1; off < kLanesPerBlock; off <<= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, off));
    return m;
}

// Eight bf16 values divided by the block's scale s (y = RN(1 / s)) and rounded to E4M3.
__device__ __forceinline__ uint2 quantize_values(const uint4 raw, float s, float y) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float v[8], qv[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
    if (s > 0x1p-100f && s < 0x1p100f) {
        // exact_div on two values per instruction (the packed fp32 forms round each half like the scalar ones)
        const F2 ys = {y, y}, ns = {-s, -s};
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            const F2 x = {v[i], v[i + 1]};
            F2 q = mul2(x, ys);
            q = fma2(fma2(ns, q, x), ys, q);
            q = fma2(fma2(ns, q, x), ys, q);
            qv[i] = copysignf(q.x, x.x);
            qv[i + 1] = copysignf(q.y, x.y);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) qv[i] = slow_div(v[i], s);      // rare: scale outside the safe exponent range
    }
    uint2 out;
    out.x = static_cast<uint32_t>(cvt_e4m3x2(qv[1], qv[0])) | (static_cast<uint32_t>(cvt_e4m3x2(qv[3], qv[2])) << 16);
    out.y = static_cast<uint32_t>(cvt_e4m3x2(qv[5], qv[4])) | (static_cast<uint32_t>(cvt_e4m3x2(qv[7], qv[6])) << 16);
    return out;
}

template <int BLOCK>
__global__ void __launch_bounds__(kQThreads) quantize_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                             int64_t ld, uint8_t* __restrict__ codes, int64_t ldq,
                                                             float* __restrict__ scales, int64_t lds) {
    constexpr int kLanesPerBlock = BLOCK / 8;
    constexpr int kBlocksPerTile = kQCols / BLOCK;
    __shared__ float sc[kBlocksPerTile][kQRows + 1];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row0 = static_cast<int64_t>(blockIdx.y) * kQRows;
    const int64_t col0 = static_cast<int64_t>(blockIdx.x) * kQCols;

    // each warp walks 4 rows; the row loop is kept rolled so that the kernel stays small in the instruction cache
    // (a fully unrolled version stalled on instruction fetch); occupancy, not prefetching, hides the load latency
#pragma unroll 1
    for (int rr = 0; rr < 4; ++rr) {
        const int r_local = warp * 4 + rr;
        const int64_t row = row0 + r_local;
        uint4 raw[kQIters];
#pragma unroll
        for (int it = 0; it < kQIters; ++it) {
            const int64_t col = col0 + it * 256 + lane * 8;
            raw[it] = (row < rows && col < cols) ? __ldg(reinterpret_cast<const uint4*>(x + row * ld + col)) : make_uint4(0, 0, 0, 0);
        }
        // block maxima of the row's four load rounds, then the scales of all the row's blocks at once: lane L derives
        // scale and reciprocal of block L of the row tile (one divergent region per row instead of one per round)
        constexpr int kBlkPerIt = 32 / kLanesPerBlock;
        constexpr int kBlkPerRow = kQIters * kBlkPerIt;
        static_assert(kBlkPerRow <= 32, "one lane per block of the row tile");
        uint32_t mine = 0;
#pragma unroll
        for (int it = 0; it < kQIters; ++it) {
            const uint32_t m = block_amax_bits<BLOCK>(raw[it]);
            const uint32_t got = __shfl_sync(0xffffffffu, m, (lane % kBlkPerIt) * kLanesPerBlock);
            if (lane / kBlkPerIt == it) mine = got;
        }
        float s_mine = 1.0f, y_mine = 1.0f;
        if (lane < kBlkPerRow && mine != 0u) {
            s_mine = __fdiv_rn(__uint_as_float(mine << 16), 448.0f);
            y_mine = __frcp_rn(s_mine);
        }
#pragma unroll
        for (int it = 0; it < kQIters; ++it) {
            const int64_t col = col0 + it * 256 + lane * 8;
            const bool in = row < rows && col < cols;
            const int blk = it * kBlkPerIt + lane / kLanesPerBlock;
            const float s = __shfl_sync(0xffffffffu, s_mine, blk);
            const float y = __shfl_sync(0xffffffffu, y_mine, blk);
            if (in) {
                *reinterpret_cast<uint2*>(codes + row * ldq + col) = quantize_values(raw[it], s, y);
                if ((lane % kLanesPerBlock) == 0) sc[(it * 256 + lane * 8) / BLOCK][r_local] = s;
            }
        }
    }
    __syncthreads();
    const int64_t kb0 = col0 / BLOCK;
    const int64_t nkb = cols / BLOCK;
    for (int idx = threadIdx.x; idx < kBlocksPerTile * kQRows; idx += kQThreads) {
        const int kb_l = idx / kQRows, r_l = idx % kQRows;
        if (kb0 + kb_l < nkb && row0 + r_l < rows) scales[(kb0 + kb_l) * lds + row0 + r_l] = sc[kb_l][r_l];
    }
}

// ------------------------------------------------------------------------------------------------
// The same quantisation for a matrix stored with the blocks running DOWN its columns (an LM head kept as [d, V]):
// block kb of column v is x[kb B .. kb B + B - 1, v].  The codes leave transposed, [V, ldq] with the block elements
// contiguous, which is the K-major operand the rollout pass wants; the scales leave block-major [d / B, lds] as always.
// A CTA stages a tile of 128 rows x 128 columns in shared memory (16-byte loads along the rows), then thread
// (v, h) walks rows 64 h .. 64 h + 63 of column v: maximum, scale, exact division, sixteen codes per 16-byte store.
// ------------------------------------------------------------------------------------------------
constexpr int kQcTile = 128;
constexpr int kQcPitch = kQcTile + 8;          // uint16 elements per shared-memory row: 272 bytes, 16-byte aligned rows

template <int BLOCK>
__global__ void __launch_bounds__(256) quantize_cols_kernel(const __nv_bfloat16* __restrict__ x, int64_t K, int64_t N, int64_t ld,
                                                            uint8_t* __restrict__ codes, int64_t ldq,
                                                            float* __restrict__ scales, int64_t lds) {
    __shared__ __align__(16) uint16_t tile[kQcTile][kQcPitch];
    __shared__ uint32_t half_max[2][kQcTile];
    const int tid = threadIdx.x;
    const int64_t k0 = static_cast<int64_t>(blockIdx.y) * kQcTile, v0 = static_cast<int64_t>(blockIdx.x) * kQcTile;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c = tid + 256 * i, r = c >> 4, c8 = (c & 15) * 8;
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (k0 + r < K && v0 + c8 < N) raw = __ldg(reinterpret_cast<const uint4*>(x + (k0 + r) * ld + v0 + c8));
        *reinterpret_cast<uint4*>(&tile[r][c8]) = raw;
    }
    __syncthreads();
    const int v = tid & (kQcTile - 1), h = tid >> 7;
    constexpr int kRun = BLOCK < 64 ? BLOCK : 64;          // rows of one block inside this thread's 64
    constexpr int kRuns = 64 / kRun;
    uint32_t amax[kRuns];
#pragma unroll
    for (int b = 0; b < kRuns; ++b) {
        uint32_t m = 0;
#pragma unroll 8
        for (int j = 0; j < kRun; ++j) m = max(m, static_cast<uint32_t>(tile[64 * h + b * kRun + j][v]) & 0x7FFFu);
        amax[b] = m;
    }
    if (BLOCK == 128) {                                      // the block spans both halves of the column
        half_max[h][v] = amax[0];
        __syncthreads();
        amax[0] = max(half_max[0][v], half_max[1][v]);
    }
    const bool in = v0 + v < N;
#pragma unroll
    for (int b = 0; b < kRuns; ++b) {
        float s = 1.0f, y = 1.0f;
        if (amax[b] != 0u) {
            s = __fdiv_rn(__uint_as_float(amax[b] << 16), 448.0f);
            y = __frcp_rn(s);
        }
        const bool fast = s > 0x1p-100f && s < 0x1p100f;
#pragma unroll
        for (int g = 0; g < kRun / 16; ++g) {
            float q[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float xv = __uint_as_float(static_cast<uint32_t>(tile[64 * h + b * kRun + g * 16 + j][v]) << 16);
                q[j] = fast ? exact_div(xv, s, y) : slow_div(xv, s);
            }
            uint4 out;
            out.x = static_cast<uint32_t>(cvt_e4m3x2(q[1], q[0])) | (static_cast<uint32_t>(cvt_e4m3x2(q[3], q[2])) << 16);
            out.y = static_cast<uint32_t>(cvt_e4m3x2(q[5], q[4])) | (static_cast<uint32_t>(cvt_e4m3x2(q[7], q[6])) << 16);
            out.z = static_cast<uint32_t>(cvt_e4m3x2(q[9], q[8])) | (static_cast<uint32_t>(cvt_e4m3x2(q[11], q[10])) << 16);
            out.w = static_cast<uint32_t>(cvt_e4m3x2(q[13], q[12])) | (static_cast<uint32_t>(cvt_e4m3x2(q[15], q[14])) << 16);
            if (in && k0 + 64 * h + b * kRun + g * 16 < K)
                *reinterpret_cast<uint4*>(codes + (v0 + v) * ldq + k0 + 64 * h + b * kRun + g * 16) = out;
        }
        const int64_t kb = (k0 + 64 * h + b * kRun) / BLOCK;
        if (in && kb * BLOCK < K && (BLOCK < 128 || h == 0)) scales[kb * lds + v0 + v] = s;
    }
}

// ------------------------------------------------------------------------------------------------
// Microscaling FP8: 32 consecutive elements share a power-of-two scale 2^X, X = floor(log2 amax) - 8, stored as the
// biased exponent X + 127 (clamped to 0..254; 127 for an all-zero block); the elements are x / 2^X on the E4M3 grid
// (round to nearest even, saturating).  With bf16 inputs everything is exact integer work on exponent fields: the
// block's amax pattern gives the scale code, and the multiplier 2^-X is a float built from its exponent field.
// Four lanes (8 elements each) form a block.  The scale codes leave in the order the block-scaled MMA wants them:
// chunks of 128 rows x 4 blocks, byte (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4 of chunk (r / 128, kb / 4); the two
// chunks of a 256-row group are adjacent: chunk start ((r / 256) * (cols / 128) + kb / 4) * 1024 + ((r % 256) / 128) * 512.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kQThreads) quantize_mx_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                                int64_t ld, uint8_t* __restrict__ codes, int64_t ldq,
                                                                uint8_t* __restrict__ scales) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row0 = static_cast<int64_t>(blockIdx.y) * kQRows;
    const int64_t col0 = static_cast<int64_t>(blockIdx.x) * kQCols;
    const int64_t nk4 = cols / 128;
#pragma unroll 1
    for (int rr = 0; rr < 4; ++rr) {
        const int64_t row = row0 + warp * 4 + rr;
        if (row >= rows) break;
#pragma unroll
        for (int it = 0; it < kQIters; ++it) {
            const int64_t col = col0 + it * 256 + lane * 8;
            const bool in = col < cols;                     // cols is a multiple of 128: a block is wholly in or out
            const uint4 raw = in ? __ldg(reinterpret_cast<const uint4*>(x + row * ld + col)) : make_uint4(0, 0, 0, 0);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t m = __vmaxu2(__vmaxu2(w[0] & 0x7FFF7FFFu, w[1] & 0x7FFF7FFFu), __vmaxu2(w[2] & 0x7FFF7FFFu, w[3] & 0x7FFF7FFFu));
            m = max(m & 0xFFFFu, m >> 16);
            m = max(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = max(m, __shfl_xor_sync(0xffffffffu, m, 2));
            const int e = static_cast<int>(m >> 7);         // biased exponent of amax (0 for zero and subnormals)
            const int code = m == 0u ? 127 : max(e - 8, 0);
            const float mult = __uint_as_float(static_cast<uint32_t>(254 - code) << 23);      // 2^(127 - code), exact
            if (!in) continue;
            float q[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                q[2 * i] = __uint_as_float(w[i] << 16) * mult;
                q[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u) * mult;
            }
            uint2 out;
            out.x = static_cast<uint32_t>(cvt_e4m3x2(q[1], q[0])) | (static_cast<uint32_t>(cvt_e4m3x2(q[3], q[2])) << 16);
            out.y = static_cast<uint32_t>(cvt_e4m3x2(q[5], q[4])) | (static_cast<uint32_t>(cvt_e4m3x2(q[7], q[6])) << 16);
            *reinterpret_cast<uint2*>(codes + row * ldq + col) = out;
            if ((lane & 3) == 0) {
                const int64_t kb = col / 32;
                scales[((row >> 8) * nk4 + (kb >> 2)) * 1024 + ((row >> 7) & 1) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4 +
                       (kb & 3)] = static_cast<uint8_t>(code);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Microscaling FP4: as above with E2M1 elements (X = floor(log2 amax) - 2), two codes per byte, the element with
// the lower index in the low nibble.  A lane turns 8 elements into 4 bytes.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cvt_e2m1x2(float hi, float lo) {
    uint32_t r;
    asm("{\n\t.reg .b8 t;\n\tcvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\tcvt.u32.u8 %0, t;\n\t}" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(kQThreads) quantize_mxfp4_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                                   int64_t ld, uint8_t* __restrict__ codes, int64_t ldq,
                                                                   uint8_t* __restrict__ scales) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row0 = static_cast<int64_t>(blockIdx.y) * kQRows;
    const int64_t col0 = static_cast<int64_t>(blockIdx.x) * kQCols;
    const int64_t nk4 = cols / 128;
#pragma unroll 1
    for (int rr = 0; rr < 4; ++rr) {
        const int64_t row = row0 + warp * 4 + rr;
        if (row >= rows) break;
#pragma unroll
        for (int it = 0; it < kQIters; ++it) {
            const int64_t col = col0 + it * 256 + lane * 8;
            const bool in = col < cols;
            const uint4 raw = in ? __ldg(reinterpret_cast<const uint4*>(x + row * ld + col)) : make_uint4(0, 0, 0, 0);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t m = __vmaxu2(__vmaxu2(w[0] & 0x7FFF7FFFu, w[1] & 0x7FFF7FFFu), __vmaxu2(w[2] & 0x7FFF7FFFu, w[3] & 0x7FFF7FFFu));
            m = max(m & 0xFFFFu, m >> 16);
            m = max(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = max(m, __shfl_xor_sync(0xffffffffu, m, 2));
            const int e = static_cast<int>(m >> 7);
            const int code = m == 0u ? 127 : max(e - 2, 0);
            const float mult = __uint_as_float(static_cast<uint32_t>(254 - code) << 23);      // 2^(127 - code), exact
            if (!in) continue;
            uint32_t out = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __uint_as_float(w[i] << 16) * mult, hi = __uint_as_float(w[i] & 0xFFFF0000u) * mult;
                out |= cvt_e2m1x2(hi, lo) << (8 * i);
            }
            *reinterpret_cast<uint32_t*>(codes + row * ldq + col / 2) = out;
            if ((lane & 3) == 0) {
                const int64_t kb = col / 32;
                scales[((row >> 8) * nk4 + (kb >> 2)) * 1024 + ((row >> 7) & 1) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4 +
                       (kb & 3)] = static_cast<uint8_t>(code);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Per-tensor dynamic scaling: one scale for the whole matrix.  Pass 1 folds max|x| (as a bf16 bit pattern; the
// patterns of non-negative values order like the values, so an integer atomicMax is exact and order-free)
// into the word that will hold the scale, pass 2 turns it into s = amax / 448, pass 3 quantises.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) tensor_amax_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols, int64_t ld,
                                                           uint32_t* __restrict__ amax_bits) {
    const int64_t vec_per_row = cols / 8;
    const int64_t total = rows * vec_per_row;
    uint32_t m = 0;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / vec_per_row, c = (i % vec_per_row) * 8;
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(x + r * ld + c));
        m = __vmaxu2(m, __vmaxu2(__vmaxu2(w.x & 0x7FFF7FFFu, w.y & 0x7FFF7FFFu), __vmaxu2(w.z & 0x7FFF7FFFu, w.w & 0x7FFF7FFFu)));
    }
    m = max(m & 0xFFFFu, m >> 16);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((threadIdx.x & 31) == 0 && m != 0u) atomicMax(amax_bits, m);
}

__global__ void tensor_scale_kernel(uint32_t* scale_word) {
    const uint32_t m = *scale_word;                        // bf16 pattern of max|x|
    const float s = (m == 0u) ? 1.0f : __fdiv_rn(__uint_as_float(m << 16), 448.0f);
    *reinterpret_cast<float*>(scale_word) = s;
}

__global__ void __launch_bounds__(256) tensor_quantize_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                               int64_t ld, uint8_t* __restrict__ codes, int64_t ldq,
                                                               const float* __restrict__ scale) {
    const float s = *scale;
    const bool fast = s > 0x1p-100f && s < 0x1p100f;
    const float y = fast ? __frcp_rn(s) : 0.f;
    const int64_t vec_per_row = cols / 8;
    const int64_t total = rows * vec_per_row;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / vec_per_row, c = (i % vec_per_row) * 8;
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(x + r * ld + c));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        float qv[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xFFFF0000u);
            qv[2 * k] = fast ? exact_div(lo, s, y) : slow_div(lo, s);
            qv[2 * k + 1] = fast ? exact_div(hi, s, y) : slow_div(hi, s);
        }
        uint2 out;
        out.x = static_cast<uint32_t>(cvt_e4m3x2(qv[1], qv[0])) | (static_cast<uint32_t>(cvt_e4m3x2(qv[3], qv[2])) << 16);
        out.y = static_cast<uint32_t>(cvt_e4m3x2(qv[5], qv[4])) | (static_cast<uint32_t>(cvt_e4m3x2(qv[7], qv[6])) << 16);
        *reinterpret_cast<uint2*>(codes + r * ldq + c) = out;
    }
}

// ------------------------------------------------------------------------------------------------
// Merge of the per-split (max, sum-exp, target-logit) triples into lp and lse.
// ------------------------------------------------------------------------------------------------
__global__ void combine_kernel(const float* __restrict__ part_m, const float* __restrict__ part_s,
                               const float* __restrict__ part_z, int nparts, int64_t part_ld,
                               const uint8_t* __restrict__ mask, int64_t T, float* __restrict__ lp,
                               float* __restrict__ lse, uint32_t* status) {
    uint32_t flags = 0;
    for (int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < T;
         t += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        float out_lp = 0.f, out_lse = 0.f;
        if (mask[t]) {
            float M = -INFINITY, zy = -INFINITY;
            for (int j = 0; j < nparts; ++j) {
                M = fmaxf(M, part_m[j * part_ld + t]);
                zy = fmaxf(zy, part_z[j * part_ld + t]);
            }
            float S = 0.f;
            for (int j = 0; j < nparts; ++j) S += part_s[j * part_ld + t] * expf(part_m[j * part_ld + t] - M);
            out_lse = M + logf(S);
            if (zy == -INFINITY) {
                out_lp = 0.f;                       // token id out of range: flagged by the producer kernel
            } else {
                out_lp = zy - out_lse;
            }
            if (!isfinite(out_lse) || !isfinite(out_lp)) {
                // a non-finite hidden state or weight reached this row: flag it, give it the neutral log-prob, and mark
                // its log-sum-exp so that the backward pass leaves the row out (gradient factor 0)
                flags |= AIS_FLAG_NONFINITE;
                out_lp = 0.f;
                out_lse = __int_as_float(0x7fc00000);
            }
        }
        lp[t] = out_lp;
        if (lse) lse[t] = out_lse;
    }
    if (flags && status) atomicOr(status, flags);
}

// ------------------------------------------------------------------------------------------------
// Segmented reductions: valid rows per sequence and group-relative advantages (Eq. grpo_adv).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// Block-wide sum in a fixed order (lanes by butterfly, then warps 0..n-1 serially); result valid in thread 0.
__device__ double block_sum(double v, double* scratch /*[32]*/) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        for (int i = 0; i < nw; ++i) tot += scratch[i];
    }
    return tot;
}

// Sum of partials[b * stride + offset] over b < nblocks by one warp, in a fixed order: lane l takes blocks l, l + 32, ...
// (loaded sixteen at a time so that the loads overlap), then the shuffle tree of warp_sum.
__device__ __forceinline__ double warp_ordered_sum(const double* __restrict__ partials, int nblocks, int stride, int offset, int lane) {
    double acc = 0.0;
    for (int base = lane; base < nblocks; base += 32 * 16) {
        double v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int b = base + 32 * j;
            v[j] = b < nblocks ? partials[b * stride + offset] : 0.0;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) acc += v[j];
    }
    return warp_sum(acc);
}

// Valid rows of each sequence: one warp per sequence, 4 mask bytes per lane and load where the row range allows it.
__global__ void __launch_bounds__(256) seq_count_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ seq_offsets,
                                                         int S, int32_t* __restrict__ n_valid_seq) {
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= S) return;
    const int lane = threadIdx.x & 31;
    const int64_t b = seq_offsets[s], e = seq_offsets[s + 1];
    const uintptr_t base = reinterpret_cast<uintptr_t>(mask);
    const int64_t b4 = b + static_cast<int64_t>((4 - ((base + b) & 3)) & 3);          // first row on a 4-byte boundary
    int cnt = 0;
    for (int64_t t = b + lane; t < (b4 < e ? b4 : e); t += 32) cnt += mask[t] != 0;
    const int64_t nwords = b4 < e ? (e - b4) / 4 : 0;
    for (int64_t i = lane; i < nwords; i += 32) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(mask + b4 + 4 * i);
        cnt += ((w & 0xFFu) != 0) + ((w & 0xFF00u) != 0) + ((w & 0xFF0000u) != 0) + ((w & 0xFF000000u) != 0);
    }
    for (int64_t t = b4 + 4 * nwords + lane; t < e; t += 32) cnt += (t >= b4 && mask[t] != 0);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if (lane == 0) n_valid_seq[s] = cnt;
}

// Group-relative advantages (Eq. grpo_adv): one thread per sequence.  With `zero_counts` the per-sequence row
// counts are cleared for the moments kernel, which adds them up.
__global__ void adv_kernel(const float* __restrict__ rewards, int S, int G, int adv_std_norm, float eps, float* __restrict__ adv,
                           int32_t* __restrict__ zero_counts) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    if (zero_counts) zero_counts[s] = 0;
    if (!rewards || !adv) return;
    const int g0 = (s / G) * G;
    double mean = 0.0;
    for (int j = 0; j < G; ++j) mean += static_cast<double>(rewards[g0 + j]);
    mean /= G;
    double a = static_cast<double>(rewards[s]) - mean;
    if (adv_std_norm) {
        double var = 0.0;
        for (int j = 0; j < G; ++j) {
            const double dlt = static_cast<double>(rewards[g0 + j]) - mean;
            var += dlt * dlt;
        }
        a /= (sqrt(var / G) + static_cast<double>(eps));
    }
    adv[s] = static_cast<float>(a);
}

// Sequence-level importance weight (Eq. is-weight): log w(x) = sum over the valid rows of a sequence of
// lp_train - lp_roll.  One warp per sequence, double accumulation in a fixed order.
__global__ void __launch_bounds__(256) seq_logw_kernel(const float* __restrict__ lp_train, const float* __restrict__ lp_roll,
                                                        const uint8_t* __restrict__ mask, const int32_t* __restrict__ seq_offsets,
                                                        int S, float* __restrict__ seq_logw) {
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= S) return;
    const int lane = threadIdx.x & 31;
    double acc = 0.0;
    for (int64_t t = static_cast<int64_t>(seq_offsets[s]) + lane; t < seq_offsets[s + 1]; t += 32)
        if (mask[t]) acc += static_cast<double>(lp_train[t]) - static_cast<double>(lp_roll[t]);
    acc = warp_sum(acc);
    if (lane == 0) seq_logw[s] = static_cast<float>(acc);
}

// One byte per 128-row tile: does any row of the tile need computing?  (mask != 0 / gradient factor != 0)
template <typename T>
__global__ void tile_flags_kernel(const T* __restrict__ pred, int64_t n, uint8_t* __restrict__ flags) {
    const int64_t tile = blockIdx.x;
    const int64_t i = tile * 128 + threadIdx.x;
    const int any = __syncthreads_or(i < n && pred[i] != T(0));
    if (threadIdx.x == 0) flags[tile] = any ? 1 : 0;
}

__device__ __forceinline__ int seq_of_row(const int32_t* __restrict__ seq_offsets, int S, int64_t t) {
    int lo = 0, hi = S;                 // largest s with seq_offsets[s] <= t
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (static_cast<int64_t>(seq_offsets[mid]) <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// ------------------------------------------------------------------------------------------------
// Whole-batch masked moments in double precision, fixed grid and fixed summation order.
//   0 N   1 sum w   2 sum w^2   3 sum |D|   4 sum A   5 sum A^2   6 sum Aw   7 sum (Aw)^2
//   8 sum (lp_roll - lp_train)   9 sum |exp(lp_train) - exp(lp_roll)|
// ------------------------------------------------------------------------------------------------
// Rows are read VEC at a time (16-byte loads of the two log-prob vectors, one 4-byte load of the mask); the
// sequence of a group's first row comes from a binary search and the following rows only step forward.  The
// exponentials are evaluated in fp32 (the inputs are fp32 and the sums need seven digits at most), the sums
// themselves in fp64.  Two groups are in flight per thread so that the fixed grid keeps HBM busy on long batches.
// rho - 1 = e^x - 1 for a run of n rows.  When every |x| of the run is at most 2^-6 a short series gives it to fp32
// accuracy RELATIVE TO ITSELF (e^x - 1 from a rounded e^x would be good to 1e-7 absolute only, i.e. to a thousandth of a
// weight that differs from 1 by 1e-4); otherwise the fast exponential is used, as everywhere else in these kernels.
template <int N>
__device__ __forceinline__ void rho_minus_one(const float (&x)[N], float (&u)[N]) {
    float amax = 0.f;
#pragma unroll
    for (int j = 0; j < N; ++j) amax = fmaxf(amax, fabsf(x[j]));
    if (amax <= 0x1p-6f) {
#pragma unroll
        for (int j = 0; j < N; ++j)
            u[j] = x[j] * fmaf(x[j], fmaf(x[j], fmaf(x[j], 1.0f / 24.0f, 1.0f / 6.0f), 0.5f), 1.0f);
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j) {
            float e;
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x[j] * 1.4426950408889634f));
            u[j] = e - 1.0f;
        }
    }
}

// Sums of w and w^2 over a short run of rows, in double precision, from fp32 sums of shifted values.  The weights
// enter as u = w - 1 (rho_minus_one above, truncated at C - 1); the run is summed as v = u - p and v^2 about the pivot
// p = u of its first valid row:  with P = 1 + p,  sum w = n P + sum v  and  sum w^2 = n P^2 + 2 P sum v + sum v^2.
// The fp32 roundings then scale with the spread of the run and with |w - 1|, not with the size of w, so that the
// variance formed later as E[w^2] - E[w]^2 in fp64 keeps its digits when the weights differ by 1e-4 of their size,
// and is exactly zero when they are all equal.  All rows of the run share the advantage A.
//   acc: 0 N   1 sum w   2 sum w^2   4 sum A   5 sum A^2   6 sum A w   7 sum (A w)^2
__device__ __forceinline__ void add_run(double* acc, int n, float p, float sv, float sv2, float A) {
    const double nd = static_cast<double>(n), P = 1.0 + static_cast<double>(p), svd = static_cast<double>(sv);
    const double Ad = static_cast<double>(A);
    const double sw = fma(nd, P, svd);
    const double sw2 = static_cast<double>(sv2) + P * fma(nd, P, 2.0 * svd);
    acc[0] += nd;
    acc[1] += sw;
    acc[2] += sw2;
    acc[4] = fma(Ad, nd, acc[4]);
    acc[5] = fma(Ad * Ad, nd, acc[5]);
    acc[6] = fma(Ad, sw, acc[6]);
    acc[7] = fma(Ad * Ad, sw2, acc[7]);
}

template <int VEC>
struct RowGroup {
    float lt[VEC], lr[VEC];
    uint8_t mk[VEC];
    bool any;
};
template <int VEC>
__device__ __forceinline__ RowGroup<VEC> load_group(const float* __restrict__ lp_train, const float* __restrict__ lp_roll,
                                                    const uint8_t* __restrict__ mask, int64_t g) {
    RowGroup<VEC> r;
    if (VEC == 4) {
        const float4 a = reinterpret_cast<const float4*>(lp_train)[g];
        const float4 b = reinterpret_cast<const float4*>(lp_roll)[g];
        const uchar4 m = reinterpret_cast<const uchar4*>(mask)[g];
        r.lt[0] = a.x; r.lt[1 % VEC] = a.y; r.lt[2 % VEC] = a.z; r.lt[3 % VEC] = a.w;
        r.lr[0] = b.x; r.lr[1 % VEC] = b.y; r.lr[2 % VEC] = b.z; r.lr[3 % VEC] = b.w;
        r.mk[0] = m.x; r.mk[1 % VEC] = m.y; r.mk[2 % VEC] = m.z; r.mk[3 % VEC] = m.w;
    } else {
        r.lt[0] = lp_train[g]; r.lr[0] = lp_roll[g]; r.mk[0] = mask[g];
    }
    r.any = false;
#pragma unroll
    for (int j = 0; j < VEC; ++j) r.any |= (r.mk[j] != 0);
    return r;
}

template <int VEC>
__global__ void __launch_bounds__(kDiagThreads) moments_kernel(const float* __restrict__ lp_train, const float* __restrict__ lp_roll,
                                                                const uint8_t* __restrict__ mask,
                                                                const int32_t* __restrict__ seq_offsets,
                                                                const float* __restrict__ adv, int64_t T, int S, float C,
                                                                double* __restrict__ partials, int32_t* __restrict__ n_valid_seq,
                                                                const float* __restrict__ seq_logw) {
    __shared__ double scratch[32];
    double acc[kNumMoments];
#pragma unroll
    for (int i = 0; i < kNumMoments; ++i) acc[i] = 0.0;
    // Every warp owns a contiguous range of row groups and its lanes interleave inside it, so a lane's rows only
    // move forward: one binary search for its first group, then the sequence index steps (the next boundary is kept
    // in a register).  Valid rows are counted per sequence on the way (integer atomics: the result does not depend
    // on their order).  The first-order sums (|D|, D, |dp|) take runs of at most 64 rows in fp32 and those short sums go
    // into the fp64 accumulators; the sums behind the three variances are formed per group of rows by add_run.
    int sq = -1, cur = -1, cnt = 0;
    int64_t next_b = 0;                                   // first row of sequence sq + 1 (or "never" for the last one)
    float f[kNumMoments];
    auto flush = [&]() {
        if (n_valid_seq && cur >= 0 && cnt > 0) atomicAdd(&n_valid_seq[cur], cnt);
        cnt = 0;
    };
    // fp32 runs are kept only for the three first-order sums (3, 8, 9); the sums behind the variances go through add_run
    auto clear = [&]() { f[3] = 0.f; f[8] = 0.f; f[9] = 0.f; };
    auto commit = [&]() {
        acc[3] += static_cast<double>(f[3]);
        acc[8] += static_cast<double>(f[8]);
        acc[9] += static_cast<double>(f[9]);
    };
    auto seek = [&](int64_t t) {
        if (sq < 0) {
            sq = seq_of_row(seq_offsets, S, t);
            next_b = sq + 1 < S ? static_cast<int64_t>(seq_offsets[sq + 1]) : (int64_t(1) << 62);
        }
        while (t >= next_b) {
            ++sq;
            next_b = sq + 1 < S ? static_cast<int64_t>(seq_offsets[sq + 1]) : (int64_t(1) << 62);
        }
    };
    auto add_row = [&](float lt, float lr, float A) {
        const float dl[1] = {lt - lr};
        float u[1];
        rho_minus_one(dl, u);                              // rho - 1; |e^lt - e^lr| = e^lr |rho - 1|
        // sequence-level variant: every row carries its sequence's truncated weight instead of its own
        const float uw = seq_logw ? fminf(__expf(seq_logw[sq]), C) - 1.0f : fminf(u[0], C - 1.0f);
        add_run(acc, 1, uw, 0.f, 0.f, A);
        f[3] += fabsf(dl[0]);
        f[8] -= dl[0];
        f[9] = fmaf(__expf(lr), fabsf(u[0]), f[9]);
        if (sq != cur) { flush(); cur = sq; }
        ++cnt;
    };
    auto add_group = [&](const RowGroup<VEC>& r, int64_t g) {
        if (!r.any) return;
        const int64_t t0 = g * VEC;
        seek(t0);
        if (VEC > 1 && t0 + VEC <= next_b) {
            // the usual case, all rows of the group in one sequence: one advantage and one weight source for the
            // group, masked rows drop out by selection, and the sums that involve A follow from sum w and sum w^2
            const float A = adv[sq];
            const float useq = seq_logw ? fminf(__expf(seq_logw[sq]), C) - 1.0f : 0.f;
            float dl[VEC], u[VEC];
#pragma unroll
            for (int j = 0; j < VEC; ++j) dl[j] = r.mk[j] != 0 ? r.lt[j] - r.lr[j] : 0.f;
            rho_minus_one(dl, u);
            float p = 0.f;
            int n = 0;
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                const bool on = r.mk[j] != 0;
                f[3] += fabsf(dl[j]);
                f[8] -= dl[j];
                f[9] += on ? __expf(r.lr[j]) * fabsf(u[j]) : 0.f;
                u[j] = seq_logw ? useq : fminf(u[j], C - 1.0f);
                if (on && n == 0) p = u[j];                        // pivot: the first valid row
                n += on ? 1 : 0;
            }
            float sv = 0.f, sv2 = 0.f;
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                const float v = r.mk[j] != 0 ? u[j] - p : 0.f;
                sv += v;
                sv2 = fmaf(v, v, sv2);
            }
            add_run(acc, n, p, sv, sv2, A);
            if (sq != cur) { flush(); cur = sq; }
            cnt += n;
            return;
        }
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            if (r.mk[j]) {
                seek(t0 + j);
                add_row(r.lt[j], r.lr[j], adv[sq]);
            }
        }
    };
    const int lane = threadIdx.x & 31;
    const int64_t ngroups = T / VEC;
    const int64_t nwarps = static_cast<int64_t>(gridDim.x) * (blockDim.x >> 5);
    const int64_t gw = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t per = ((ngroups + nwarps - 1) / nwarps + 63) / 64 * 64;             // groups per warp
    const int64_t g_end = (gw + 1) * per < ngroups ? (gw + 1) * per : ngroups;
    int64_t g = gw * per + lane;
    clear();
    for (int pass = 0; g + 32 < g_end; g += 64) {                                      // two groups in flight per lane
        const RowGroup<VEC> r0 = load_group<VEC>(lp_train, lp_roll, mask, g);
        const RowGroup<VEC> r1 = load_group<VEC>(lp_train, lp_roll, mask, g + 32);
        add_group(r0, g);
        add_group(r1, g + 32);
        if ((++pass & 7) == 0) {                                                       // at most 64 rows per fp32 run
            commit();
            clear();
        }
    }
    if (g < g_end) add_group(load_group<VEC>(lp_train, lp_roll, mask, g), g);
    flush();
    // rows after the last whole group: the first threads of the grid, one row each
    {
        const int64_t t = ngroups * VEC + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
        if (t < T && mask[t]) {
            sq = -1;
            cur = -1;
            seek(t);
            add_row(lp_train[t], lp_roll[t], adv[sq]);
            flush();
        }
    }
    commit();
    for (int i = 0; i < kNumMoments; ++i) {
        const double tot = block_sum(acc[i], scratch);
        if (threadIdx.x == 0) partials[blockIdx.x * kNumMoments + i] = tot;
    }
}

// The same moments for 16-byte aligned inputs, fed by bulk asynchronous copies: a block walks a contiguous range of
// 2048-row tiles; thread 0 keeps three tiles (two log-prob vectors and the mask bytes, 18 KB each) in flight into a
// ring of shared-memory stages, completion arrives on one mbarrier per stage, and every thread takes the eight rows
// 8 tid .. 8 tid + 7 of each tile from shared memory.  Memory latency is carried by the copies in flight (54 KB per
// block, four blocks per SM) instead of by registers, and the work per row is kept to about twenty instructions
// (flush-to-zero exponentials, 32-bit row indices, the group's sequence looked up before the data arrives, the
// per-tile bookkeeping shared by eight rows), because at 9 bytes per row the instruction issue rate is the next limit
// after HBM.  Rows after the last whole tile are read directly.  Summation order is fixed by the grid as above.
constexpr int kMomRows = 2048;
constexpr int kMomStages = 3;
constexpr int kMomStageBytes = kMomRows * 9;
constexpr int kMomSmemBytes = kMomStages * kMomStageBytes + 128;


// (add2 / sub2 / mul2 / fma2: the packed two-element fp32 instructions, ptx.cuh.)  The staged kernel is bound by
// instruction issue right after HBM, and half of its per-row work is additions, multiplications and multiply-adds.
__device__ __forceinline__ float ex2_ftz(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The waiting part of a bounded mbarrier wait, kept out of line so that the loop around it stays small.
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, int* abort_flag) {
    return mbar_wait(bar, parity, abort_flag);
}

// SEQ: every row carries its sequence's truncated weight instead of its own.  EXACT: the second of two launches (see
// add_rows below): a block returns at once unless the first launch found all of its log-probability gaps tiny.
template <bool SEQ, bool EXACT>
__global__ void __launch_bounds__(kDiagThreads, 4) moments_staged_kernel(const float* __restrict__ lp_train,
                                                                         const float* __restrict__ lp_roll,
                                                                         const uint8_t* __restrict__ mask,
                                                                         const int32_t* __restrict__ seq_offsets,
                                                                         const float* __restrict__ adv, int T, int S, float C,
                                                                         double* __restrict__ partials,
                                                                         int32_t* __restrict__ n_valid_seq,
                                                                         const float* __restrict__ seq_logw) {
    static_assert(kDiagThreads * 8 == kMomRows, "one 8-row group per thread and tile");
    extern __shared__ __align__(128) uint8_t stages[];          // kMomStages stages, then the barriers
    uint64_t* full = reinterpret_cast<uint64_t*>(stages + kMomStages * kMomStageBytes);
    __shared__ double scratch[32];
    __shared__ int abort_flag;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int ntiles = T / kMomRows;
    const int per = (ntiles + gridDim.x - 1) / gridDim.x;
    const int tile0 = blockIdx.x * per < ntiles ? blockIdx.x * per : ntiles;
    const int tile1 = tile0 + per < ntiles ? tile0 + per : ntiles;
    if (EXACT) {
        // slots 10 and 11 of the block's partial sums: its groups with a gap above 2^-6 and its groups of valid rows without,
        // as counted by the first launch; slot 0 is NaN when that launch gave up on a wait
        const double big = partials[blockIdx.x * kNumMoments + 10], small = partials[blockIdx.x * kNumMoments + 11];
        const double n0 = partials[blockIdx.x * kNumMoments];
        if (big != 0.0 || small == 0.0 || n0 != n0) return;
    }
    if (tid == 0) {
        for (int i = 0; i < kMomStages; ++i) mbar_init(&full[i], 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    auto issue = [&](int tile, int st) {               // thread 0: the three copies of one tile onto the stage's barrier
        uint8_t* dst = stages + st * kMomStageBytes;
        const size_t r0 = static_cast<size_t>(tile) * kMomRows;
        mbar_expect_tx(&full[st], kMomStageBytes);
        bulk_load(dst, lp_train + r0, kMomRows * 4, &full[st]);
        bulk_load(dst + kMomRows * 4, lp_roll + r0, kMomRows * 4, &full[st]);
        bulk_load(dst + kMomRows * 8, mask + r0, kMomRows, &full[st]);
    };

    // Everything a thread sums stays in fp32 while it walks its tiles and turns into fp64 once, at the end: the first-order
    // sums (|D|, D, |dp|) as they are, the sums behind the three variances as SHIFTED sums about pivots taken from the
    // thread's own data -- v = (w - 1) - pivot for the weights, dA = A - A_pivot for the advantages, and
    // x = A w - A_pivot (1 + pivot) = A v + dA (1 + pivot) for their product -- so that the fp32 roundings scale with the
    // spread of the data and not with its size, and are exactly zero when all rows are equal.  A thread sees at most
    // T / 151,552 rows.
    float f3, f9, g_v, g_v2, g_dA, g_dA2, g_x, g_x2;
    F2 f8p;                                             // sum of D, two rows at a time
    int nrows;                                          // valid rows of the thread
    int nbig, nsmall;                                   // groups with a gap above 2^-6 / with all gaps below (see add_rows)
    float pivot, A_pivot, dA;
    bool have_pivot;                                    // both pivots come from the thread's first group with a valid row
    constexpr int kNever = 0x7fffffff;
    int sq, cur;
    int next_b;                                         // first row of sequence sq + 1 (or "never" for the last one)
    float A = 0.f, wseq = 0.f;                          // advantage and sequence-level weight of sequence `cur`
    int wsq = -1, wcnt = 0;                             // lane 0: valid rows of the warp's strips counted for sequence wsq
    auto reset = [&]() {
        f3 = f9 = g_v = g_v2 = g_dA = g_dA2 = g_x = g_x2 = 0.f;
        f8p = F2{0.f, 0.f};
        nrows = 0;
        nbig = 0;
        nsmall = 0;
        pivot = A_pivot = dA = 0.f;
        have_pivot = false;
        sq = cur = -1;
        next_b = 0;
    };
    reset();
    auto seek = [&](int t) {
        if (sq < 0) {
            sq = seq_of_row(seq_offsets, S, t);
            next_b = sq + 1 < S ? seq_offsets[sq + 1] : kNever;
        }
        while (t >= next_b) {
            ++sq;
            next_b = sq + 1 < S ? seq_offsets[sq + 1] : kNever;
        }
    };
    auto enter = [&]() {                                // the row's sequence becomes the current one
        if (sq != cur) {
            cur = sq;
            A = adv[sq];
            dA = have_pivot ? A - A_pivot : 0.f;
            if (SEQ) wseq = fminf(__expf(seq_logw[sq]), C);
        }
    };
    // Sums over the rows of a group whose mask byte (rows 0..3 in `m0`, 4..7 in `m1`) is set, all of them in sequence
    // `cur`; returns how many they are.  Rows go two at a time through the packed fp32 instructions.  The weight pivot
    // is w - 1 of the first valid row this thread meets and stays: any value of the data serves.
    // rho - 1 comes from the fast exponential, which is good to 1e-7 ABSOLUTE: enough unless the gaps D themselves are
    // tiny, when it is only a thousandth of a weight that differs from 1 by 1e-4.  The EXACT form of this kernel uses a
    // short series for groups whose |D| are all at most 2^-6 (their sum is), which gives e^D - 1 to fp32 accuracy
    // relative to itself.  It is slower (the second path costs registers and scheduling freedom: a fifth of the
    // bandwidth), so the fast form runs first and counts each block's groups above 2^-6, and the exact form is launched
    // after it: there only the blocks that met no such group walk their tiles again and replace their partial sums.
    auto add_rows = [&](const float (&lt)[8], const float (&lr)[8], uint32_t m0, uint32_t m1) -> int {
        const uint32_t v0 = __vcmpne4(m0, 0u), v1 = __vcmpne4(m1, 0u);     // 0xFF in the byte of every valid row
        const int n = (__popc(v0) + __popc(v1)) >> 3;
        bool on[8];
        float dl[8], u[8], e[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) on[j] = ((j < 4 ? v0 : v1) & (0x80u << (8 * (j & 3)))) != 0u;
        float s3 = 0.f;
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const F2 d = sub2(F2{lt[j], lt[j + 1]}, F2{lr[j], lr[j + 1]});
            dl[j] = on[j] ? d.x : 0.f;                             // a masked row enters with D = 0
            dl[j + 1] = on[j + 1] ? d.y : 0.f;
            f8p = add2(f8p, F2{dl[j], dl[j + 1]});
            s3 += fabsf(dl[j]);
            s3 += fabsf(dl[j + 1]);
        }
        f3 += s3;
        if (EXACT && s3 <= 0x1p-6f) {
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const F2 x = {dl[j], dl[j + 1]};
                F2 q = fma2(x, F2{1.0f / 24.0f, 1.0f / 24.0f}, F2{1.0f / 6.0f, 1.0f / 6.0f});
                q = fma2(x, q, F2{0.5f, 0.5f});
                q = fma2(x, q, F2{1.0f, 1.0f});
                q = mul2(x, q);
                u[j] = q.x;
                u[j + 1] = q.y;
            }
        } else {
            if (!EXACT) {
                nbig += s3 > 0x1p-6f ? 1 : 0;
                nsmall += (s3 <= 0x1p-6f && n > 0) ? 1 : 0;
            }
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const F2 x = mul2(F2{dl[j], dl[j + 1]}, F2{1.4426950408889634f, 1.4426950408889634f});
                const F2 r = add2(F2{ex2_ftz(x.x), ex2_ftz(x.y)}, F2{-1.0f, -1.0f});
                u[j] = r.x;
                u[j + 1] = r.y;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; j += 2) {                           // |e^lt - e^lr| = e^lr |rho - 1|
            const F2 y = mul2(F2{on[j] ? lr[j] : 0.f, on[j + 1] ? lr[j + 1] : 0.f}, F2{1.4426950408889634f, 1.4426950408889634f});
            e[j] = ex2_ftz(y.x);
            e[j + 1] = ex2_ftz(y.y);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            f9 = fmaf(e[j], fabsf(u[j]), f9);
            u[j] = SEQ ? wseq - 1.0f : fminf(u[j], C - 1.0f);      // truncated weight minus one
        }
        if (!have_pivot) {
#pragma unroll
            for (int j = 7; j >= 0; --j) pivot = on[j] ? u[j] : pivot;
            A_pivot = A;
            dA = 0.f;
            have_pivot = n > 0;
        }
        F2 sv = {0.f, 0.f}, sv2 = {0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const F2 d = sub2(F2{u[j], u[j + 1]}, F2{pivot, pivot});
            const F2 v = {on[j] ? d.x : 0.f, on[j + 1] ? d.y : 0.f};
            sv = add2(sv, v);
            sv2 = fma2(v, v, sv2);
        }
        const float svs = sv.x + sv.y, sv2s = sv2.x + sv2.y, nf = static_cast<float>(n);
        const float c1 = dA * (1.0f + pivot);                      // x = A v + c1 on every valid row of the group
        g_v += svs;
        g_v2 += sv2s;
        g_dA = fmaf(dA, nf, g_dA);
        g_dA2 = fmaf(dA * dA, nf, g_dA2);
        g_x += fmaf(A, svs, c1 * nf);
        g_x2 += fmaf(A * A, sv2s, fmaf(2.0f * A * c1, svs, c1 * c1 * nf));
        nrows += n;
        return n;
    };

    // The walk over the block's tiles; the first launch also adds up the valid rows per sequence on the way.
    constexpr bool count = !EXACT;
    bool failed = false;
    {
        constexpr int base = 0;
        int issued = tile0;                             // first tile not yet requested (thread 0)
        if (tid == 0)
            for (; issued < tile1 && issued < tile0 + kMomStages; ++issued) issue(issued, (base + issued - tile0) % kMomStages);
        for (int tile = tile0; tile < tile1; ++tile) {
            const unsigned k = static_cast<unsigned>(base + tile - tile0);
            const unsigned st = k % kMomStages;
            // the group's sequence, advantage and weight source do not depend on the tile's data: fetched before the wait
            const int t0 = tile * kMomRows + 8 * tid;
            seek(t0);
            const bool single = t0 + 8 <= next_b;          // the usual case: the eight rows belong to one sequence
            if (single) enter();
            const uint32_t parity = (k / kMomStages) & 1u;
            bool ok = mbar_try_wait(&full[st], parity);
            if (!ok) ok = mbar_wait_slow(&full[st], parity, &abort_flag);
            int n = 0;
            if (ok) {
                const uint8_t* src = stages + st * kMomStageBytes;
                const float4* pa = reinterpret_cast<const float4*>(src) + 2 * tid;
                const float4* pb = reinterpret_cast<const float4*>(src + kMomRows * 4) + 2 * tid;
                const float4 a0 = pa[0], a1 = pa[1], b0 = pb[0], b1 = pb[1];
                const uint2 mk = reinterpret_cast<const uint2*>(src + kMomRows * 8)[tid];
                const float lt[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                const float lr[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                if (single) {
                    if ((mk.x | mk.y) != 0u) n = add_rows(lt, lr, mk.x, mk.y);
                } else if ((mk.x | mk.y) != 0u) {
                    const uint64_t m64 = (static_cast<uint64_t>(mk.y) << 32) | mk.x;
                    int j = 0;
                    while (j < 8) {                         // a boundary inside the group: one run of rows per sequence
                        seek(t0 + j);
                        const int left = next_b - (t0 + j);
                        const int j1 = left < 8 - j ? j + left : 8;
                        enter();
                        const uint64_t run = (j1 == 8 ? ~uint64_t(0) : (uint64_t(1) << (8 * j1)) - 1u) & ~((uint64_t(1) << (8 * j)) - 1u);
                        const int nr = add_rows(lt, lr, static_cast<uint32_t>(m64 & run), static_cast<uint32_t>((m64 & run) >> 32));
                        if (count && n_valid_seq && nr > 0) atomicAdd(&n_valid_seq[sq], nr);
                        j = j1;
                    }
                }
            }
            if (count && n_valid_seq) {
                // valid rows per sequence: a warp's 256-row strip usually lies in one sequence, whose count lane 0 keeps in
                // a register until the strip moves on (integer atomics: the result does not depend on their order)
                const int sq0 = __shfl_sync(0xffffffffu, sq, 0);
                if (__all_sync(0xffffffffu, single && sq == sq0)) {
                    const int tot = __reduce_add_sync(0xffffffffu, n);
                    if (lane == 0) {
                        if (sq0 != wsq) {
                            if (wsq >= 0 && wcnt > 0) atomicAdd(&n_valid_seq[wsq], wcnt);
                            wsq = sq0;
                            wcnt = 0;
                        }
                        wcnt += tot;
                    }
                } else if (single && n > 0) {
                    atomicAdd(&n_valid_seq[sq], n);
                }
            }
            // everyone is done with the stage (or someone gave up): the stage can take the tile three ahead
            if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
            if (tid == 0 && issued < tile1) { issue(issued, st); ++issued; }
        }
        if (failed && tid == 0) {
            // let the copies still in flight land before the block's shared memory is given up
            for (int i = 0; i < issued - tile0; ++i)
                if (issued - tile0 - i <= kMomStages) {
                    const unsigned q = static_cast<unsigned>(base + i);
                    mbar_wait_drain(&full[q % kMomStages], (q / kMomStages) & 1u);
                }
        }
    }
    if (count && n_valid_seq && lane == 0 && wsq >= 0 && wcnt > 0) atomicAdd(&n_valid_seq[wsq], wcnt);
    // rows after the last whole tile: the first threads of the grid, one row each
    for (int t = ntiles * kMomRows + static_cast<int>(blockIdx.x * blockDim.x) + tid; t < T; t += gridDim.x * blockDim.x) {
        if (!mask[t]) continue;
        sq = -1;
        seek(t);
        enter();
        const float lt[8] = {lp_train[t], 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, lr[8] = {lp_roll[t], 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        add_rows(lt, lr, 1u, 0u);
        if (count && n_valid_seq) atomicAdd(&n_valid_seq[sq], 1);
    }
    double acc[10];
    {
        // from the shifted sums to the sums of w, w^2, A, A^2, A w, (A w)^2 in fp64, once per thread:
        // w = P + v with P = 1 + pivot;  A = Ap + dA;  A w = K + x with K = Ap P
        const double P = 1.0 + static_cast<double>(pivot), Ap = static_cast<double>(A_pivot), K = Ap * P;
        const double N = static_cast<double>(nrows);
        const double SV = static_cast<double>(g_v), SDA = static_cast<double>(g_dA), SX = static_cast<double>(g_x);
        acc[0] = N;
        acc[1] = fma(P, N, SV);
        acc[2] = static_cast<double>(g_v2) + P * fma(P, N, 2.0 * SV);
        acc[3] = static_cast<double>(f3);
        acc[4] = fma(Ap, N, SDA);
        acc[5] = static_cast<double>(g_dA2) + Ap * fma(Ap, N, 2.0 * SDA);
        acc[6] = fma(K, N, SX);
        acc[7] = static_cast<double>(g_x2) + K * fma(K, N, 2.0 * SX);
        acc[8] = -(static_cast<double>(f8p.x) + static_cast<double>(f8p.y));
        acc[9] = static_cast<double>(f9);
    }
    if (failed) acc[0] = __longlong_as_double(0x7ff8000000000000LL);     // a NaN count marks the batch as not reduced
    // slots 10 and 11: what the second launch looks at (no moments; the reductions over the blocks leave them out)
    const double big = EXACT ? 0.0 : block_sum(static_cast<double>(nbig), scratch);
    const double small = EXACT ? 0.0 : block_sum(static_cast<double>(nsmall), scratch);
#pragma unroll
    for (int i = 0; i < kNumMoments; ++i) {
        const double tot = i < 10 ? block_sum(acc[i < 10 ? i : 0], scratch) : 0.0;
        if (tid == 0) partials[blockIdx.x * kNumMoments + i] = i == 10 ? big : i == 11 ? small : tot;
    }
}

__global__ void diag_finalize_kernel(const double* __restrict__ partials, int nblocks, ais_params p, ais_diag* __restrict__ diag) {
    // one warp per moment sums the partials in a fixed order;
    // thread 0 then derives the diagnostics
    __shared__ double m[kNumMoments];
    if (blockIdx.x != 0) return;
    {
        const int i = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const double acc = warp_ordered_sum(partials, nblocks, kNumMoments, i, lane);
        if (lane == 0) m[i] = acc;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    ais_diag d;
    d.status_flags = 0;
    d.reserved = 0;
    d.loss = 0.0;
    d.kl_ref = 0.0;
    const double N = m[0];
    d.n_valid = N;
    if (N <= 0.0) {
        d.mean_w = 1.0; d.cv2 = 0.0; d.ess = 0.0; d.ess_ratio = 1.0; d.alpha_ess = 1.0; d.d_bar = 0.0;
        d.alpha_mis = 0.0; d.std_A = 0.0; d.std_Aw = 0.0; d.delta_sigma = 0.0; d.alpha_var = 0.0;
        d.alpha_adaptive = 0.0; d.kl_k1 = 0.0; d.mean_abs_dp = 0.0;
        d.status_flags |= AIS_FLAG_EMPTY;
    } else {
        // Population variance E[x^2] - E[x]^2 in fp64.  The sums reach this point with fp64 accuracy relative to the
        // spread of the data (add_run), so what is left is the rounding of the fp64 additions themselves: a result
        // below 2^-44 of the mean square (a few hundred ulps of it; a standard deviation below 2.4e-7 of the rms
        // value) is that rounding and is reported as exactly zero.
        auto variance = [&](double sum, double sumsq) {
            const double mean = sum / N, ms = sumsq / N;
            const double v = ms - mean * mean;
            return v > ms * 0x1p-44 ? v : 0.0;
        };
        const double mu = m[1] / N;
        const double var = variance(m[1], m[2]);
        d.mean_w = mu;
        d.cv2 = var / (mu * mu);
        d.ess = m[1] * m[1] / m[2];
        d.ess_ratio = d.ess / N;
        d.alpha_ess = 1.0 / sqrt(1.0 + d.cv2);
        d.d_bar = m[3] / N;
        d.alpha_mis = fmin(1.0, d.d_bar / static_cast<double>(p.delta));
        d.std_A = sqrt(variance(m[4], m[5]));
        d.std_Aw = sqrt(variance(m[6], m[7]));
        d.delta_sigma = d.std_Aw / (d.std_A + static_cast<double>(p.eps));
        d.alpha_var = fmax(0.0, (d.delta_sigma - static_cast<double>(p.gamma)) / static_cast<double>(p.gamma));
        d.alpha_adaptive = fmin(1.0, fmax(0.0, d.alpha_ess - static_cast<double>(p.beta_var) * d.alpha_var)) * d.alpha_mis;
        d.kl_k1 = m[8] / N;
        d.mean_abs_dp = m[9] / N;
    }
    if (isnan(N)) d.status_flags |= AIS_FLAG_TIMEOUT;       // a block of the moments kernel gave up on a bounded wait
    d.alpha = isnan(p.alpha_override) ? d.alpha_adaptive : static_cast<double>(p.alpha_override);
    *diag = d;
}

// Sums the per-block partial moments in block order into one vector of kNumMoments doubles.
// One warp per moment, fixed order.
__global__ void moments_reduce_kernel(const double* __restrict__ partials, int nblocks, double* __restrict__ moments) {
    if (blockIdx.x != 0) return;
    const int i = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const double m = i < 10 ? warp_ordered_sum(partials, nblocks, kNumMoments, i, lane) : 0.0;   // 10, 11 are no moments
    if (lane == 0) moments[i] = m;
}

template <int VEC>
__global__ void __launch_bounds__(256) rectify_kernel(const float* __restrict__ lp_train, const float* __restrict__ lp_roll,
                                                      const uint8_t* __restrict__ mask, int64_t T, float C,
                                                      const ais_diag* __restrict__ diag, float* __restrict__ rho,
                                                      float* __restrict__ w_tilde, const int32_t* __restrict__ seq_offsets,
                                                      int S, const float* __restrict__ seq_logw) {
    const float alpha = static_cast<float>(diag->alpha);
    auto one = [&](float lt, float lr, uint8_t mk, float& r, float& wt, int64_t t) {
        r = 1.0f;
        wt = 1.0f;
        if (mk) {
            const float dl = lt - lr;
            r = __expf(dl);
            const float w = seq_logw ? __expf(seq_logw[seq_of_row(seq_offsets, S, t)]) : r;      // sequence-level variant
            wt = fmaf(alpha, fminf(w, C) - 1.0f, 1.0f);
        }
    };
    const int64_t ngroups = T / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < ngroups; g += stride) {
        const RowGroup<VEC> in = load_group<VEC>(lp_train, lp_roll, mask, g);
        float r[VEC], wt[VEC];
#pragma unroll
        for (int j = 0; j < VEC; ++j) one(in.lt[j], in.lr[j], in.mk[j], r[j], wt[j], g * VEC + j);
        if (VEC == 4) {
            if (rho) reinterpret_cast<float4*>(rho)[g] = make_float4(r[0], r[1 % VEC], r[2 % VEC], r[3 % VEC]);
            reinterpret_cast<float4*>(w_tilde)[g] = make_float4(wt[0], wt[1 % VEC], wt[2 % VEC], wt[3 % VEC]);
        } else {
            if (rho) rho[g] = r[0];
            w_tilde[g] = wt[0];
        }
    }
    for (int64_t t = ngroups * VEC + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < T; t += stride) {
        float r, wt;
        one(lp_train[t], lp_roll[t], mask[t], r, wt, t);
        if (rho) rho[t] = r;
        w_tilde[t] = wt;
    }
}

// ------------------------------------------------------------------------------------------------
// Per-token gradient factor c_t and the surrogate loss (Eq. ais-grpo without the KL term).
// ------------------------------------------------------------------------------------------------
template <int VEC>
__global__ void __launch_bounds__(kDiagThreads) loss_coef_kernel(const float* __restrict__ lp_train, const float* __restrict__ lp_old,
                                                                  const float* __restrict__ lp_ref, double beta_kl,
                                                                  const uint8_t* __restrict__ mask,
                                                                  const int32_t* __restrict__ seq_offsets,
                                                                  const float* __restrict__ adv, const float* __restrict__ w_tilde,
                                                                  const int32_t* __restrict__ n_valid_seq, int64_t T, int S,
                                                                  int S_norm, double clip_eps, double* __restrict__ partials,
                                                                  float* __restrict__ coef, const float* __restrict__ lse) {
    __shared__ double scratch[32];
    double J = 0.0, KL = 0.0;
    // one valid row of sequence sq: its share of the objective, of the KL estimate, and its gradient factor
    auto one = [&](int64_t t, int sq, float wtf) -> float {
        if (!isfinite(lse[t])) return 0.f;       // the forward pass marked this row (non-finite logits): it takes no part
        const double A = adv[sq];
        const int n = n_valid_seq[sq] > 0 ? n_valid_seq[sq] : 1;
        const double norm = 1.0 / (static_cast<double>(S_norm) * static_cast<double>(n));
        const double rho_on = lp_old ? exp(static_cast<double>(lp_train[t]) - static_cast<double>(lp_old[t])) : 1.0;
        const double un = rho_on * A;
        const double cl = fmin(fmax(rho_on, 1.0 - clip_eps), 1.0 + clip_eps) * A;
        const double wt = wtf;
        double c = 0.0;
        J += wt * fmin(un, cl) * norm;
        if (un <= cl) c = wt * A * rho_on * norm;
        if (lp_ref) {
            // KL(pi_theta || pi_ref) estimate r - log r - 1, r = pi_ref / pi_theta; its slope in lp_theta is 1 - r
            const double log_r = static_cast<double>(lp_ref[t]) - static_cast<double>(lp_train[t]);
            const double r = exp(log_r);
            KL += (r - log_r - 1.0) * norm;
            c -= beta_kl * (1.0 - r) * norm;
        }
        return static_cast<float>(c);
    };
    const int64_t ngroups = T / VEC;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < ngroups; g += stride) {
        float c[VEC], wt[VEC];
        uint8_t mk[VEC];
        bool any = false;
        if (VEC == 4) {
            const uchar4 m = reinterpret_cast<const uchar4*>(mask)[g];
            const float4 w4 = reinterpret_cast<const float4*>(w_tilde)[g];
            mk[0] = m.x; mk[1 % VEC] = m.y; mk[2 % VEC] = m.z; mk[3 % VEC] = m.w;
            wt[0] = w4.x; wt[1 % VEC] = w4.y; wt[2 % VEC] = w4.z; wt[3 % VEC] = w4.w;
        } else {
            mk[0] = mask[g];
            wt[0] = w_tilde[g];
        }
#pragma unroll
        for (int j = 0; j < VEC; ++j) { c[j] = 0.f; any |= (mk[j] != 0); }
        if (any) {
            const int64_t t0 = g * VEC;
            int sq = seq_of_row(seq_offsets, S, t0);
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                while (sq + 1 < S && static_cast<int64_t>(seq_offsets[sq + 1]) <= t0 + j) ++sq;
                if (mk[j]) c[j] = one(t0 + j, sq, wt[j]);
            }
        }
        if (VEC == 4) reinterpret_cast<float4*>(coef)[g] = make_float4(c[0], c[1 % VEC], c[2 % VEC], c[3 % VEC]);
        else coef[g] = c[0];
    }
    for (int64_t t = ngroups * VEC + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < T; t += stride)
        coef[t] = mask[t] ? one(t, seq_of_row(seq_offsets, S, t), w_tilde[t]) : 0.f;
    const double tot = block_sum(J, scratch);
    const double tot_kl = block_sum(KL, scratch);
    if (threadIdx.x == 0) {
        partials[2 * blockIdx.x] = tot;
        partials[2 * blockIdx.x + 1] = tot_kl;
    }
}

__global__ void loss_finalize_kernel(const double* __restrict__ partials, int nblocks, double beta_kl, float* loss,
                                     ais_diag* diag) {
    // one warp, fixed order
    if (threadIdx.x >= 32 || blockIdx.x != 0) return;
    const double J = warp_ordered_sum(partials, nblocks, 2, 0, threadIdx.x);
    const double KL = warp_ordered_sum(partials, nblocks, 2, 1, threadIdx.x);
    if (threadIdx.x != 0) return;
    const double total = -J + beta_kl * KL;
    if (loss) *loss = static_cast<float>(total);
    if (diag) {
        diag->loss = total;
        diag->kl_ref = KL;
    }
}

// 16-byte loads need every per-row vector on a 16-byte boundary (the mask on a 4-byte one).
inline bool vec4_ok(const void* a, const void* b, const void* c, const void* d, const void* m) {
    const uintptr_t f = reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c) |
                        reinterpret_cast<uintptr_t>(d);
    return (f % 16 == 0) && (reinterpret_cast<uintptr_t>(m) % 4 == 0);
}

void launch_moments_kernel(const float* lp_train, const float* lp_roll, const uint8_t* mask, const int32_t* seq_offsets,
                           const float* adv, int64_t T, int S, float C, double* partials, int32_t* n_valid_seq,
                           float* seq_logw, cudaStream_t stream) {
    if (seq_logw && S > 0) seq_logw_kernel<<<(S + 7) / 8, 256, 0, stream>>>(lp_train, lp_roll, mask, seq_offsets, S, seq_logw);
    if (vec4_ok(lp_train, lp_roll, nullptr, nullptr, mask) && reinterpret_cast<uintptr_t>(mask) % 16 == 0 && T < (int64_t(1) << 31) - 2 * kMomRows) {      // 32-bit row indices inside
        // the fast form, then the exact form for the blocks whose gaps were all tiny (usually none: those blocks return at once)
        const int Ti = static_cast<int>(T);
        if (seq_logw) {
            moments_staged_kernel<true, false><<<kDiagBlocks, kDiagThreads, kMomSmemBytes, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, Ti, S, C, partials, n_valid_seq, seq_logw);
            moments_staged_kernel<true, true><<<kDiagBlocks, kDiagThreads, kMomSmemBytes, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, Ti, S, C, partials, n_valid_seq, seq_logw);
        } else {
            moments_staged_kernel<false, false><<<kDiagBlocks, kDiagThreads, kMomSmemBytes, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, Ti, S, C, partials, n_valid_seq, seq_logw);
            moments_staged_kernel<false, true><<<kDiagBlocks, kDiagThreads, kMomSmemBytes, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, Ti, S, C, partials, n_valid_seq, seq_logw);
        }
    } else if (vec4_ok(lp_train, lp_roll, nullptr, nullptr, mask))
        moments_kernel<4><<<kDiagBlocks, kDiagThreads, 0, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, T, S, C, partials,
                                                                      n_valid_seq, seq_logw);
    else
        moments_kernel<1><<<kDiagBlocks, kDiagThreads, 0, stream>>>(lp_train, lp_roll, mask, seq_offsets, adv, T, S, C, partials,
                                                                      n_valid_seq, seq_logw);
}

void launch_rectify_kernel(const float* lp_train, const float* lp_roll, const uint8_t* mask, int64_t T, float C,
                           const ais_diag* diag, float* rho, float* w_tilde, const int32_t* seq_offsets, int S,
                           const float* seq_logw, cudaStream_t stream) {
    const int64_t groups = (T + 3) / 4;
    const int blocks = static_cast<int>(((groups + 255) / 256) < 2368 ? ((groups + 255) / 256) : 2368);
    if (vec4_ok(lp_train, lp_roll, rho, w_tilde, mask))
        rectify_kernel<4><<<blocks, 256, 0, stream>>>(lp_train, lp_roll, mask, T, C, diag, rho, w_tilde, seq_offsets, S, seq_logw);
    else
        rectify_kernel<1><<<blocks, 256, 0, stream>>>(lp_train, lp_roll, mask, T, C, diag, rho, w_tilde, seq_offsets, S, seq_logw);
}

}  // namespace

cudaError_t stream_prepare() {
    cudaError_t e = cudaFuncSetAttribute(moments_staged_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMomSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(moments_staged_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMomSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(moments_staged_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMomSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(moments_staged_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMomSmemBytes);
}

// ------------------------------------------------------------------------------------------------ launchers
cudaError_t launch_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int block, uint8_t* codes,
                            int64_t ldq, float* scales, int64_t lds, cudaStream_t stream) {
    if (rows == 0 || cols == 0) return cudaSuccess;
    dim3 grid(static_cast<unsigned>((cols + kQCols - 1) / kQCols), static_cast<unsigned>((rows + kQRows - 1) / kQRows));
    const __nv_bfloat16* xp = static_cast<const __nv_bfloat16*>(x);
    switch (block) {
        case 32:  quantize_kernel<32><<<grid, kQThreads, 0, stream>>>(xp, rows, cols, ld, codes, ldq, scales, lds); break;
        case 64:  quantize_kernel<64><<<grid, kQThreads, 0, stream>>>(xp, rows, cols, ld, codes, ldq, scales, lds); break;
        case 128: quantize_kernel<128><<<grid, kQThreads, 0, stream>>>(xp, rows, cols, ld, codes, ldq, scales, lds); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_cols(const void* x, int64_t K, int64_t N, int64_t ld, int block, uint8_t* codes, int64_t ldq,
                                 float* scales, int64_t lds, cudaStream_t stream) {
    if (K == 0 || N == 0) return cudaSuccess;
    dim3 grid(static_cast<unsigned>((N + kQcTile - 1) / kQcTile), static_cast<unsigned>((K + kQcTile - 1) / kQcTile));
    const __nv_bfloat16* xp = static_cast<const __nv_bfloat16*>(x);
    switch (block) {
        case 32:  quantize_cols_kernel<32><<<grid, 256, 0, stream>>>(xp, K, N, ld, codes, ldq, scales, lds); break;
        case 64:  quantize_cols_kernel<64><<<grid, 256, 0, stream>>>(xp, K, N, ld, codes, ldq, scales, lds); break;
        case 128: quantize_cols_kernel<128><<<grid, 256, 0, stream>>>(xp, K, N, ld, codes, ldq, scales, lds); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_mx(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq,
                               uint8_t* scales, size_t scale_bytes, bool fp4, cudaStream_t stream) {
    // rows that pad the last chunks carry the neutral scale
    cudaError_t e = cudaMemsetAsync(scales, 127, scale_bytes, stream);
    if (e != cudaSuccess) return e;
    if (rows == 0 || cols == 0) return cudaSuccess;
    dim3 grid(static_cast<unsigned>((cols + kQCols - 1) / kQCols), static_cast<unsigned>((rows + kQRows - 1) / kQRows));
    if (fp4)
        quantize_mxfp4_kernel<<<grid, kQThreads, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), rows, cols, ld, codes, ldq, scales);
    else
        quantize_mx_kernel<<<grid, kQThreads, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), rows, cols, ld, codes, ldq, scales);
    return cudaGetLastError();
}

cudaError_t launch_quantize_tensor(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq,
                                   float* scale, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(scale, 0, sizeof(float), stream);
    if (e != cudaSuccess) return e;
    const __nv_bfloat16* xp = static_cast<const __nv_bfloat16*>(x);
    const int64_t total = rows * (cols / 8);
    const int blocks = static_cast<int>(total <= 0 ? 1 : ((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16));
    if (total > 0) tensor_amax_kernel<<<blocks, 256, 0, stream>>>(xp, rows, cols, ld, reinterpret_cast<uint32_t*>(scale));
    tensor_scale_kernel<<<1, 1, 0, stream>>>(reinterpret_cast<uint32_t*>(scale));
    if (total > 0) tensor_quantize_kernel<<<blocks, 256, 0, stream>>>(xp, rows, cols, ld, codes, ldq, scale);
    return cudaGetLastError();
}

cudaError_t launch_combine(const float* part_m, const float* part_s, const float* part_z, int nparts, int64_t part_ld,
                           const uint8_t* mask, int64_t T, float* lp, float* lse, uint32_t* status, cudaStream_t stream) {
    if (T == 0) return cudaSuccess;
    const int blocks = static_cast<int>(((T + 255) / 256) < 1184 ? ((T + 255) / 256) : 1184);
    combine_kernel<<<blocks, 256, 0, stream>>>(part_m, part_s, part_z, nparts, part_ld, mask, T, lp, lse, status);
    return cudaGetLastError();
}

cudaError_t launch_tile_flags_mask(const uint8_t* mask, int64_t T, uint8_t* flags, cudaStream_t stream) {
    if (T <= 0) return cudaSuccess;
    tile_flags_kernel<uint8_t><<<static_cast<unsigned>((T + 127) / 128), 128, 0, stream>>>(mask, T, flags);
    return cudaGetLastError();
}

cudaError_t launch_tile_flags_coef(const float* coef, int64_t T, uint8_t* flags, cudaStream_t stream) {
    if (T <= 0) return cudaSuccess;
    tile_flags_kernel<float><<<static_cast<unsigned>((T + 127) / 128), 128, 0, stream>>>(coef, T, flags);
    return cudaGetLastError();
}

cudaError_t launch_seq_counts(const uint8_t* mask, const int32_t* seq_offsets, int S, int32_t* n_valid_seq, cudaStream_t stream) {
    if (S == 0) return cudaSuccess;
    seq_count_kernel<<<(S + 7) / 8, 256, 0, stream>>>(mask, seq_offsets, S, n_valid_seq);
    return cudaGetLastError();
}

cudaError_t launch_advantages(const float* rewards, int S, int G, int adv_std_norm, float eps, float* adv, int32_t* zero_counts,
                              cudaStream_t stream) {
    if (S == 0) return cudaSuccess;
    adv_kernel<<<(S + 255) / 256, 256, 0, stream>>>(rewards, S, G, adv_std_norm, eps, adv, zero_counts);
    return cudaGetLastError();
}

cudaError_t launch_diag(const float* lp_train, const float* lp_roll, const uint8_t* mask, const int32_t* seq_offsets,
                        const float* adv, int64_t T, int S, const ais_params& p, double* partials, int32_t* n_valid_seq,
                        float* seq_logw, float* rho, float* w_tilde, ais_diag* diag, cudaStream_t stream) {
    const float C = p.C;
    launch_moments_kernel(lp_train, lp_roll, mask, seq_offsets, adv, T, S, C, partials, n_valid_seq, seq_logw, stream);
    diag_finalize_kernel<<<1, 32 * kNumMoments, 0, stream>>>(partials, kDiagBlocks, p, diag);
    if (T > 0) launch_rectify_kernel(lp_train, lp_roll, mask, T, C, diag, rho, w_tilde, seq_offsets, S, seq_logw, stream);
    return cudaGetLastError();
}

cudaError_t launch_moments(const float* lp_train, const float* lp_roll, const uint8_t* mask, const int32_t* seq_offsets,
                           const float* adv, int64_t T, int S, const ais_params& p, double* partials, int32_t* n_valid_seq,
                           float* seq_logw, double* moments, cudaStream_t stream) {
    launch_moments_kernel(lp_train, lp_roll, mask, seq_offsets, adv, T, S, p.C, partials, n_valid_seq, seq_logw, stream);
    moments_reduce_kernel<<<1, 32 * kNumMoments, 0, stream>>>(partials, kDiagBlocks, moments);
    return cudaGetLastError();
}

cudaError_t launch_finalize(const double* moments, const float* lp_train, const float* lp_roll, const uint8_t* mask, int64_t T,
                            const ais_params& p, float* rho, float* w_tilde, ais_diag* diag, const int32_t* seq_offsets, int S,
                            const float* seq_logw, cudaStream_t stream) {
    diag_finalize_kernel<<<1, 32 * kNumMoments, 0, stream>>>(moments, 1, p, diag);
    if (T > 0) launch_rectify_kernel(lp_train, lp_roll, mask, T, p.C, diag, rho, w_tilde, seq_offsets, S, seq_logw, stream);
    return cudaGetLastError();
}

cudaError_t launch_loss_coef(const float* lp_train, const float* lp_old, const float* lp_ref, float beta_kl, const uint8_t* mask,
                             const int32_t* seq_offsets,
                             const float* adv, const float* w_tilde, const int32_t* n_valid_seq, int64_t T, int S, int S_norm,
                             float clip_eps, double* partials, float* coef, float* loss, ais_diag* diag, const float* lse,
                             cudaStream_t stream) {
    const float* ref = (beta_kl != 0.f) ? lp_ref : nullptr;
    if (vec4_ok(w_tilde, coef, nullptr, nullptr, mask))
        loss_coef_kernel<4><<<kDiagBlocks, kDiagThreads, 0, stream>>>(lp_train, lp_old, ref, static_cast<double>(beta_kl), mask,
                                                                        seq_offsets, adv, w_tilde, n_valid_seq, T, S, S_norm,
                                                                        static_cast<double>(clip_eps), partials, coef, lse);
    else
        loss_coef_kernel<1><<<kDiagBlocks, kDiagThreads, 0, stream>>>(lp_train, lp_old, ref, static_cast<double>(beta_kl), mask,
                                                                        seq_offsets, adv, w_tilde, n_valid_seq, T, S, S_norm,
                                                                        static_cast<double>(clip_eps), partials, coef, lse);
    loss_finalize_kernel<<<1, 32, 0, stream>>>(partials, kDiagBlocks, ref ? static_cast<double>(beta_kl) : 0.0, loss, diag);
    return cudaGetLastError();
}

}  // namespace ais

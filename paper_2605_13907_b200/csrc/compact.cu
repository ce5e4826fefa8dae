// Row compaction for scattered validity masks (masked-diffusion batches): the valid rows of every sequence are
// packed, in order, into a dense batch; the tensor-core passes then only see rows that matter, and the results
// are scattered back.  Declarations and contracts live in include/ais.h.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ais.h"

namespace {

constexpr int kThreads = 256;

// Exclusive scan of the per-sequence valid counts -> packed row offsets (one block; S is small).
__global__ void scan_counts_kernel(const int32_t* __restrict__ n_valid_seq, int S, int32_t* __restrict__ packed_offsets) {
    __shared__ int64_t carry;
    __shared__ int32_t buf[kThreads];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < S; base += kThreads) {
        const int s = base + threadIdx.x;
        const int32_t v = s < S ? n_valid_seq[s] : 0;
        buf[threadIdx.x] = v;
        __syncthreads();
        for (int off = 1; off < kThreads; off <<= 1) {           // Hillis-Steele inclusive scan of the chunk
            const int32_t add = threadIdx.x >= off ? buf[threadIdx.x - off] : 0;
            __syncthreads();
            buf[threadIdx.x] += add;
            __syncthreads();
        }
        if (s < S) packed_offsets[s] = static_cast<int32_t>(carry + buf[threadIdx.x] - v);
        __syncthreads();
        if (threadIdx.x == kThreads - 1) carry += buf[threadIdx.x];
        __syncthreads();
    }
    if (threadIdx.x == 0) packed_offsets[S] = static_cast<int32_t>(carry);
}

__global__ void count_valid_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ seq_offsets,
                                   int32_t* __restrict__ n_valid_seq) {
    __shared__ int32_t part[kThreads / 32];
    const int s = blockIdx.x;
    const int b = seq_offsets[s], e = seq_offsets[s + 1];
    int32_t cnt = 0;
    for (int t = b + threadIdx.x; t < e; t += blockDim.x) cnt += mask[t] ? 1 : 0;
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t tot = 0;
        for (int i = 0; i < kThreads / 32; ++i) tot += part[i];
        n_valid_seq[s] = tot;
    }
}

// One block per sequence: ordered list of its valid rows, written at the sequence's packed offset.
__global__ void row_index_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ seq_offsets,
                                 const int32_t* __restrict__ packed_offsets, int32_t* __restrict__ row_index) {
    __shared__ int32_t warp_tot[kThreads / 32];
    __shared__ int32_t base;
    const int s = blockIdx.x;
    const int b = seq_offsets[s], e = seq_offsets[s + 1];
    if (threadIdx.x == 0) base = packed_offsets[s];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int t0 = b; t0 < e; t0 += kThreads) {
        const int t = t0 + threadIdx.x;
        const bool v = t < e && mask[t] != 0;
        const uint32_t ballot = __ballot_sync(0xffffffffu, v);
        const int in_warp = __popc(ballot & ((1u << lane) - 1u));
        if (lane == 0) warp_tot[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            if (w < warp) before += warp_tot[w];
            total += warp_tot[w];
        }
        if (v) row_index[base + before + in_warp] = t;
        __syncthreads();
        if (threadIdx.x == 0) base += total;
        __syncthreads();
    }
}

// dst[i, :] = src[row_index[i], :] for rows of `row_bytes` bytes (a multiple of 16).
__global__ void gather_rows_kernel(const uint8_t* __restrict__ src, int64_t src_stride, const int32_t* __restrict__ row_index,
                                   int64_t n, int64_t vec_per_row, uint8_t* __restrict__ dst, int64_t dst_stride) {
    const int64_t total = n * vec_per_row;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / vec_per_row, c = i % vec_per_row;
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + static_cast<int64_t>(row_index[r]) * src_stride) + c);
        reinterpret_cast<uint4*>(dst + r * dst_stride)[c] = v;
    }
}

// dst[row_index[i], :] = src[i, :]
__global__ void scatter_rows_kernel(const uint8_t* __restrict__ src, int64_t src_stride, const int32_t* __restrict__ row_index,
                                    int64_t n, int64_t vec_per_row, uint8_t* __restrict__ dst, int64_t dst_stride) {
    const int64_t total = n * vec_per_row;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / vec_per_row, c = i % vec_per_row;
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + r * src_stride) + c);
        reinterpret_cast<uint4*>(dst + static_cast<int64_t>(row_index[r]) * dst_stride)[c] = v;
    }
}

__global__ void gather_words_kernel(const uint32_t* __restrict__ src, const int32_t* __restrict__ row_index, int64_t n,
                                    uint32_t* __restrict__ dst) {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        dst[i] = src[row_index[i]];
}

// dst[row_index[i]] = src[i] for 32-bit elements (the destination is filled with its neutral value first)
__global__ void scatter_words_kernel(const uint32_t* __restrict__ src, const int32_t* __restrict__ row_index, int64_t n,
                                     uint32_t* __restrict__ dst) {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        dst[row_index[i]] = src[i];
}

__global__ void fill_words_kernel(uint32_t* __restrict__ dst, int64_t n, uint32_t value) {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        dst[i] = value;
}

inline int grid_for(int64_t work) {
    const int64_t b = (work + kThreads - 1) / kThreads;
    return static_cast<int>(b < 1 ? 1 : (b > 148 * 16 ? 148 * 16 : b));
}
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" {

int ais_compact_index(const uint8_t* mask, const int32_t* seq_offsets, int32_t S, int32_t* n_valid_seq,
                      int32_t* packed_offsets, int32_t* row_index, void* stream) {
    if (!mask || !seq_offsets || !n_valid_seq || !packed_offsets || !row_index) return AIS_ERR_NULL;
    if (S <= 0) return AIS_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    count_valid_kernel<<<S, kThreads, 0, s>>>(mask, seq_offsets, n_valid_seq);
    scan_counts_kernel<<<1, kThreads, 0, s>>>(n_valid_seq, S, packed_offsets);
    row_index_kernel<<<S, kThreads, 0, s>>>(mask, seq_offsets, packed_offsets, row_index);
    return cudaGetLastError() == cudaSuccess ? AIS_OK : AIS_ERR_DEVICE;
}

int ais_gather_rows(const void* src, int64_t src_stride_bytes, const int32_t* row_index, int64_t n, int64_t row_bytes,
                    void* dst, int64_t dst_stride_bytes, void* stream) {
    if (!src || !row_index || !dst) return AIS_ERR_NULL;
    if (n < 0 || row_bytes <= 0 || src_stride_bytes < row_bytes || dst_stride_bytes < row_bytes) return AIS_ERR_SHAPE;
    if (row_bytes % 16 != 0 || src_stride_bytes % 16 != 0 || dst_stride_bytes % 16 != 0 || !aligned(src, 16) || !aligned(dst, 16))
        return AIS_ERR_ALIGN;
    if (n == 0) return AIS_OK;
    gather_rows_kernel<<<grid_for(n * (row_bytes / 16)), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(src), src_stride_bytes, row_index, n, row_bytes / 16, static_cast<uint8_t*>(dst), dst_stride_bytes);
    return cudaGetLastError() == cudaSuccess ? AIS_OK : AIS_ERR_DEVICE;
}

int ais_scatter_rows(const void* src, int64_t src_stride_bytes, const int32_t* row_index, int64_t n, int64_t row_bytes,
                     void* dst, int64_t dst_stride_bytes, int64_t dst_rows, void* stream) {
    if (!src || !row_index || !dst) return AIS_ERR_NULL;
    if (n < 0 || dst_rows < n || row_bytes <= 0 || src_stride_bytes < row_bytes || dst_stride_bytes < row_bytes) return AIS_ERR_SHAPE;
    if (row_bytes % 16 != 0 || src_stride_bytes % 16 != 0 || dst_stride_bytes % 16 != 0 || !aligned(src, 16) || !aligned(dst, 16))
        return AIS_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // only the row_bytes of every row: the padding between rows (and whatever follows the last row) is the caller's
    if (dst_rows > 0 && cudaMemset2DAsync(dst, static_cast<size_t>(dst_stride_bytes), 0, static_cast<size_t>(row_bytes),
                                          static_cast<size_t>(dst_rows), s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (n == 0) return AIS_OK;
    scatter_rows_kernel<<<grid_for(n * (row_bytes / 16)), kThreads, 0, s>>>(static_cast<const uint8_t*>(src), src_stride_bytes, row_index,
                                                                             n, row_bytes / 16, static_cast<uint8_t*>(dst),
                                                                             dst_stride_bytes);
    return cudaGetLastError() == cudaSuccess ? AIS_OK : AIS_ERR_DEVICE;
}

int ais_gather_words(const void* src, const int32_t* row_index, int64_t n, void* dst, void* stream) {
    if (!src || !row_index || !dst) return AIS_ERR_NULL;
    if (n < 0) return AIS_ERR_SHAPE;
    if (n == 0) return AIS_OK;
    gather_words_kernel<<<grid_for(n), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint32_t*>(src), row_index, n,
                                                                                          static_cast<uint32_t*>(dst));
    return cudaGetLastError() == cudaSuccess ? AIS_OK : AIS_ERR_DEVICE;
}

int ais_scatter_words(const void* src, const int32_t* row_index, int64_t n, void* dst, int64_t dst_rows, uint32_t fill_bits,
                      void* stream) {
    if (!src || !row_index || !dst) return AIS_ERR_NULL;
    if (n < 0 || dst_rows < n) return AIS_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (dst_rows > 0) fill_words_kernel<<<grid_for(dst_rows), kThreads, 0, s>>>(static_cast<uint32_t*>(dst), dst_rows, fill_bits);
    if (n > 0) scatter_words_kernel<<<grid_for(n), kThreads, 0, s>>>(static_cast<const uint32_t*>(src), row_index, n, static_cast<uint32_t*>(dst));
    return cudaGetLastError() == cudaSuccess ? AIS_OK : AIS_ERR_DEVICE;
}

}  // extern "C"

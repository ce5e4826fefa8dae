// Arguments shared by the host launcher and the LM-head tensor-core kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace ais {

enum LmheadMode : int {
    kFwdBf16 = 0,   // z = H W^T (bf16), streaming log-sum-exp + target pick -> partial triples
    kFwdFp8  = 1,   // z^ from E4M3 codes with per-block scale promotion, same epilogue
    kBwdP    = 2,   // recompute z (bf16), write u = softmax - onehot as bf16 scratch
    kBwdDh   = 3,   // dH = c (.) (U W), contraction over the vocabulary
    kFwdFp8T = 4,   // E4M3 codes with one scale per tensor: whole contraction in tensor memory, one multiply after
    kBwdDw   = 5,   // dW += U^T H, contraction over the rows (both operands read with the contraction axis as rows)
    kFwdMx   = 6,   // E4M3 codes with one power-of-two (E8M0) scale per 32 elements: hardware block-scaled MMA
    kFwdMx4  = 7,   // packed E2M1 (FP4) codes with one E8M0 scale per 32 elements
    // the same three bf16 passes with W stored [d, V] (one row per hidden unit): the forward passes then read W as an
    // MN-major B operand (four 64-column boxes per stage, like the dH pass of the other layout) and the dH pass reads it
    // K-major (like the forward passes of the other layout)
    kFwdBf16Dv = 8,
    kBwdPDv    = 9,
    kBwdDhDv   = 10
};

// What a mode computes (its epilogue and work-unit shape), whatever the layout of W.
__host__ __device__ constexpr int base_mode(int mode) {
    return mode == kFwdBf16Dv ? kFwdBf16 : mode == kBwdPDv ? kBwdP : mode == kBwdDhDv ? kBwdDh : mode;
}
// B operand stored with the output column as the contiguous axis (MN-major)?
__host__ __device__ constexpr bool b_mn_major(int mode) {
    return mode == kBwdDh || mode == kBwdDw || mode == kFwdBf16Dv || mode == kBwdPDv;
}

constexpr int kBM = 128;                 // rows per tile (TMEM lanes)
constexpr int kBN = 256;                 // columns per tile (TMEM columns of one accumulator)
constexpr int kStageKBytes = 128;        // bytes of K per shared-memory stage row (one swizzle span)
constexpr int kAStageBytes = kBM * kStageKBytes;
constexpr int kBStageBytes = kBN * kStageKBytes;
constexpr int kStageBytes = kAStageBytes + kBStageBytes;
constexpr int kStages = 4;
// dH pass: a CTA owns two row tiles (256 rows) so that every W tile it loads feeds two accumulators
constexpr int kDhRows = 2 * kBM;
constexpr int kDhStageBytes = 2 * kAStageBytes + kBStageBytes;
constexpr int kDhStages = 3;
static_assert(kDhStages * kDhStageBytes <= kStages * kStageBytes, "the dH stage ring must fit the same shared memory");
constexpr int kNumBarriers = 3 * kStages + 4 + 1;
// microscaling passes: per 128-byte K stage one 512-byte scale chunk for the 128 rows of A and two for the 256 rows of B
// (FP8: 128 elements per stage), twice that with FP4 operands (256 elements per stage)
constexpr int kMxChunkBytes = 512;
constexpr int kMxStageScaleBytes = 6 * kMxChunkBytes;
constexpr int kThreads = 384;            // warp 0 TMA, warp 1 MMA, warps 2..3 idle, warps 4..11 epilogue
constexpr int kEpiWarps = 8;
constexpr int kMxThreads = 512;          // microscaling passes: warps 12..15 move the block scales into tensor memory
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kStages * kMxStageScaleBytes + kNumBarriers * 8 + 64;

// Pacing of the CTAs of a launch (lmhead_common.cuh): stage fills per announcement, counters in the ring.
constexpr int kPaceFills = 16;
constexpr int kPaceSettle = 4;     // stage fills between an announcement and the look at the counter it waits for
constexpr int kPaceRing = 4096;

struct LmheadArgs {
    int64_t rows;          // valid rows handled by this launch
    int64_t row0;          // global index of local row 0 (per-row vectors are indexed globally)
    int32_t n_row_tiles;   // row tiles of 128 rows (dH pass: of 256 rows)
    int32_t ncols;         // output columns: V (forward, recompute) or d (dH)
    int32_t n_col_tiles;
    int32_t ksteps;        // shared-memory stages per accumulator tile
    int32_t nsplit;        // forward / recompute: independent column ranges per row tile
    int32_t sgroups;       // FP8: scale blocks per stage (128 / fp8_block)
    const uint8_t* tile_active;   // one byte per global 128-row tile: 0 = nothing to compute there (may be NULL)
    const int32_t* tokens;
    const uint8_t* mask;
    float* part_m;         // [nsplit*2][part_ld] running maxima (natural log units)
    float* part_s;         // sums of exp(z - m)
    float* part_z;         // target logit or -inf
    int64_t part_ld;
    const float* lse;      // recompute: log-sum-exp of the trainer pass
    __nv_bfloat16* U;      // recompute output / dH input scratch [rows_pad, ldU]
    int64_t ldU;
    const float* scale_a;  // per-tensor FP8: the two scales (one float each, on the device)
    const float* scale_b;
    const float* coef;     // recompute: per-row factor c_t folded into the scratch
    const uint8_t* sf_a;   // microscaling: packed scale chunks of A [row chunks of 128][d/128][512 bytes]
    const uint8_t* sf_b;   // and of B
    int32_t nk4;           // d / 128: scale chunks per 128 rows
    float* dW;             // dW pass: [V, lddw] fp32
    int64_t lddw;
    int32_t dw_accumulate; // dW pass: add to what dW holds instead of overwriting it
    __nv_bfloat16* dH;
    int64_t lddh;
    uint32_t* status;
    int64_t wait_cycles;   // bound of every device-side wait in clock ticks; 0 = the default (about two seconds)
    uint32_t* pace;        // ring of kPaceRing zeroed counters that keeps the CTAs of the launch in step; NULL = no pacing
    int32_t pace_per_unit; // announcements per unit = ceil(largest number of stage fills of a unit / fills per announcement)
};

// Launches one pass.  tmSA / tmSB are only read in kFwdFp8 mode.
cudaError_t launch_lmhead(int mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                          const CUtensorMap& tmSB, const LmheadArgs& args, int num_ctas, cudaStream_t stream);
cudaError_t lmhead_prepare();   // sets the dynamic shared-memory attribute of every instantiation

// The rollout pass with per-block scales (mode kFwdFp8; args.sgroups = 128 / block = 1, 2 or 4).  tmSA / tmSB map the
// block-major scale arrays with boxes of (128 rows, sgroups) and (256 rows, sgroups).
cudaError_t launch_lmhead_fp8_block(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                                    const CUtensorMap& tmSB, const LmheadArgs& args, int num_ctas, cudaStream_t stream);
cudaError_t lmhead_fp8_block_prepare();

}  // namespace ais

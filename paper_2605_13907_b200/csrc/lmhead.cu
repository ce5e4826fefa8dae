// LM-head tensor-core passes for sm_100a: TMA-fed tcgen05.mma with accumulators in tensor memory and
// fused epilogues (streaming log-sum-exp + target pick, softmax-minus-onehot scratch, dH scaling).
//
// One persistent CTA of three warpgroups per SM.  Warp 0 issues TMA tile loads, warp 1 issues the MMAs
// (warps 2, 3 idle), warps 4..11 are the epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 (one row per
// thread) and column half (w-4)/4 of the 256-column accumulator.  The dH pass gives a CTA two row tiles
// (256 rows, both accumulators) so that every W slice it loads is used twice; its contraction over the
// vocabulary is so long that the one epilogue per unit need not overlap anything.  Two 256-column accumulators
// alternate so that the epilogue of one tile overlaps the MMAs of the next.  The microscaling modes add a fourth
// warpgroup (warps 12..15) that moves each stage's block scales from shared to tensor memory, where the
// block-scaled MMA reads them; their scale columns leave room for one accumulator only.  The rollout pass with
// fp32 per-block scales has a kernel of its own (lmhead_fp8.cu).
#include <type_traits>

#include "lmhead_common.cuh"
#include "../../include/ais.h"

namespace ais {

namespace {

constexpr int threads_of(int mode) { return (mode == kFwdMx || mode == kFwdMx4) ? kMxThreads : kThreads; }

template <int MODE>
__global__ void __launch_bounds__(threads_of(MODE), 1)
lmhead_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const LmheadArgs a) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned start, as an offset from the array so that the compiler still knows the address space
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* stage_base = smem;
    uint8_t* mx_scale_base = smem + kStages * kStageBytes;      // microscaling pass: one scale triple per stage
    uint64_t* bars = reinterpret_cast<uint64_t*>(mx_scale_base + kStages * kMxStageScaleBytes);
    uint64_t* full = bars;                       // [kStages]   TMA -> MMA
    uint64_t* empty = full + kStages;            // [kStages]   MMA -> TMA
    uint64_t* tfull = empty + kStages;           // [2]         MMA -> epilogue
    uint64_t* tempty = tfull + 2;                // [2]         epilogue -> MMA
    uint64_t* done = tempty + 2;                 // [1]         all MMAs of this CTA have completed
    uint64_t* sfull = done + 1;                  // [kStages]   scale warps -> MMA (microscaling passes)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBarriers);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* issued_slot = tmem_slot + 2;     // stage fills the producer has requested (written when it leaves its loop)

    constexpr int BASE = base_mode(MODE);                                       // what is computed, whatever W's layout
    constexpr bool B_MN = b_mn_major(MODE);                                     // B tile arrives as four 64-column boxes
    constexpr bool TWO_ACC = (BASE == kBwdDh || BASE == kBwdDw);                // two 128-row tiles per CTA, one B slice
    constexpr int STG = TWO_ACC ? kDhStages : kStages;                          // depth of the stage ring
    constexpr int STG_BYTES = TWO_ACC ? kDhStageBytes : kStageBytes;
    constexpr int A_BYTES = TWO_ACC ? 2 * kAStageBytes : kAStageBytes;
    constexpr bool MX = (MODE == kFwdMx || MODE == kFwdMx4);                    // block scales live in tensor memory
    constexpr bool FP4 = (MODE == kFwdMx4);                                     // 256 packed 4-bit elements per stage
    constexpr int MX_SCALE_BYTES = FP4 ? 6 * kMxChunkBytes : 3 * kMxChunkBytes;
    constexpr int NBUF = (TWO_ACC || MX) ? 1 : 2;                               // accumulator sets that alternate
    constexpr uint32_t kMxScaleCol = 256;                                       // MX: scale columns after the accumulator,
    constexpr uint32_t kMxSetCols = 32;                                         // one set of 32 per stage of the ring
    constexpr int kScaleWarp0 = 12;                                             // MX: first of the four scale warps
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_units = TWO_ACC ? a.n_row_tiles * a.n_col_tiles : a.n_row_tiles * a.nsplit;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); mbar_init(&sfull[i], 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpiWarps); }
        mbar_init(done, 1);
        *abort_flag = 0;
        *issued_slot = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Microscaling pass: its one accumulator is read into registers in one go so that it can go back to the MMA
    // issuer at once; the other warps hand the registers for that to the epilogue (512 x 128 = 256 x 32 + 256 x 224).
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (MX) reg_dealloc<32>();
        if (lane == 0) {
            Pipe st(STG);
            uint32_t issued = 0;
            bool ok = true;
            Pacer pacer(a.pace, a.pace_per_unit);
            int n = 0;                                          // ordinal of this CTA's unit (its wave)
            for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x, ++n) {
                const Unit w = decode_unit<BASE>(a, u);
                if (!unit_active<BASE>(a, w)) {
                    if (pacer.ring) pacer.top_up(n, 0);
                    continue;
                }
                int fills = 0;                                  // stage fills of this unit so far
                for (int t = w.t0; t < w.t1 && ok; ++t) {
                    for (int ks = 0; ks < a.ksteps; ++ks, ++fills) {
                        if (pacer.ring && fills % kPaceFills == 0) pacer.announce(n, fills / kPaceFills);
                        if (pacer.ring && fills % kPaceFills == kPaceSettle) pacer.settle();
                        if (!mbar_wait(&empty[st.idx], st.phase ^ 1u, abort_flag, a.wait_cycles)) { ok = false; break; }
                        uint8_t* sA = stage_base + st.idx * STG_BYTES;
                        uint8_t* sB = sA + A_BYTES;
                        mbar_expect_tx(&full[st.idx], MX ? STG_BYTES + MX_SCALE_BYTES : STG_BYTES);
                        const int kelem = (MODE == kFwdFp8T || MX) ? ks * 128 : ks * 64;
                        if (MX) {
                            // the stage's scales (see the layout at ais_quantize_mxfp8): A's chunk(s) of this row tile, then the
                            // adjacent chunk pair(s) of B's 256 rows; with FP4 a stage spans two chunk columns
                            uint8_t* sS = mx_scale_base + st.idx * kMxStageScaleBytes;
                            constexpr int KC = FP4 ? 2 : 1;                    // chunk columns per stage
                            const int64_t k4 = static_cast<int64_t>(ks) * KC;
#pragma unroll
                            for (int c = 0; c < KC; ++c)
                                bulk_load(sS + c * kMxChunkBytes,
                                          a.sf_a + (static_cast<int64_t>(w.rt >> 1) * a.nk4 + k4 + c) * (2 * kMxChunkBytes) +
                                              (w.rt & 1) * kMxChunkBytes,
                                          kMxChunkBytes, &full[st.idx]);
                            bulk_load(sS + KC * kMxChunkBytes, a.sf_b + (static_cast<int64_t>(t) * a.nk4 + k4) * (2 * kMxChunkBytes),
                                      KC * 2 * kMxChunkBytes, &full[st.idx]);
                        }
                        if (BASE == kBwdDh) {
                            tma_load_2d(sA, &tmA, &full[st.idx], kelem, w.rt * kDhRows);
                            tma_load_2d(sA + kAStageBytes, &tmA, &full[st.idx], kelem, w.rt * kDhRows + kBM);
                        } else if (BASE == kBwdDw) {
                            // A is U[t, v]: the output row v is the contiguous axis -> four 64-wide boxes of 64 rows t
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                tma_load_2d(sA + j * (kAStageBytes / 2), &tmA, &full[st.idx], w.rt * kDhRows + j * 64, kelem);
                        } else {
                            tma_load_2d(sA, &tmA, &full[st.idx], kelem, w.rt * kBM);
                        }
                        if (B_MN) {
                            // B is stored with the output column as the contiguous axis (W[v, n] in the dH pass, H[t, n] in
                            // the dW pass, W[k, v] in the forward passes over a [d, V] head) -> four 64-column boxes
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                tma_load_2d(sB + j * (kBStageBytes / 4), &tmB, &full[st.idx], t * kBN + j * 64, kelem);
                        } else {
                            tma_load_2d(sB, &tmB, &full[st.idx], kelem, t * kBN);
                        }
                        ++issued;
                        st.advance();
                    }
                }
                if (pacer.ring) pacer.top_up(n, (fills + kPaceFills - 1) / kPaceFills);
            }
            if (pacer.ring)                                     // units of the last wave that this CTA does not have
                for (const int waves = (num_units + gridDim.x - 1) / gridDim.x; n < waves; ++n) pacer.top_up(n, 0);
            *issued_slot = issued;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (MX) reg_dealloc<32>();
        if (lane == 0) {
            constexpr uint32_t idesc =
                (MODE == kFwdFp8T || MX) ? make_idesc(kFmtE4M3, kFmtE4M3, kBM, kBN, 0, 0)
                                  : make_idesc(kFmtBF16, kFmtBF16, kBM, kBN, BASE == kBwdDw ? 1 : 0, B_MN ? 1 : 0);
            Pipe st(STG), tb(NBUF);
            bool ok = true;
            for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
                const Unit w = decode_unit<BASE>(a, u);
                if (!unit_active<BASE>(a, w)) continue;
                for (int t = w.t0; t < w.t1 && ok; ++t) {
                    if (!mbar_wait(&tempty[tb.idx], tb.phase ^ 1u, abort_flag, a.wait_cycles)) { ok = false; break; }
                    tc_fence_after();
                    for (int ks = 0; ks < a.ksteps; ++ks) {
                        if (!mbar_wait(&full[st.idx], st.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sA = smem_u32(stage_base + st.idx * STG_BYTES);
                        const uint32_t sB = sA + A_BYTES;
                        if (BASE == kBwdDh) {
                            // two row tiles share every B slice: accumulators at TMEM columns 0 and 256
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint64_t bdesc = B_MN ? smem_desc_sw128(sB + j * 2048, kBStageBytes / 4, 1024)
                                                            : smem_desc_sw128(sB + j * 32, 16, 1024);
                                const uint32_t accum = (ks > 0 || j > 0) ? 1u : 0u;
                                mma_f16(tmem_base, smem_desc_sw128(sA + j * 32, 16, 1024), bdesc, idesc, accum);
                                mma_f16(tmem_base + kBN, smem_desc_sw128(sA + kAStageBytes + j * 32, 16, 1024), bdesc, idesc, accum);
                            }
                        } else if (BASE == kBwdDw) {
                            // both operands have the contraction axis t as rows of 128 bytes: 16 rows (2048 bytes) per
                            // MMA; 64-wide chunks of the output axis are 8 KB apart
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint64_t bdesc = smem_desc_sw128(sB + j * 2048, kBStageBytes / 4, 1024);
                                const uint32_t accum = (ks > 0 || j > 0) ? 1u : 0u;
                                mma_f16(tmem_base, smem_desc_sw128(sA + j * 2048, kAStageBytes / 2, 1024), bdesc, idesc, accum);
                                mma_f16(tmem_base + kBN, smem_desc_sw128(sA + kAStageBytes + j * 2048, kAStageBytes / 2, 1024), bdesc,
                                        idesc, accum);
                            }
                        } else if (MX) {
                            // the scale warps have put this stage's scales into its column set: A's chunks first (4 columns
                            // each), then B's (4 columns per 128 rows and chunk).  One block-scaled instruction per 32 bytes
                            // of K, each with its scale id.
                            constexpr int KC = FP4 ? 2 : 1;
                            if (!mbar_wait(&sfull[st.idx], st.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                            tc_fence_after();
                            const uint32_t tsf = tmem_base + kMxScaleCol + st.idx * kMxSetCols;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint64_t adesc = smem_desc_sw128(sA + j * 32, 16, 1024);
                                const uint64_t bdesc = smem_desc_sw128(sB + j * 32, 16, 1024);
                                const uint32_t accum = (ks > 0 || j > 0) ? 1u : 0u;
                                if (FP4) {
                                    // instruction j covers scale blocks 2j, 2j+1: chunk j / 2, bytes 2 (j % 2) and the next
                                    const uint32_t id = 2u * (j & 1), sel = id << 30;
                                    mma_mxf4(tmem_base, adesc, bdesc, make_idesc_mx(kBM, kBN, id, 1u), (tsf + 4 * (j >> 1)) | sel,
                                             (tsf + 4 * KC + 8 * (j >> 1)) | sel, accum);
                                } else {
                                    const uint32_t sel = static_cast<uint32_t>(j) << 30;      // byte of the scale columns
                                    mma_mxf8(tmem_base, adesc, bdesc, make_idesc_mx(kBM, kBN, j), tsf | sel, (tsf + 4) | sel, accum);
                                }
                            }
                        } else {
                            const uint32_t dcol = tmem_base + tb.idx * kBN;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint64_t adesc = smem_desc_sw128(sA + j * 32, 16, 1024);
                                const uint64_t bdesc = B_MN ? smem_desc_sw128(sB + j * 2048, kBStageBytes / 4, 1024)
                                                            : smem_desc_sw128(sB + j * 32, 16, 1024);
                                if (MODE == kFwdFp8T) mma_f8(dcol, adesc, bdesc, idesc, (ks > 0 || j > 0) ? 1u : 0u);
                                else mma_f16(dcol, adesc, bdesc, idesc, (ks > 0 || j > 0) ? 1u : 0u);
                            }
                        }
                        tc_commit(&empty[st.idx]);
                        st.advance();
                    }
                    if (ok) {
                        tc_commit(&tfull[tb.idx]);
                        tb.advance();
                    }
                }
            }
            // everything issued has to finish before the tensor memory is given back
            tc_commit(done);
        }
    } else if (warp < 4) {
        if (MX) reg_dealloc<32>();          // the idle warps of the first warpgroup give their registers away too
    } else if (MX && warp >= kScaleWarp0) {
        // ------------------------------------------------------------------ scale warps (microscaling passes)
        // A scale chunk in shared memory is 32 rows of 16 bytes: row l holds, for each of four 32-row groups, the
        // four E8M0 bytes of the stage's K blocks.  The MMA reads scales from tensor memory, lane l of every lane
        // quarter, one 32-bit column per group: warp 12 + q copies the stage's chunks to quarter q with plain stores
        // (a tcgen05.cp from the MMA thread would queue in front of the MMAs and costs about a tenth of the pass).
        // A stage's column set is free again once its `empty` barrier has completed, which the producer waited for
        // before the loads that complete `full`.
        reg_dealloc<32>();
        constexpr int KC = FP4 ? 2 : 1;
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        Pipe st(STG);
        bool ok = true;
        for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            const Unit w = decode_unit<BASE>(a, u);
            if (!unit_active<BASE>(a, w)) continue;
            for (int t = w.t0; t < w.t1 && ok; ++t) {
                for (int ks = 0; ks < a.ksteps; ++ks) {
                    if (!mbar_wait_warp(&full[st.idx], st.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                    const uint4* src = reinterpret_cast<const uint4*>(mx_scale_base + st.idx * kMxStageScaleBytes) + lane;
                    const uint32_t tsf = tmem_base + lane_addr + kMxScaleCol + st.idx * kMxSetCols;
#pragma unroll
                    for (int c = 0; c < 3 * KC; ++c) tmem_st_32x32b_x4(tsf + 4 * c, src[c * (kMxChunkBytes / 16)]);
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sfull[st.idx]);
                    st.advance();
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        if (MX) reg_alloc<224>();
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int half = (warp - 4) >> 2;             // column half of the accumulator
        const int r_in_tile = q * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        Pipe tb(NBUF);
        bool ok = true;
        uint32_t flags = 0;
        for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            const Unit w = decode_unit<BASE>(a, u);
            if (!unit_active<BASE>(a, w)) {
                // nothing was loaded or multiplied for this unit: write the neutral output where later passes read it
                if (BASE == kBwdDh) {
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        const int64_t lr = static_cast<int64_t>(w.rt) * kDhRows + sub * kBM + r_in_tile;
                        if (lr < a.rows) {
                            uint4* dst = reinterpret_cast<uint4*>(a.dH + (a.row0 + lr) * a.lddh + w.t0 * kBN + half * 128);
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (w.t0 * kBN + half * 128 + j * 8 < a.ncols) dst[j] = make_uint4(0, 0, 0, 0);
                        }
                    }
                } else if (BASE == kBwdP) {
                    const int64_t lr = static_cast<int64_t>(w.rt) * kBM + r_in_tile;
                    if (lr < a.rows) {
                        for (int t = w.t0; t < w.t1; ++t) {
                            uint4* dst = reinterpret_cast<uint4*>(a.U + lr * a.ldU + t * kBN + half * 128);
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (t * kBN + half * 128 + j * 8 < a.ncols) dst[j] = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                continue;       // forward passes: the rows are masked, the merge kernel never reads their partials
            }
            if (BASE == kBwdDh) {
                // one unit = 256 rows x 256 columns of dH, finished after the whole contraction over the vocabulary
                if (!mbar_wait_warp(&tfull[0], tb.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    const int64_t lrow2 = static_cast<int64_t>(w.rt) * kDhRows + sub * kBM + r_in_tile;
                    const bool in = lrow2 < a.rows;
                    const int64_t grow2 = a.row0 + lrow2;
                    const uint32_t taddr2 = tmem_base + lane_addr + sub * kBN + half * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int col0 = w.t0 * kBN + half * 128 + c * 32;
                        uint32_t v[32];
                        tmem_ld32(taddr2 + c * 32, v);
                        tmem_ld_wait(v);
                        if (in && col0 < a.ncols) {
                            uint32_t pk[16];
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                pk[i >> 1] = pack_bf16(__uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                            }
                            uint4* dst = reinterpret_cast<uint4*>(a.dH + grow2 * a.lddh + col0);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                if (col0 + j * 8 < a.ncols) dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[0]);
                tb.advance();
                continue;
            }
            if (BASE == kBwdDw) {
                // one unit = 256 vocabulary rows x 256 columns of dW after the contraction over this launch's rows
                if (!mbar_wait_warp(&tfull[0], tb.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    const int64_t vrow = static_cast<int64_t>(w.rt) * kDhRows + sub * kBM + r_in_tile;
                    const bool in = vrow < a.rows;
                    const uint32_t taddr2 = tmem_base + lane_addr + sub * kBN + half * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int col0 = w.t0 * kBN + half * 128 + c * 32;
                        uint32_t v[32];
                        tmem_ld32(taddr2 + c * 32, v);
                        tmem_ld_wait(v);
                        if (in && col0 < a.ncols) {
                            float4* dst = reinterpret_cast<float4*>(a.dW + vrow * a.lddw + col0);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (col0 + j * 4 < a.ncols) {
                                    float4 o = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                           __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                                    if (a.dw_accumulate) {
                                        const float4 old = dst[j];
                                        o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                                    }
                                    dst[j] = o;
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[0]);
                tb.advance();
                continue;
            }
            const int64_t lrow = static_cast<int64_t>(w.rt) * kBM + r_in_tile;   // row inside this launch
            const bool row_ok = lrow < a.rows;
            const int64_t grow = a.row0 + lrow;
            int y = -1;
            bool valid = false;
            if (row_ok) {
                y = a.tokens[grow];
                valid = a.mask[grow] != 0;
                if (valid && (y < 0 || y >= a.ncols)) { flags |= AIS_FLAG_TOKEN_RANGE; y = -1; }
            }
            float m2 = kNegBig, s = 0.f, zy = -INFINITY;       // log2-domain running max, sum, target logit
            const float tscale = (MODE == kFwdFp8T) ? (*a.scale_a) * (*a.scale_b) : 1.f;
            float lse2 = 0.f;
            float cf = 0.f;                                    // recompute: c_t, folded into the scratch
            if (BASE == kBwdP && row_ok) {
                lse2 = a.lse[grow] * kLog2e;
                cf = a.coef[grow];
                if (cf == 0.f) valid = false;                  // rows without gradient are written as exact zeros
            }

            for (int t = w.t0; t < w.t1 && ok; ++t) {
                const int col_base = t * kBN + half * 128;    // first output column of this thread's half
                {
                    if (!mbar_wait_warp(&tfull[tb.idx], tb.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                    tc_fence_after();
                }

                const uint32_t taddr = tmem_base + lane_addr + tb.idx * kBN + half * 128;
                uint32_t vv[MX ? 4 : 1][32];
                if (MX) {
                    // the thread's 128 columns at once, then the accumulator is free for the next tile's MMAs
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(taddr + c * 32, vv[MX ? c : 0]);
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld_wait(vv[MX ? c : 0]);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tempty[tb.idx]);
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int col0 = col_base + c * 32;
                    float x[32];
                    if (MX) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(vv[MX ? c : 0][i]);
                    } else {
                        uint32_t v[32];
                        tmem_ld32(taddr + c * 32, v);
                        tmem_ld_wait(v);
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(v[i]);
                        if (MODE == kFwdFp8T) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) x[i] *= tscale;
                        }
                    }
                    if (BASE == kFwdBf16 || MODE == kFwdFp8T || MX) {
                        if (y >= col0 && y < col0 + 32) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (col0 + i == y) zy = x[i];
                        }
                        if (col0 + 32 > a.ncols) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (col0 + i >= a.ncols) x[i] = -INFINITY;
                        }
                        float cm = x[0];
#pragma unroll
                        for (int i = 1; i < 32; ++i) cm = fmaxf(cm, x[i]);
                        const float m_new = fmaxf(m2, cm * kLog2e);
                        float add = 0.f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) add += ex2(fmaf(x[i], kLog2e, -m_new));
                        s = fmaf(s, ex2(m2 - m_new), add);
                        m2 = m_new;
                    } else if (BASE == kBwdP) {
                        if (row_ok && col0 < a.ncols) {
                            uint32_t pk[16];
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                float p0 = valid ? ex2(fmaf(x[i], kLog2e, -lse2)) : 0.f;
                                float p1 = valid ? ex2(fmaf(x[i + 1], kLog2e, -lse2)) : 0.f;
                                if (col0 + i == y) p0 -= 1.f;
                                if (col0 + i + 1 == y) p1 -= 1.f;
                                pk[i >> 1] = pack_bf16(valid ? cf * p0 : 0.f, valid ? cf * p1 : 0.f);
                            }
                            uint4* dst = reinterpret_cast<uint4*>(a.U + lrow * a.ldU + col0);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                if (col0 + j * 8 < a.ncols) dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                        }
                    }
                }
                if (!MX) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tempty[tb.idx]);
                }
                tb.advance();
            }
            if (ok && row_ok && (BASE == kFwdBf16 || MODE == kFwdFp8T || MX)) {
                const int64_t o = static_cast<int64_t>(w.part * 2 + half) * a.part_ld + grow;
                a.part_m[o] = m2 * kLn2;
                a.part_s[o] = s;
                a.part_z[o] = zy;
            }
        }
        if (flags && a.status) atomicOr(a.status, flags);
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (lane == 0) mbar_wait_drain(done, 0);   // immediate unless the CTA is giving up early
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && *abort_flag) {
        // some role gave up on a wait: let the producer's copies still in flight land before the CTA exits
        drain_stage_copies(full, *issued_slot, STG);
        if (a.status) atomicOr(a.status, AIS_FLAG_TIMEOUT);
    }
}

}  // namespace

template <int MODE>
static cudaError_t launch_mode(const CUtensorMap& tmA, const CUtensorMap& tmB, const LmheadArgs& args, int num_ctas,
                               cudaStream_t stream) {
    lmhead_kernel<MODE><<<num_ctas, threads_of(MODE), kSmemBytes, stream>>>(tmA, tmB, args);
    return cudaGetLastError();
}

cudaError_t launch_lmhead(int mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                          const CUtensorMap& tmSB, const LmheadArgs& args, int num_ctas, cudaStream_t stream) {
    switch (mode) {
        case kFwdBf16: return launch_mode<kFwdBf16>(tmA, tmB, args, num_ctas, stream);
        case kFwdFp8:  return launch_lmhead_fp8_block(tmA, tmB, tmSA, tmSB, args, num_ctas, stream);
        case kBwdP:    return launch_mode<kBwdP>(tmA, tmB, args, num_ctas, stream);
        case kBwdDh:   return launch_mode<kBwdDh>(tmA, tmB, args, num_ctas, stream);
        case kFwdFp8T: return launch_mode<kFwdFp8T>(tmA, tmB, args, num_ctas, stream);
        case kBwdDw:   return launch_mode<kBwdDw>(tmA, tmB, args, num_ctas, stream);
        case kFwdMx:   return launch_mode<kFwdMx>(tmA, tmB, args, num_ctas, stream);
        case kFwdMx4:  return launch_mode<kFwdMx4>(tmA, tmB, args, num_ctas, stream);
        case kFwdBf16Dv: return launch_mode<kFwdBf16Dv>(tmA, tmB, args, num_ctas, stream);
        case kBwdPDv:    return launch_mode<kBwdPDv>(tmA, tmB, args, num_ctas, stream);
        case kBwdDhDv:   return launch_mode<kBwdDhDv>(tmA, tmB, args, num_ctas, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t lmhead_prepare() {
    cudaError_t e;
    e = cudaFuncSetAttribute(lmhead_kernel<kFwdBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = lmhead_fp8_block_prepare();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kBwdP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kBwdDh>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kFwdFp8T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kBwdDw>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kFwdMx>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kFwdBf16Dv>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kBwdPDv>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_kernel<kBwdDhDv>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(lmhead_kernel<kFwdMx4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

}  // namespace ais

// Rollout log-probabilities from E4M3 codes with one fp32 scale per block of 128 / 64 / 32 elements along d.
//
// The scales are arbitrary fp32 numbers, so the hardware's block-scaled MMA kinds (power-of-two scales) do not
// apply: every scale block's partial sum is accumulated alone in tensor memory, read back and promoted on the
// CUDA cores as acc += (partial * sH[row]) * sW[col], two columns per instruction (packed fp32).  One persistent CTA per SM:
//   warp 0      TMA producer: one stage = 128 K-bytes of A (128 rows) and B (256 rows) plus the stage's scale
//               vectors, all completing on the stage's barrier
//   warps 1, 2  MMA issuers: SG blocks per stage, PER = 4 / SG instructions per block, one commit per block; two
//               256-column tensor-memory buffers alternate between blocks, issuer i owning buffer i
//   warps 4-11  promotion + streaming log-sum-exp: warp w reads lane quarter w % 4, column half (w - 4) / 4 in the
//               16x256b fragment shape (a thread owns 4 rows x 32 columns, so it needs 4 + 32 scale values per
//               block).  The four 32-register pieces of a partial tile are software-pipelined: the load of piece
//               p + 1 is in flight during the arithmetic of piece p, and the buffer goes back to its MMA issuer as
//               soon as the last piece has landed.
// The epilogue never waits for the scales separately: an MMA issuer saw the stage barrier complete before it
// issued the block whose completion the epilogue waits for.  The first warpgroup hands registers to the other
// two (384 threads x 168 registers at launch = 128 x 40 + 256 x 232).
// What sets the pace is the chain of one promotion warp per block -- wait for the block, four tensor-memory loads of
// about 190 clocks each with the arithmetic of the piece before in their shadow, hand-over -- which is why the
// arithmetic is packed (it then fits the shadow) and why the MMA side is spread over two threads (one thread, sharing
// its scheduler with two promotion warps, needed about 1,300 clocks per block for wait, four MMAs and two commits).
#include <type_traits>

#include "lmhead_common.cuh"
#include "../../include/ais.h"

namespace ais {

namespace {

template <int SG>
struct Fp8Cfg {
    static constexpr int kSlots = (SG == 4) ? 5 : 8;                  // scale slots: more than stages + buffers in flight
    static constexpr int kSlotBytes = SG * (kBM + kBN) * 4;
    static constexpr int kSlotBOffset = SG * kBM * 4;
    static constexpr int kBarriers = 2 * kStages + 4 + kSlots + 1;
    static constexpr int kSmem = 1024 + kStages * kStageBytes + kSlots * kSlotBytes + kBarriers * 8 + 64;
};
static_assert(Fp8Cfg<4>::kSmem <= 232448 && Fp8Cfg<1>::kSmem <= 232448, "shared memory of the FP8 pass");

template <int SG>
__global__ void __launch_bounds__(kThreads, 1)
lmhead_fp8_block_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        const __grid_constant__ CUtensorMap tmSA, const __grid_constant__ CUtensorMap tmSB,
                        const LmheadArgs a) {
    using C = Fp8Cfg<SG>;
    constexpr int PER = 4 / SG;                     // MMAs (32 K-bytes each) per scale block
    constexpr int MODE = kFwdFp8;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned start, as an offset from the array so that the compiler still knows the address space
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* stage_base = smem;
    uint8_t* scale_base = smem + kStages * kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(scale_base + C::kSlots * C::kSlotBytes);
    uint64_t* full = bars;                       // [kStages]  TMA -> MMA (operands and scales of the stage)
    uint64_t* empty = full + kStages;            // [kStages]  MMA -> TMA
    uint64_t* tfull = empty + kStages;           // [2]        MMA -> epilogue: a block's partial sums are complete
    uint64_t* tempty = tfull + 2;                // [2]        epilogue -> MMA: the partial sums are in registers
    uint64_t* sempty = tempty + 2;               // [kSlots]   epilogue -> TMA: the stage's scales have been used
    uint64_t* done = sempty + C::kSlots;         // [1]        all MMAs of this CTA have completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kBarriers);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* issued_slot = tmem_slot + 2;     // stage fills the producer has requested (written when it leaves its loop)

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_units = a.n_row_tiles * a.nsplit;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], SG > 1 ? 2 : 1); }   // both issuers use a stage when it holds several blocks
        for (int i = 0; i < 2; ++i) { mbar_init(&tfull[i], 1); mbar_init(&tempty[i], kEpiWarps); }
        for (int i = 0; i < C::kSlots; ++i) mbar_init(&sempty[i], kEpiWarps);
        mbar_init(done, 2);
        *abort_flag = 0;
        *issued_slot = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmSA);
        tma_prefetch_desc(&tmSB);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
        reg_dealloc<40>();
        if (warp == 0) {
            // ------------------------------------------------------------------ TMA producer
            if (lane == 0) {
                Pipe st(kStages), sc(C::kSlots);
                uint32_t issued = 0;
                bool ok = true;
                for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
                    const Unit w = decode_unit<MODE>(a, u);
                    if (!unit_active<MODE>(a, w)) continue;
                    for (int t = w.t0; t < w.t1 && ok; ++t) {
                        for (int ks = 0; ks < a.ksteps; ++ks) {
                            if (!mbar_wait(&empty[st.idx], st.phase ^ 1u, abort_flag, a.wait_cycles)) { ok = false; break; }
                            if (!mbar_wait(&sempty[sc.idx], sc.phase ^ 1u, abort_flag, a.wait_cycles)) { ok = false; break; }
                            uint8_t* sA = stage_base + st.idx * kStageBytes;
                            uint8_t* sS = scale_base + sc.idx * C::kSlotBytes;
                            mbar_expect_tx(&full[st.idx], kStageBytes + C::kSlotBytes);
                            tma_load_2d(sS, &tmSA, &full[st.idx], w.rt * kBM, ks * SG);
                            tma_load_2d(sS + C::kSlotBOffset, &tmSB, &full[st.idx], t * kBN, ks * SG);
                            tma_load_2d(sA, &tmA, &full[st.idx], ks * 128, w.rt * kBM);
                            tma_load_2d(sA + kAStageBytes, &tmB, &full[st.idx], ks * 128, t * kBN);
                            ++issued;
                            st.advance();
                            sc.advance();
                        }
                    }
                }
                *issued_slot = issued;
            }
        } else if (warp == 1 || warp == 2) {
            // ------------------------------------------------------------------ MMA issuers
            // Two of them, on two schedulers: issuer `me` owns tensor-memory buffer `me` and takes every other scale
            // block (block n of the CTA goes to buffer n % 2).  One thread cannot keep up: it shares its scheduler with
            // two promotion warps, and wait + four MMAs + two commits took it about 1,300 clocks per block against the
            // 542 the tensor core needs.  The two threads are independent: different buffers, different barriers.
            if (lane == 0) {
                const uint32_t me = warp - 1;
                constexpr uint32_t idesc = make_idesc(kFmtE4M3, kFmtE4M3, kBM, kBN, 0, 0);
                const uint64_t desc0 = smem_desc_sw128(0, 16, 1024);           // descriptor of address 0: add (address >> 4)
                const uint32_t dcol = tmem_base + me * kBN;
                Pipe st(kStages);
                uint32_t tphase = 0;                                            // phase of this issuer's buffer barriers
                uint32_t nstage = 0;                                            // stages seen so far (SG == 1: parity picks the owner)
                bool ok = true;
                for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
                    const Unit w = decode_unit<MODE>(a, u);
                    if (!unit_active<MODE>(a, w)) continue;
                    const int nst = (w.t1 - w.t0) * a.ksteps;
                    for (int i = 0; i < nst && ok; ++i, ++nstage) {
                        if (SG > 1 || (nstage & 1u) == me) {
                            if (!mbar_wait(&full[st.idx], st.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                            const uint64_t adesc = desc0 + (smem_u32(stage_base + st.idx * kStageBytes) >> 4);
#pragma unroll
                            for (int g = 0; g < SG; ++g) {
                                if (SG > 1 && (g & 1) != static_cast<int>(me)) continue;
                                if (!mbar_wait(&tempty[me], tphase ^ 1u, abort_flag, a.wait_cycles)) { ok = false; break; }
                                tc_fence_after();
#pragma unroll
                                for (int j = 0; j < PER; ++j) {
                                    const uint64_t ad = adesc + 2 * (g * PER + j);       // 32 bytes of K further on
                                    mma_f8(dcol, ad, ad + (kAStageBytes >> 4), idesc, j > 0 ? 1u : 0u);
                                }
                                tc_commit(&tfull[me]);
                                tphase ^= 1u;
                            }
                            if (!ok) break;
                            tc_commit(&empty[st.idx]);
                        }
                        st.advance();
                    }
                }
                // everything issued has to finish before the tensor memory is given back
                tc_commit(done);
            }
        }
    } else {
        // ------------------------------------------------------------------ promotion and streaming log-sum-exp
        reg_alloc<232>();
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int half = (warp - 4) >> 2;             // column half of the partial tile
        const int rg = lane >> 2, cp = lane & 3;      // fragment coordinates of this thread
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        Pipe tb(2), sc(C::kSlots);
        bool ok = true;
        uint32_t flags = 0;
        uint32_t va[32], vb[32];
        auto ld_piece = [&](uint32_t buf, int hh, int nb, uint32_t (&v)[32]) {
            tmem_ld_16x256b_x8(tmem_base + lane_base + (static_cast<uint32_t>(hh * 16) << 16) + buf * kBN + half * 128 + nb * 64, v);
        };
        for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            const Unit w = decode_unit<MODE>(a, u);
            if (!unit_active<MODE>(a, w)) continue;     // every row masked: the merge kernel never reads these partials
            int64_t grow4[4];
            bool rok4[4];
            int y4[4];
            float m4[4], s4[4], zy4[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int64_t lr = static_cast<int64_t>(w.rt) * kBM + q * 32 + (r >> 1) * 16 + (r & 1) * 8 + rg;
                rok4[r] = lr < a.rows;
                grow4[r] = a.row0 + lr;
                y4[r] = -1;
                if (rok4[r]) {
                    y4[r] = a.tokens[grow4[r]];
                    if (a.mask[grow4[r]] != 0 && (y4[r] < 0 || y4[r] >= a.ncols)) { flags |= AIS_FLAG_TOKEN_RANGE; y4[r] = -1; }
                }
                m4[r] = kNegBig; s4[r] = 0.f; zy4[r] = -INFINITY;
            }
            for (int t = w.t0; t < w.t1 && ok; ++t) {
                F2 acc[4][16];                             // [row][8-column group]: the pair of columns 8 n + 2 cp, + 1
#pragma unroll
                for (int r = 0; r < 4; ++r)
#pragma unroll
                    for (int n = 0; n < 16; ++n) acc[r][n] = F2{0.f, 0.f};
                for (int ks = 0; ks < a.ksteps && ok; ++ks) {
                    const float* sS = reinterpret_cast<const float*>(scale_base + sc.idx * C::kSlotBytes);
#pragma unroll 1
                    for (int g = 0; g < SG; ++g) {
                        if (!mbar_wait_warp(&tfull[tb.idx], tb.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t buf = tb.idx;
                        ld_piece(buf, 0, 0, va);
                        F2 sh[4];
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const float x = sS[g * kBM + q * 32 + (r >> 1) * 16 + (r & 1) * 8 + rg];
                            sh[r] = F2{x, x};
                        }
                        const float2* sw2 = reinterpret_cast<const float2*>(sS + (C::kSlotBOffset / 4) + g * kBN + half * 128) + cp;
                        // (lane half of the quarter) x (column half of the piece); the indices are compile-time constants so
                        // that the accumulators stay in registers
                        auto promote = [&](auto HH, auto NB, uint32_t (&v)[32]) {
                            constexpr int hh = decltype(HH)::value, nb = decltype(NB)::value;
#pragma unroll
                            for (int mq = 0; mq < 8; ++mq) {
                                const float2 swf = sw2[(nb * 8 + mq) * 4];         // columns 8n + 2cp, +1 of this thread
                                const F2 sw = {swf.x, swf.y};
#pragma unroll
                                for (int e = 0; e < 2; ++e) {
                                    const F2 x = {__uint_as_float(v[4 * mq + 2 * e]), __uint_as_float(v[4 * mq + 2 * e + 1])};
                                    acc[hh * 2 + e][nb * 8 + mq] = fma2(mul2(x, sh[hh * 2 + e]), sw, acc[hh * 2 + e][nb * 8 + mq]);
                                }
                            }
                        };
                        using I0 = std::integral_constant<int, 0>;
                        using I1 = std::integral_constant<int, 1>;
                        tmem_ld_wait(va);
                        ld_piece(buf, 0, 1, vb);
                        promote(I0{}, I0{}, va);
                        tmem_ld_wait(vb);
                        ld_piece(buf, 1, 0, va);
                        promote(I0{}, I1{}, vb);
                        tmem_ld_wait(va);
                        ld_piece(buf, 1, 1, vb);
                        promote(I1{}, I0{}, va);
                        tmem_ld_wait(vb);
                        // the whole partial tile is in registers: hand the buffer back before the last arithmetic
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&tempty[buf]);
                        tb.advance();
                        promote(I1{}, I1{}, vb);
                    }
                    if (!ok) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sempty[sc.idx]);
                    sc.advance();
                }
                if (!ok) break;
                // streaming log-sum-exp over this thread's 32 columns of each of its 4 rows
                const int cbase = t * kBN + half * 128 + 2 * cp;           // column of acc[.][0][0]
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int yy = y4[r] - cbase;                          // = 8n + e for an owned column
                    if (yy >= 0 && yy < 128 && (yy & 6) == 0) {
                        // written as a running maximum on purpose: a chain of "if (k == n) z = acc[n]" is folded by
                        // the compiler into acc[k], and a dynamically indexed array leaves the register file
#pragma unroll
                        for (int n = 0; n < 16; ++n) {
                            zy4[r] = fmaxf(zy4[r], (yy == 8 * n) ? acc[r][n].x : -INFINITY);
                            zy4[r] = fmaxf(zy4[r], (yy == 8 * n + 1) ? acc[r][n].y : -INFINITY);
                        }
                    }
                    if (t * kBN + kBN > a.ncols) {
#pragma unroll
                        for (int n = 0; n < 16; ++n) {
                            if (cbase + 8 * n >= a.ncols) acc[r][n].x = -INFINITY;
                            if (cbase + 8 * n + 1 >= a.ncols) acc[r][n].y = -INFINITY;
                        }
                    }
                    float cm = acc[r][0].x;
#pragma unroll
                    for (int n = 0; n < 16; ++n) cm = fmaxf(cm, fmaxf(acc[r][n].x, acc[r][n].y));
                    const float m_new = fmaxf(m4[r], cm * kLog2e);
                    float add = 0.f;
#pragma unroll
                    for (int n = 0; n < 16; ++n)
                        add += ex2(fmaf(acc[r][n].x, kLog2e, -m_new)) + ex2(fmaf(acc[r][n].y, kLog2e, -m_new));
                    s4[r] = fmaf(s4[r], ex2(m4[r] - m_new), add);
                    m4[r] = m_new;
                }
            }
            // the four threads that share a row merge their (max, sum, target) and one of them writes the partial
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float M = fmaxf(m4[r], __shfl_xor_sync(0xffffffffu, m4[r], 1));
                M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));
                float ssum = s4[r] * ex2(m4[r] - M);
                ssum += __shfl_xor_sync(0xffffffffu, ssum, 1);
                ssum += __shfl_xor_sync(0xffffffffu, ssum, 2);
                float z = fmaxf(zy4[r], __shfl_xor_sync(0xffffffffu, zy4[r], 1));
                z = fmaxf(z, __shfl_xor_sync(0xffffffffu, z, 2));
                if (ok && rok4[r] && cp == 0) {
                    const int64_t o = static_cast<int64_t>(w.part * 2 + half) * a.part_ld + grow4[r];
                    a.part_m[o] = M * kLn2;
                    a.part_s[o] = ssum;
                    a.part_z[o] = z;
                }
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
        drain_stage_copies(full, *issued_slot, kStages);
        if (a.status) atomicOr(a.status, AIS_FLAG_TIMEOUT);
    }
}

}  // namespace

cudaError_t launch_lmhead_fp8_block(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmSA,
                                    const CUtensorMap& tmSB, const LmheadArgs& args, int num_ctas, cudaStream_t stream) {
    switch (args.sgroups) {
        case 1: lmhead_fp8_block_kernel<1><<<num_ctas, kThreads, Fp8Cfg<1>::kSmem, stream>>>(tmA, tmB, tmSA, tmSB, args); break;
        case 2: lmhead_fp8_block_kernel<2><<<num_ctas, kThreads, Fp8Cfg<2>::kSmem, stream>>>(tmA, tmB, tmSA, tmSB, args); break;
        case 4: lmhead_fp8_block_kernel<4><<<num_ctas, kThreads, Fp8Cfg<4>::kSmem, stream>>>(tmA, tmB, tmSA, tmSB, args); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t lmhead_fp8_block_prepare() {
    cudaError_t e;
    e = cudaFuncSetAttribute(lmhead_fp8_block_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp8Cfg<1>::kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(lmhead_fp8_block_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp8Cfg<2>::kSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(lmhead_fp8_block_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fp8Cfg<4>::kSmem);
}

}  // namespace ais

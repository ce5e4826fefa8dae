// Rollout log-probabilities from E4M3 codes with one fp32 scale per block of 128 / 64 / 32 elements along d.
//
// The scales are arbitrary fp32 numbers, so the hardware's block-scaled MMA kinds (power-of-two scales) do not
// apply: every scale block's partial sum is accumulated alone in tensor memory, read back and promoted on the
// CUDA cores as acc += (partial * sH[row]) * sW[col], two columns per instruction (packed fp32).  One persistent CTA per SM:
//   warp 0      TMA producer: one stage = 128 K-bytes of A (128 rows) and B (256 rows) plus the stage's scale
//               vectors, all completing on the stage's barrier
//   warps 1, 2  MMA issuers: SG blocks per stage, PER = 4 / SG instructions per block, one commit per block; two
//               256-column tensor-memory buffers alternate between blocks, issuer i owning buffer i
//   warps 4-11  promotion + streaming log-sum-exp: warp w reads lane quarter w % 4, column half (w - 4) / 4 with
//               32x32b loads (a thread owns one row x 128 columns: its row scale is one register, the column
//               scales come as broadcast 16-byte shared-memory loads).  The four 32-register pieces of a partial
//               tile are software-pipelined: the load of piece p + 1 is in flight during the arithmetic of piece
//               p, and the buffer goes back to its MMA issuer as soon as the last piece has landed.
// The epilogue never waits for the scales separately: an MMA issuer saw the stage barrier complete before it
// issued the block whose completion the epilogue waits for.  The first warpgroup hands registers to the other
// two (384 threads x 168 registers at launch = 128 x 40 + 256 x 232).
// Measured per 128 x 256 x 128 block on the busiest SM: about 1,280 clocks against 542 of tensor-core time.  No single
// unit is the bound (timing-only variants: 790 clocks with an epilogue that only hands the buffers back, 660 without
// the operand copies as well; the tensor-memory loads need about 280 clocks at the 32x32b shape and twice that at
// the 16x256b fragment shape, the packed arithmetic about 350, the column-scale loads about 225): the block goes
// round MMA -> commit -> wait -> load -> release -> wait -> MMA through two buffers, every hand-over costing
// 200-300 clocks, which is why the MMA side is spread over two threads, the arithmetic is packed, and the promotion
// warps poll their barrier without blocking (the blocking form cost 70 clocks per block).
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
                Pacer pacer(a.pace, a.pace_per_unit);
                int n = 0;                                      // ordinal of this CTA's unit (its wave)
                for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x, ++n) {
                    const Unit w = decode_unit<MODE>(a, u);
                    if (!unit_active<MODE>(a, w)) {
                        if (pacer.ring) pacer.top_up(n, 0);
                        continue;
                    }
                    int fills = 0;                              // stage fills of this unit so far
                    for (int t = w.t0; t < w.t1 && ok; ++t) {
                        for (int ks = 0; ks < a.ksteps; ++ks, ++fills) {
                            if (pacer.ring && fills % kPaceFills == 0) pacer.announce(n, fills / kPaceFills);
                            if (pacer.ring && fills % kPaceFills == kPaceSettle) pacer.settle();
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
                    if (pacer.ring) pacer.top_up(n, (fills + kPaceFills - 1) / kPaceFills);
                }
                if (pacer.ring)                                 // units of the last wave that this CTA does not have
                    for (const int waves = (num_units + gridDim.x - 1) / gridDim.x; n < waves; ++n) pacer.top_up(n, 0);
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
        const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
        Pipe tb(2), sc(C::kSlots);
        bool ok = true;
        uint32_t flags = 0;
        uint32_t va[32], vb[32];
        auto ld_piece = [&](uint32_t buf, int p, uint32_t (&v)[32]) {
            tmem_ld32(tmem_base + lane_base + buf * kBN + half * 128 + p * 32, v);
        };
        for (int u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            const Unit w = decode_unit<MODE>(a, u);
            if (!unit_active<MODE>(a, w)) continue;     // every row masked: the merge kernel never reads these partials
            const int64_t lr = static_cast<int64_t>(w.rt) * kBM + q * 32 + lane;
            const bool rok = lr < a.rows;
            const int64_t grow = a.row0 + lr;
            int y = -1;
            if (rok) {
                y = a.tokens[grow];
                if (a.mask[grow] != 0 && (y < 0 || y >= a.ncols)) { flags |= AIS_FLAG_TOKEN_RANGE; y = -1; }
            }
            float m_run = kNegBig, s_run = 0.f, zy = -INFINITY;
            for (int t = w.t0; t < w.t1 && ok; ++t) {
                F2 acc[64];                                // columns 2 n, 2 n + 1 of this thread's 128
#pragma unroll
                for (int n = 0; n < 64; ++n) acc[n] = F2{0.f, 0.f};
                for (int ks = 0; ks < a.ksteps && ok; ++ks) {
                    const float* sS = reinterpret_cast<const float*>(scale_base + sc.idx * C::kSlotBytes);
#pragma unroll 1
                    for (int g = 0; g < SG; ++g) {
                        if (!mbar_wait_warp_spin(&tfull[tb.idx], tb.phase, abort_flag, a.wait_cycles)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t buf = tb.idx;
                        ld_piece(buf, 0, va);
                        const float shx = sS[g * kBM + q * 32 + lane];
                        const F2 sh = {shx, shx};
                        // every lane reads the same column scales: broadcast 16-byte loads
                        const float4* sw4 = reinterpret_cast<const float4*>(sS + (C::kSlotBOffset / 4) + g * kBN + half * 128);
                        auto promote = [&](auto PP, uint32_t (&v)[32]) {
                            constexpr int pp = decltype(PP)::value;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float4 swf = sw4[pp * 8 + j];
                                const F2 x0 = {__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1])};
                                const F2 x1 = {__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])};
                                acc[pp * 16 + 2 * j] = fma2(mul2(x0, sh), F2{swf.x, swf.y}, acc[pp * 16 + 2 * j]);
                                acc[pp * 16 + 2 * j + 1] = fma2(mul2(x1, sh), F2{swf.z, swf.w}, acc[pp * 16 + 2 * j + 1]);
                            }
                        };
                        using I0 = std::integral_constant<int, 0>;
                        using I1 = std::integral_constant<int, 1>;
                        using I2 = std::integral_constant<int, 2>;
                        using I3 = std::integral_constant<int, 3>;
                        tmem_ld_wait(va);
                        ld_piece(buf, 1, vb);
                        promote(I0{}, va);
                        tmem_ld_wait(vb);
                        ld_piece(buf, 2, va);
                        promote(I1{}, vb);
                        tmem_ld_wait(va);
                        ld_piece(buf, 3, vb);
                        promote(I2{}, va);
                        tmem_ld_wait(vb);
                        // the whole partial tile is in registers: hand the buffer back before the last arithmetic
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&tempty[buf]);
                        tb.advance();
                        promote(I3{}, vb);
                    }
                    if (!ok) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sempty[sc.idx]);
                    sc.advance();
                }
                if (!ok) break;
                // streaming log-sum-exp over this thread's 128 columns of its row
                const int cbase = t * kBN + half * 128;                    // column of acc[0].x
                const int yy = y - cbase;
                if (yy >= 0 && yy < 128) {
                    // written as a running maximum on purpose: a chain of "if (k == n) z = acc[n]" is folded by
                    // the compiler into acc[k], and a dynamically indexed array leaves the register file
#pragma unroll
                    for (int n = 0; n < 64; ++n) {
                        zy = fmaxf(zy, (yy == 2 * n) ? acc[n].x : -INFINITY);
                        zy = fmaxf(zy, (yy == 2 * n + 1) ? acc[n].y : -INFINITY);
                    }
                }
                if (t * kBN + kBN > a.ncols) {
#pragma unroll
                    for (int n = 0; n < 64; ++n) {
                        if (cbase + 2 * n >= a.ncols) acc[n].x = -INFINITY;
                        if (cbase + 2 * n + 1 >= a.ncols) acc[n].y = -INFINITY;
                    }
                }
                float cm = acc[0].x;
#pragma unroll
                for (int n = 0; n < 64; ++n) cm = fmaxf(cm, fmaxf(acc[n].x, acc[n].y));
                const float m_new = fmaxf(m_run, cm * kLog2e);
                float add = 0.f;
#pragma unroll
                for (int n = 0; n < 64; ++n)
                    add += ex2(fmaf(acc[n].x, kLog2e, -m_new)) + ex2(fmaf(acc[n].y, kLog2e, -m_new));
                s_run = fmaf(s_run, ex2(m_run - m_new), add);
                m_run = m_new;
            }
            if (ok && rok) {
                const int64_t o = static_cast<int64_t>(w.part * 2 + half) * a.part_ld + grow;
                a.part_m[o] = m_run * kLn2;
                a.part_s[o] = s_run;
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

// Device helpers shared by the LM-head tensor-core kernels: stage-ring bookkeeping, warp-wide bounded waits,
// register re-splitting, work-unit decoding and the test for row tiles without work.
#pragma once

#include "lmhead.cuh"
#include "ptx.cuh"

namespace ais {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegBig = -1.0e30f;

struct Pipe {
    uint32_t idx = 0, phase = 0;
    int n;
    __device__ explicit Pipe(int n_) : n(n_) {}
    __device__ __forceinline__ void advance() {
        if (++idx == static_cast<uint32_t>(n)) { idx = 0; phase ^= 1u; }
    }
};

// Pacing of the persistent CTAs of one launch.  CTAs that share operand tiles through L2 (the column slices of a row
// pair, the row tiles of a vocabulary range) only hit there while they stay within a few dozen stage fills of each
// other, and left alone they drift apart by several per cent of a unit per unit.  Each CTA's producer therefore
// announces every kPaceFills-th stage fill of its n-th unit on a ring of counters in the workspace and lets the slowest
// CTA catch up to within kPaceLag announcements before it goes on.  The wait is advisory and bounded: after
// kPaceWait clock ticks the producer goes on regardless, and after three such give-ups in a row it stops waiting
// for the rest of the launch (it still announces), so CTAs that are not all resident at once cost time, not progress.
// Every announcement index receives exactly gridDim.x arrivals: units without work and the missing units of the
// last wave are announced in one go.
constexpr int kPaceLag = 2;
constexpr long long kPaceWait = 200000;  // clock ticks

struct Pacer {
    uint32_t* ring;      // nullptr: no pacing
    int per_unit;        // announcements per unit (the same for every unit of the launch)
    int strikes = 0;
    const volatile uint32_t* slot = nullptr;   // counter this CTA still has to see reach `want` (nullptr: nothing pending)
    uint32_t want = 0, seen = 0;
    __device__ Pacer(uint32_t* r, int c) : ring(r), per_unit(c) {}
    // Announcement c of unit n.  The counter to wait for is read here and looked at in settle(), a few stage fills
    // later, so that the read's round trip to L2 is not spent waiting.
    __device__ __forceinline__ void announce(int n, int c) {
        const long long k = static_cast<long long>(n) * per_unit + c;
        atomicAdd(&ring[k % kPaceRing], 1u);
        const long long kw = k - kPaceLag;
        if (kw < 0 || strikes >= 3) return;
        want = static_cast<uint32_t>(gridDim.x) * static_cast<uint32_t>(kw / kPaceRing + 1);
        slot = ring + (kw % kPaceRing);
        seen = *slot;
    }
    __device__ __forceinline__ void settle() {
        if (slot == nullptr) return;
        if (seen < want) {
            const long long t0 = clock64();
            while (*slot < want) {
                if (clock64() - t0 > kPaceWait) { ++strikes; slot = nullptr; return; }
            }
        }
        strikes = 0;
        slot = nullptr;
    }
    // announcements c_from .. per_unit - 1 of unit n without waiting (unit ended early, had no work, or does not exist)
    __device__ __forceinline__ void top_up(int n, int c_from) {
        for (int c = c_from; c < per_unit; ++c)
            atomicAdd(&ring[(static_cast<long long>(n) * per_unit + c) % kPaceRing], 1u);
    }
};

// Warp-wide wait: every lane polls (so every lane observes the completed phase itself) and the outcome is
// made uniform, because the tcgen05.ld / __syncwarp that follow need the whole warp.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                               long long limit = 0) {
    const bool r = mbar_wait(bar, parity, abort_flag, limit);
    return __all_sync(0xffffffffu, r);
}

__device__ __forceinline__ bool mbar_wait_warp_spin(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                    long long limit = 0) {
    const bool r = mbar_wait_spin(bar, parity, abort_flag, limit);
    return __all_sync(0xffffffffu, r);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int N>
__device__ __forceinline__ void reg_alloc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_dealloc() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Which row tile and which column tiles a work unit covers.
struct Unit {
    int rt, t0, t1, part;
};
template <int MODE>
__device__ __forceinline__ Unit decode_unit(const LmheadArgs& a, int u) {
    Unit w;
    if (MODE == kBwdDh || MODE == kBwdDw) {
        w.rt = u / a.n_col_tiles;
        w.t0 = u % a.n_col_tiles;
        w.t1 = w.t0 + 1;
        w.part = 0;
    } else {
        w.rt = u / a.nsplit;
        const int c = u % a.nsplit;
        w.t0 = static_cast<int>((static_cast<int64_t>(c) * a.n_col_tiles) / a.nsplit);
        w.t1 = static_cast<int>((static_cast<int64_t>(c + 1) * a.n_col_tiles) / a.nsplit);
        w.part = c;
    }
    return w;
}

// Row tiles in which no row needs computing (all rows masked in the forward passes, all gradient factors zero in
// the backward passes) are skipped by all three roles alike; the epilogue writes the neutral output where one is
// needed.  The dW pass contracts over rows, so it has nothing to skip.
template <int MODE>
__device__ __forceinline__ bool unit_active(const LmheadArgs& a, const Unit& w) {
    if (MODE == kBwdDw || a.tile_active == nullptr) return true;
    const int64_t g = a.row0 / kBM;
    if (MODE == kBwdDh) {
        const int64_t t0 = g + 2 * static_cast<int64_t>(w.rt);
        const bool second = (2 * static_cast<int64_t>(w.rt) + 1) * kBM < a.rows;
        return a.tile_active[t0] != 0 || (second && a.tile_active[t0 + 1] != 0);
    }
    return a.tile_active[g + w.rt] != 0;
}

// After every role has left its loops: if the CTA gave up on a wait, the tile copies that the producer issued last
// (one per stage of the ring at most) may still be in flight.  Wait for them, so that no copy writes into shared
// memory that the CTA has already given back; `issued` counts the producer's stage fills.
__device__ __forceinline__ void drain_stage_copies(uint64_t* full, uint32_t issued, uint32_t stages) {
    const uint32_t pending = issued < stages ? issued : stages;
    for (uint32_t i = 0; i < pending; ++i) {
        const uint32_t n = issued - 1 - i;                 // n-th fill overall: stage n % stages, phase n / stages
        mbar_wait_drain(&full[n % stages], (n / stages) & 1u);
    }
}

}  // namespace

}  // namespace ais

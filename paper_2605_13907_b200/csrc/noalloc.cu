// Trainer log-probabilities without any caller-provided scratch: the per-split partial triples live in a
// fixed array that is part of the library image (see ais_logprob_train_static in include/ais.h).
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/ais.h"
#include "host_setup.cuh"
#include "lmhead.cuh"
#include "stream_kernels.cuh"

namespace {

using namespace ais;

constexpr int kStaticNsplit = 4;                                   // vocabulary ranges per row tile
constexpr int kStaticParts = 2 * kStaticNsplit;                    // two column halves per range
constexpr int64_t kStaticLd = AIS_STATIC_MAX_ROWS;                 // rows per partial plane
constexpr size_t kStaticFloats = static_cast<size_t>(3) * kStaticParts * kStaticLd;

// 3 planes (running max, sum of exponentials, target logit) x 8 parts x 16384 rows of float = 1.5 MiB.
// Every GPU on which the library is loaded holds this array until the process exits.
static __device__ __align__(256) float g_static_partials[kStaticFloats];

constexpr int kMaxDevices = 64;
float* g_static_addr[kMaxDevices];      // device address of g_static_partials on each device, once resolved
std::mutex g_smutex;

// Once per device, with that device current: the library's common set-up, then the device address of the static
// array (its name is only a host-side handle in host code).  A failure is not remembered here, so a later call
// tries again; the common set-up remembers a wrong architecture itself.
int static_setup(float** partials, int* num_sms) {
    const int st = device_setup(num_sms);
    if (st != AIS_OK) return st;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AIS_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_smutex);
    if (!g_static_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) return AIS_ERR_DEVICE;
        g_static_addr[dev] = static_cast<float*>(p);
    }
    *partials = g_static_addr[dev];
    return AIS_OK;
}

}  // namespace

extern "C" int ais_logprob_train_static(const ais_shape* shape, const void* H, const void* W, const int32_t* tokens,
                                        const uint8_t* mask, float* lp_train, float* lse_train, uint32_t* dev_status,
                                        void* stream) {
    if (!shape || !H || !W || !tokens || !mask || !lp_train) return AIS_ERR_NULL;
    if (shape->T < 0 || shape->d <= 0 || shape->V <= 0 || shape->w_layout != AIS_W_VD) return AIS_ERR_SHAPE;
    if (shape->d % 64 != 0 || shape->V % 8 != 0 || shape->ldh < shape->d || shape->ldw < shape->d) return AIS_ERR_SHAPE;
    if (shape->ldh % 8 != 0 || shape->ldw % 8 != 0) return AIS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(H) | reinterpret_cast<uintptr_t>(W)) % 16 != 0) return AIS_ERR_ALIGN;
    if (shape->T > AIS_STATIC_MAX_ROWS) return AIS_ERR_LIMIT;       // the fixed scratch holds no more rows
    float* partials = nullptr;
    int num_sms = 0;
    const int st = static_setup(&partials, &num_sms);
    if (st != AIS_OK) return st;
    if (shape->T == 0) return AIS_OK;

    const int n_col_tiles = (shape->V + kBN - 1) / kBN;
    const int nsplit = n_col_tiles < kStaticNsplit ? n_col_tiles : kStaticNsplit;
    LmheadArgs a;
    memset(&a, 0, sizeof(a));
    a.wait_cycles = wait_cycles();
    a.rows = shape->T;
    a.row0 = 0;
    a.n_row_tiles = static_cast<int32_t>((shape->T + kBM - 1) / kBM);
    a.ncols = shape->V;
    a.n_col_tiles = n_col_tiles;
    a.ksteps = shape->d / 64;
    a.nsplit = nsplit;
    a.sgroups = 1;
    a.tokens = tokens;
    a.mask = mask;
    a.part_m = partials;
    a.part_s = partials + static_cast<size_t>(kStaticParts) * kStaticLd;
    a.part_z = partials + static_cast<size_t>(2 * kStaticParts) * kStaticLd;
    a.part_ld = kStaticLd;
    a.status = dev_status;
    CUtensorMap tmA, tmB;
    if (!make_tmap(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, H, static_cast<uint64_t>(shape->d), static_cast<uint64_t>(shape->T),
                   shape->ldh * 2, 64, kBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, static_cast<uint64_t>(shape->d), static_cast<uint64_t>(shape->V),
                   shape->ldw * 2, 64, kBN, CU_TENSOR_MAP_SWIZZLE_128B))
        return AIS_ERR_DEVICE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int units = a.n_row_tiles * nsplit;
    // Every slot of the scratch that the merge reads (parts 0 .. 2*nsplit-1, rows 0 .. T-1) is written by the
    // pass just before it, so nothing left over from an earlier call is ever read and nothing needs zeroing.
    if (launch_lmhead(kFwdBf16, tmA, tmB, tmA, tmB, a, units < num_sms ? units : num_sms, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (launch_combine(a.part_m, a.part_s, a.part_z, nsplit * 2, kStaticLd, mask, shape->T, lp_train, lse_train, dev_status, s) !=
        cudaSuccess)
        return AIS_ERR_DEVICE;
    return AIS_OK;
}

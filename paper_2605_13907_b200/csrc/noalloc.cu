// Trainer log-probabilities without any caller-provided scratch: the per-split partial triples live in a
// fixed array that is part of the library image (see ais_logprob_train_static in include/ais.h).
#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/ais.h"
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
struct StaticDev {
    bool tried = false;
    int status = AIS_ERR_DEVICE;
    int num_sms = 0;
    float* partials = nullptr;          // device address of g_static_partials on this device
};
StaticDev g_sdev[kMaxDevices];
std::mutex g_smutex;
PFN_cuTensorMapEncodeTiled_v12000 g_sencode = nullptr;

// Once per device, with that device current: resolve the device address of the static array (its name
// is only a host-side handle in host code), check the architecture and prepare the kernels.
int static_setup(StaticDev** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AIS_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_smutex);
    StaticDev& sd = g_sdev[dev];
    if (!sd.tried) {
        sd.tried = true;
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess || prop.major != 10) return sd.status;
        if (!g_sencode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
                qres != cudaDriverEntryPointSuccess || !fn)
                return sd.status;
            g_sencode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
        }
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) return sd.status;
        if (lmhead_prepare() != cudaSuccess) return sd.status;
        sd.partials = static_cast<float*>(p);
        sd.num_sms = prop.multiProcessorCount;
        sd.status = AIS_OK;
    }
    *out = &sd;
    return sd.status;
}

bool static_tmap(CUtensorMap* map, const void* base, uint64_t dim0, uint64_t dim1, uint64_t stride1_bytes, uint32_t box1) {
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {stride1_bytes};
    cuuint32_t box[2] = {64, box1};
    cuuint32_t estr[2] = {1, 1};
    return g_sencode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

extern "C" int ais_logprob_train_static(const ais_shape* shape, const void* H, const void* W, const int32_t* tokens,
                                        const uint8_t* mask, float* lp_train, float* lse_train, uint32_t* dev_status,
                                        void* stream) {
    if (!shape || !H || !W || !tokens || !mask || !lp_train) return AIS_ERR_NULL;
    if (shape->T < 0 || shape->d <= 0 || shape->V <= 0) return AIS_ERR_SHAPE;
    if (shape->d % 64 != 0 || shape->V % 8 != 0 || shape->ldh < shape->d || shape->ldw < shape->d) return AIS_ERR_SHAPE;
    if (shape->ldh % 8 != 0 || shape->ldw % 8 != 0) return AIS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(H) | reinterpret_cast<uintptr_t>(W)) % 16 != 0) return AIS_ERR_ALIGN;
    if (shape->T > AIS_STATIC_MAX_ROWS) return AIS_ERR_LIMIT;       // the fixed scratch holds no more rows
    StaticDev* sd = nullptr;
    const int st = static_setup(&sd);
    if (st != AIS_OK) return st;
    if (shape->T == 0) return AIS_OK;

    const int n_col_tiles = (shape->V + kBN - 1) / kBN;
    const int nsplit = n_col_tiles < kStaticNsplit ? n_col_tiles : kStaticNsplit;
    LmheadArgs a;
    memset(&a, 0, sizeof(a));
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
    a.part_m = sd->partials;
    a.part_s = sd->partials + static_cast<size_t>(kStaticParts) * kStaticLd;
    a.part_z = sd->partials + static_cast<size_t>(2 * kStaticParts) * kStaticLd;
    a.part_ld = kStaticLd;
    a.status = dev_status;
    CUtensorMap tmA, tmB;
    if (!static_tmap(&tmA, H, static_cast<uint64_t>(shape->d), static_cast<uint64_t>(shape->T), shape->ldh * 2, kBM) ||
        !static_tmap(&tmB, W, static_cast<uint64_t>(shape->d), static_cast<uint64_t>(shape->V), shape->ldw * 2, kBN))
        return AIS_ERR_DEVICE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int units = a.n_row_tiles * nsplit;
    // Every slot of the scratch that the merge reads (parts 0 .. 2*nsplit-1, rows 0 .. T-1) is written by the
    // pass just before it, so nothing left over from an earlier call is ever read and nothing needs zeroing.
    if (launch_lmhead(kFwdBf16, tmA, tmB, tmA, tmB, a, units < sd->num_sms ? units : sd->num_sms, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (launch_combine(a.part_m, a.part_s, a.part_z, nsplit * 2, kStaticLd, mask, shape->T, lp_train, lse_train, dev_status, s) !=
        cudaSuccess)
        return AIS_ERR_DEVICE;
    return AIS_OK;
}

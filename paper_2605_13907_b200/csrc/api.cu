// C ABI of the library: argument validation, workspace carving, tensor-map construction and the order
// in which the kernels of each entry point are enqueued.  Declarations and contracts live in include/ais.h.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "../../include/ais.h"
#include "host_setup.cuh"
#include "lmhead.cuh"
#include "stream_kernels.cuh"

namespace ais {

namespace {
constexpr int kMaxDevices = 64;
struct DeviceInfo {
    bool ready = false;      // set-up succeeded on this device
    bool wrong_arch = false; // not an sm_100 device: remembered, every later call fails at once
    int num_sms = 0;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_mutex;
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::atomic<long long> g_wait_cycles{0};
}  // namespace

int64_t wait_cycles() { return g_wait_cycles.load(); }

// Per-device set-up, done once per device with that device current: checks the architecture, raises the kernels'
// dynamic shared-memory limit and resolves the driver's tensor-map encoder.  Only the architecture check is
// remembered as a failure; any other failed step (a CUDA call that could not get resources, say) is tried again
// by the next call.
int device_setup(int* num_sms) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AIS_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo& info = g_dev[dev];
    if (info.wrong_arch) return AIS_ERR_DEVICE;
    if (!info.ready) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return AIS_ERR_DEVICE;
        if (prop.major != 10) {
            info.wrong_arch = true;
            return AIS_ERR_DEVICE;
        }
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
                qres != cudaDriverEntryPointSuccess || !fn)
                return AIS_ERR_DEVICE;
            g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
        }
        if (lmhead_prepare() != cudaSuccess || stream_prepare() != cudaSuccess) return AIS_ERR_DEVICE;
        info.num_sms = prop.multiProcessorCount;
        info.ready = true;
    }
    if (num_sms) *num_sms = info.num_sms;
    return AIS_OK;
}

// 2-D row-major tensor map: dim0 is the contiguous axis.
bool make_tmap(CUtensorMap* map, CUtensorMapDataType dtype, const void* base, uint64_t dim0, uint64_t dim1,
               uint64_t stride1_bytes, uint32_t box0, uint32_t box1, CUtensorMapSwizzle swz) {
    if (!g_encode) return false;
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {stride1_bytes};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, dtype, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace ais

namespace {

using namespace ais;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_shape(const ais_shape* s) {
    if (!s) return AIS_ERR_NULL;
    if (s->T < 0 || s->T > (int64_t(1) << 31) - 1024) return AIS_ERR_SHAPE;
    if (s->d <= 0 || s->V <= 0 || s->P <= 0 || s->G <= 0) return AIS_ERR_SHAPE;
    if (s->d % 128 != 0 || s->V % 8 != 0) return AIS_ERR_SHAPE;
    if (s->fp8_block != 0 && s->fp8_block != 32 && s->fp8_block != 64 && s->fp8_block != 128 && s->fp8_block != AIS_FP8_MX32 &&
        s->fp8_block != AIS_FP4_MX32)
        return AIS_ERR_SHAPE;
    if (s->fp8_block == AIS_FP4_MX32 && (s->d % 256 != 0 || s->ldh % 32 != 0 || s->ldw % 32 != 0)) return AIS_ERR_SHAPE;
    if (s->fp8_block > 0 && s->d % s->fp8_block != 0) return AIS_ERR_SHAPE;
    if (s->w_layout != AIS_W_VD && s->w_layout != AIS_W_DV) return AIS_ERR_SHAPE;
    if (s->w_layout == AIS_W_DV) {
        // [d, V] head: the block-scaled variants and the per-tensor variant take the [V, d] layout only
        if (s->fp8_block != 32 && s->fp8_block != 64 && s->fp8_block != 128) return AIS_ERR_SHAPE;
        if (s->ldh < s->d || s->ldw < s->V) return AIS_ERR_SHAPE;
        if (s->ldh % 16 != 0 || s->ldw % 8 != 0) return AIS_ERR_ALIGN;
    } else {
        if (s->ldh < s->d || s->ldw < s->d) return AIS_ERR_SHAPE;
        if (s->ldh % 16 != 0 || s->ldw % 16 != 0) return AIS_ERR_ALIGN;
    }
    if (static_cast<int64_t>(s->P) * s->G > (1 << 24)) return AIS_ERR_SHAPE;
    if (s->P_total != 0 && (s->P_total < s->P || static_cast<int64_t>(s->P_total) * s->G > (int64_t(1) << 30))) return AIS_ERR_SHAPE;
    return AIS_OK;
}

int check_params(const ais_params* p) {
    if (!p) return AIS_ERR_NULL;
    if (!(p->C >= 1.0f) || !(p->delta > 0.f) || !(p->gamma > 0.f) || !(p->eps >= 0.f) || !(p->clip_eps >= 0.f) ||
        !(p->beta_var >= 0.f))
        return AIS_ERR_PARAM;
    if (!isnan(p->alpha_override) && !(p->alpha_override >= 0.f && p->alpha_override <= 1.f)) return AIS_ERR_PARAM;
    if (p->vocab_chunk < 0 || !(p->beta_kl >= 0.f)) return AIS_ERR_PARAM;
    return AIS_OK;
}

int pick_nsplit(const ais_shape* s, const ais_params* p) {
    const int n_col_tiles = (s->V + kBN - 1) / kBN;
    int nsplit = 4;
    if (p->vocab_chunk > 0) nsplit = (s->V + p->vocab_chunk - 1) / p->vocab_chunk;
    if (nsplit > 64) nsplit = 64;
    if (nsplit > n_col_tiles) nsplit = n_col_tiles;
    if (nsplit < 1) nsplit = 1;
    return nsplit;
}

struct Layout {
    int64_t t_ld;          // padded length of per-row vectors
    int nsplit, nparts;
    size_t off_part_m, off_part_s, off_part_z;   // forward partials
    size_t off_diag;                              // reduction partials (doubles)
    size_t off_flags;                             // one byte per 128-row tile: anything to compute there?
    size_t off_pace;                              // ring of counters that keeps the CTAs of a tensor-core launch in step
    size_t off_coef, off_nseq;                    // backward: c_t, valid rows per sequence
    size_t off_seqw;                              // sequence-level variant: log weight per sequence
    size_t off_u;                                 // backward scratch
    int64_t ldU;
    size_t fixed_bytes;                           // everything but the scratch rows
    size_t u_row_bytes;
};

Layout make_layout(const ais_shape* s, const ais_params* p) {
    Layout L;
    L.t_ld = static_cast<int64_t>(align_up(static_cast<size_t>(s->T > 0 ? s->T : 1), 64));
    L.nsplit = pick_nsplit(s, p);
    L.nparts = L.nsplit * 2;
    size_t off = 0;
    const size_t part_bytes = align_up(static_cast<size_t>(L.nparts) * L.t_ld * sizeof(float), 256);
    L.off_part_m = off; off += part_bytes;
    L.off_part_s = off; off += part_bytes;
    L.off_part_z = off; off += part_bytes;
    L.off_flags = off;  off += align_up(static_cast<size_t>(L.t_ld / kBM + 2), 256);
    L.off_pace = off;   off += align_up(static_cast<size_t>(kPaceRing) * sizeof(uint32_t), 256);
    L.off_diag = off;   off += align_up(static_cast<size_t>(kDiagBlocks) * kNumMoments * sizeof(double), 256);
    L.off_coef = off;   off += align_up(static_cast<size_t>(L.t_ld) * sizeof(float), 256);
    L.off_nseq = off;   off += align_up(static_cast<size_t>(s->P) * s->G * sizeof(int32_t), 256);
    L.off_seqw = off;   off += align_up(static_cast<size_t>(s->P) * s->G * sizeof(float), 256);
    L.off_u = off;
    L.ldU = static_cast<int64_t>(align_up(static_cast<size_t>(s->V), 64));
    L.fixed_bytes = off;
    L.u_row_bytes = static_cast<size_t>(L.ldU) * sizeof(__nv_bfloat16);
    return L;
}

constexpr int64_t kBwdRowsRecommended = 2 * 148 * kBM;

// Zeroes the pacing ring and points the launch at it.  tiles_per_unit = the largest number of column tiles a unit of
// the launch walks; a launch of a single wave has nobody to keep in step with over time and runs without pacing only
// when it has a single CTA.
cudaError_t arm_pace(LmheadArgs& a, uint8_t* ws, const Layout& L, int tiles_per_unit, int ctas, cudaStream_t s) {
    a.pace = nullptr;
    a.pace_per_unit = 0;
    if (ctas < 2) return cudaSuccess;
    const int64_t fills = static_cast<int64_t>(tiles_per_unit) * a.ksteps;
    a.pace = reinterpret_cast<uint32_t*>(ws + L.off_pace);
    a.pace_per_unit = static_cast<int32_t>((fills + kPaceFills - 1) / kPaceFills);
    return cudaMemsetAsync(a.pace, 0, static_cast<size_t>(kPaceRing) * sizeof(uint32_t), s);
}

}  // namespace

extern "C" {

int ais_version(void) { return AIS_VERSION; }

int ais_set_wait_cycles(int64_t cycles) {
    if (cycles < 0) return AIS_ERR_PARAM;
    g_wait_cycles.store(cycles);
    return AIS_OK;
}

const char* ais_strerror(int status) {
    switch (status) {
        case AIS_OK: return "ok";
        case AIS_ERR_NULL: return "a required pointer is NULL";
        case AIS_ERR_SHAPE: return "invalid or inconsistent shape";
        case AIS_ERR_ALIGN: return "pointer or leading dimension not aligned as required";
        case AIS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case AIS_ERR_DEVICE: return "no sm_100 device, or a CUDA call failed";
        case AIS_ERR_PARAM: return "hyper-parameter out of range";
        case AIS_ERR_LIMIT: return "size beyond a fixed limit of this entry point";
        default: return "unknown status";
    }
}

void ais_default_params(ais_params* p) {
    if (!p) return;
    p->C = 5.0f;
    p->delta = 0.02f;
    p->gamma = 1.2f;
    p->eps = 1e-6f;
    p->beta_var = 1.0f;
    p->clip_eps = 0.2f;
    p->alpha_override = NAN;
    p->adv_std_norm = 0;
    p->vocab_chunk = 0;
    p->beta_kl = 0.0f;
    p->seq_level_weights = 0;
}

size_t ais_workspace_min_bytes(const ais_shape* shape, const ais_params* params) {
    if (check_shape(shape) != AIS_OK || check_params(params) != AIS_OK) return 0;
    const Layout L = make_layout(shape, params);
    return L.fixed_bytes + static_cast<size_t>(kBM) * L.u_row_bytes;
}

size_t ais_workspace_bytes(const ais_shape* shape, const ais_params* params) {
    if (check_shape(shape) != AIS_OK || check_params(params) != AIS_OK) return 0;
    const Layout L = make_layout(shape, params);
    int64_t rows = static_cast<int64_t>(align_up(static_cast<size_t>(shape->T > 0 ? shape->T : 1), kBM));
    if (rows > kBwdRowsRecommended) rows = kBwdRowsRecommended;
    return L.fixed_bytes + static_cast<size_t>(rows) * L.u_row_bytes;
}

int ais_quantize_fp8(const void* x, int64_t rows, int64_t cols, int64_t ld, int block, uint8_t* codes, int64_t ldq,
                     float* scales, int64_t lds, void* stream) {
    if (!x || !codes || !scales) return AIS_ERR_NULL;
    if (rows < 0 || cols < 0 || (block != 32 && block != 64 && block != 128)) return AIS_ERR_SHAPE;
    if (cols % block != 0 || ld < cols || ldq < cols || lds < rows) return AIS_ERR_SHAPE;
    if (ld % 8 != 0 || ldq % 8 != 0 || !aligned(x, 16) || !aligned(codes, 8) || !aligned(scales, 4)) return AIS_ERR_ALIGN;
    if (rows > (int64_t(1) << 31) - 1024) return AIS_ERR_SHAPE;
    int st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    return launch_quantize(x, rows, cols, ld, block, codes, ldq, scales, lds, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AIS_OK
               : AIS_ERR_DEVICE;
}

int ais_quantize_fp8_cols(const void* x, int64_t rows, int64_t cols, int64_t ld, int block, uint8_t* codes, int64_t ldq,
                          float* scales, int64_t lds, void* stream) {
    if (!x || !codes || !scales) return AIS_ERR_NULL;
    if (rows < 0 || cols < 0 || (block != 32 && block != 64 && block != 128)) return AIS_ERR_SHAPE;
    if (rows % 128 != 0 || cols % 8 != 0 || ld < cols || ldq < rows || lds < cols) return AIS_ERR_SHAPE;
    if (ld % 8 != 0 || ldq % 16 != 0 || !aligned(x, 16) || !aligned(codes, 16) || !aligned(scales, 4)) return AIS_ERR_ALIGN;
    if (cols > (int64_t(1) << 31) - 1024 || rows > (int64_t(1) << 24)) return AIS_ERR_SHAPE;
    int st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    return launch_quantize_cols(x, rows, cols, ld, block, codes, ldq, scales, lds, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AIS_OK
               : AIS_ERR_DEVICE;
}

int ais_quantize_fp8_tensor(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq, float* scale,
                            void* stream) {
    if (!x || !codes || !scale) return AIS_ERR_NULL;
    if (rows < 0 || cols < 0 || cols % 8 != 0 || ld < cols || ldq < cols) return AIS_ERR_SHAPE;
    if (ld % 8 != 0 || ldq % 8 != 0 || !aligned(x, 16) || !aligned(codes, 8) || !aligned(scale, 4)) return AIS_ERR_ALIGN;
    if (rows > (int64_t(1) << 31) - 1024) return AIS_ERR_SHAPE;
    int st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    return launch_quantize_tensor(x, rows, cols, ld, codes, ldq, scale, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AIS_OK
               : AIS_ERR_DEVICE;
}

size_t ais_mx_scale_bytes(int64_t rows, int64_t cols) {
    if (rows < 0 || cols <= 0 || cols % 128 != 0) return 0;
    const int64_t chunks = (rows + 255) / 256 * 2;          // 128-row chunks, an even number of them
    return static_cast<size_t>(chunks > 0 ? chunks : 2) * static_cast<size_t>(cols / 128) * 512;
}

int ais_quantize_mxfp8(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq, uint8_t* scales,
                       void* stream) {
    if (!x || !codes || !scales) return AIS_ERR_NULL;
    if (rows < 0 || cols <= 0 || cols % 128 != 0 || ld < cols || ldq < cols) return AIS_ERR_SHAPE;
    if (ld % 8 != 0 || ldq % 8 != 0 || !aligned(x, 16) || !aligned(codes, 8) || !aligned(scales, 16)) return AIS_ERR_ALIGN;
    if (rows > (int64_t(1) << 31) - 1024) return AIS_ERR_SHAPE;
    int st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    return launch_quantize_mx(x, rows, cols, ld, codes, ldq, scales, ais_mx_scale_bytes(rows, cols), false,
                              static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AIS_OK
               : AIS_ERR_DEVICE;
}

int ais_quantize_mxfp4(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq, uint8_t* scales,
                       void* stream) {
    if (!x || !codes || !scales) return AIS_ERR_NULL;
    if (rows < 0 || cols <= 0 || cols % 128 != 0 || ld < cols || ldq < cols / 2) return AIS_ERR_SHAPE;
    if (ld % 8 != 0 || ldq % 4 != 0 || !aligned(x, 16) || !aligned(codes, 4) || !aligned(scales, 16)) return AIS_ERR_ALIGN;
    if (rows > (int64_t(1) << 31) - 1024) return AIS_ERR_SHAPE;
    int st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    return launch_quantize_mx(x, rows, cols, ld, codes, ldq, scales, ais_mx_scale_bytes(rows, cols), true,
                              static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AIS_OK
               : AIS_ERR_DEVICE;
}

int ais_logprob_fwd(const ais_shape* shape, const ais_params* params, const void* H, const void* W, const uint8_t* qH,
                    const void* sH_, int64_t ldsH, const uint8_t* qW, const void* sW_, int64_t ldsW, const int32_t* tokens,
                    const uint8_t* mask, float* lp_train, float* lse_train, float* lp_roll, float* lse_roll,
                    uint32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream) {
    int st = check_shape(shape);
    if (st != AIS_OK) return st;
    st = check_params(params);
    if (st != AIS_OK) return st;
    if (!tokens || !mask) return AIS_ERR_NULL;
    const float* sH = static_cast<const float*>(sH_);
    const float* sW = static_cast<const float*>(sW_);
    const bool do_train = lp_train != nullptr, do_roll = lp_roll != nullptr;
    if (do_train && (!H || !W)) return AIS_ERR_NULL;
    if (do_roll && (!qH || !sH || !qW || !sW)) return AIS_ERR_NULL;
    if (do_train && (!aligned(H, 16) || !aligned(W, 16))) return AIS_ERR_ALIGN;
    const bool per_tensor = shape->fp8_block == 0;
    const bool fp4 = shape->fp8_block == AIS_FP4_MX32;
    const bool mx = shape->fp8_block == AIS_FP8_MX32 || fp4;
    if (do_roll) {
        if (!aligned(qH, 16) || !aligned(qW, 16) || !aligned(sH, 4) || !aligned(sW, 4)) return AIS_ERR_ALIGN;
        if (mx && (!aligned(sH, 16) || !aligned(sW, 16))) return AIS_ERR_ALIGN;
        if (!per_tensor && !mx) {
            if (!aligned(sH, 16) || !aligned(sW, 16)) return AIS_ERR_ALIGN;
            if (ldsH < shape->T || ldsW < shape->V) return AIS_ERR_SHAPE;
            if (ldsH % 4 != 0 || ldsW % 4 != 0) return AIS_ERR_ALIGN;
        }
    }
    const Layout L = make_layout(shape, params);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < L.off_diag) return AIS_ERR_WORKSPACE;
    int num_sms = 0;
    st = device_setup(&num_sms);
    if (st != AIS_OK) return st;
    if (shape->T == 0 || (!do_train && !do_roll)) return AIS_OK;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    LmheadArgs a;
    memset(&a, 0, sizeof(a));
    a.wait_cycles = wait_cycles();
    a.rows = shape->T;
    a.row0 = 0;
    a.n_row_tiles = static_cast<int32_t>((shape->T + kBM - 1) / kBM);
    a.ncols = shape->V;
    a.n_col_tiles = (shape->V + kBN - 1) / kBN;
    a.nsplit = L.nsplit;
    a.sgroups = (per_tensor || mx) ? 1 : 128 / shape->fp8_block;
    a.tokens = tokens;
    a.mask = mask;
    a.part_m = reinterpret_cast<float*>(ws + L.off_part_m);
    a.part_s = reinterpret_cast<float*>(ws + L.off_part_s);
    a.part_z = reinterpret_cast<float*>(ws + L.off_part_z);
    a.part_ld = L.t_ld;
    a.status = dev_status;
    // row tiles without a single valid row are skipped by the tensor-core passes
    a.tile_active = ws + L.off_flags;
    if (launch_tile_flags_mask(mask, shape->T, ws + L.off_flags, s) != cudaSuccess) return AIS_ERR_DEVICE;
    const int units = a.n_row_tiles * a.nsplit;
    const int ctas = units < num_sms ? units : num_sms;
    const uint64_t T = static_cast<uint64_t>(shape->T), V = static_cast<uint64_t>(shape->V), d = static_cast<uint64_t>(shape->d);

    CUtensorMap tmA, tmB, tmSA, tmSB;
    const bool dv = shape->w_layout == AIS_W_DV;
    if (do_train) {
        // W [V, d]: K-major boxes of 64 hidden units x 256 vocabulary rows.  W [d, V]: the vocabulary is the contiguous
        // axis, boxes of 64 vocabulary columns x 64 hidden units (four of them per stage)
        if (!make_tmap(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, H, d, T, shape->ldh * 2, 64, kBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !(dv ? make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, V, d, shape->ldw * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)
                 : make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, d, V, shape->ldw * 2, 64, kBN, CU_TENSOR_MAP_SWIZZLE_128B)))
            return AIS_ERR_DEVICE;
        a.ksteps = shape->d / 64;
        if (arm_pace(a, ws, L, (a.n_col_tiles + a.nsplit - 1) / a.nsplit, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_lmhead(dv ? kFwdBf16Dv : kFwdBf16, tmA, tmB, tmA, tmB, a, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_combine(a.part_m, a.part_s, a.part_z, L.nparts, L.t_ld, mask, shape->T, lp_train, lse_train, dev_status, s) !=
            cudaSuccess)
            return AIS_ERR_DEVICE;
    }
    if (do_roll && mx) {
        // power-of-two scales per 32 elements: the block-scaled MMA applies them, the contraction stays in tensor memory
        // FP4 codes are two per byte: the maps see d / 2 bytes per row with half the row stride
        const uint64_t kb = fp4 ? d / 2 : d;
        if (!make_tmap(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, qH, kb, T, fp4 ? shape->ldh / 2 : shape->ldh, 128, kBM,
                       CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, qW, kb, V, fp4 ? shape->ldw / 2 : shape->ldw, 128, kBN,
                       CU_TENSOR_MAP_SWIZZLE_128B))
            return AIS_ERR_DEVICE;
        a.ksteps = static_cast<int32_t>(kb / 128);
        a.sf_a = static_cast<const uint8_t*>(sH_);
        a.sf_b = static_cast<const uint8_t*>(sW_);
        a.nk4 = shape->d / 128;
        if (arm_pace(a, ws, L, (a.n_col_tiles + a.nsplit - 1) / a.nsplit, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_lmhead(fp4 ? kFwdMx4 : kFwdMx, tmA, tmB, tmA, tmB, a, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_combine(a.part_m, a.part_s, a.part_z, L.nparts, L.t_ld, mask, shape->T, lp_roll, lse_roll, dev_status, s) !=
            cudaSuccess)
            return AIS_ERR_DEVICE;
    } else if (do_roll && per_tensor) {
        // one scale per tensor: the whole contraction accumulates in tensor memory, the scales meet in the epilogue
        if (!make_tmap(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, qH, d, T, shape->ldh, 128, kBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, qW, d, V, shape->ldw, 128, kBN, CU_TENSOR_MAP_SWIZZLE_128B))
            return AIS_ERR_DEVICE;
        a.ksteps = shape->d / 128;
        a.scale_a = sH;
        a.scale_b = sW;
        if (arm_pace(a, ws, L, (a.n_col_tiles + a.nsplit - 1) / a.nsplit, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_lmhead(kFwdFp8T, tmA, tmB, tmA, tmB, a, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_combine(a.part_m, a.part_s, a.part_z, L.nparts, L.t_ld, mask, shape->T, lp_roll, lse_roll, dev_status, s) !=
            cudaSuccess)
            return AIS_ERR_DEVICE;
    } else if (do_roll) {
        const uint64_t nkb = d / shape->fp8_block;
        if (!make_tmap(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, qH, d, T, shape->ldh, 128, kBM, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, qW, d, V, dv ? d : shape->ldw, 128, kBN, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap(&tmSA, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sH, T, nkb, ldsH * 4, kBM, a.sgroups, CU_TENSOR_MAP_SWIZZLE_NONE) ||
            !make_tmap(&tmSB, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sW, V, nkb, ldsW * 4, kBN, a.sgroups, CU_TENSOR_MAP_SWIZZLE_NONE))
            return AIS_ERR_DEVICE;
        a.ksteps = shape->d / 128;
        if (arm_pace(a, ws, L, (a.n_col_tiles + a.nsplit - 1) / a.nsplit, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_lmhead(kFwdFp8, tmA, tmB, tmSA, tmSB, a, ctas, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_combine(a.part_m, a.part_s, a.part_z, L.nparts, L.t_ld, mask, shape->T, lp_roll, lse_roll, dev_status, s) !=
            cudaSuccess)
            return AIS_ERR_DEVICE;
    }
    return AIS_OK;
}

int ais_diagnostics(const ais_shape* shape, const ais_params* params, const float* lp_train, const float* lp_roll,
                    const uint8_t* mask, const int32_t* seq_offsets, const float* rewards, float* adv, int32_t* n_valid_seq,
                    float* rho, float* w_tilde, ais_diag* diag, void* workspace, size_t workspace_bytes, void* stream) {
    int st = check_shape(shape);
    if (st != AIS_OK) return st;
    st = check_params(params);
    if (st != AIS_OK) return st;
    if (!lp_train || !lp_roll || !mask || !seq_offsets || !rewards || !adv || !w_tilde || !diag) return AIS_ERR_NULL;
    if (!aligned(diag, 8)) return AIS_ERR_ALIGN;
    const Layout L = make_layout(shape, params);
    const bool seq_level = params->seq_level_weights != 0;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < (seq_level ? L.off_u : L.off_coef)) return AIS_ERR_WORKSPACE;
    st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int S = shape->P * shape->G;
    if (launch_advantages(rewards, S, shape->G, params->adv_std_norm, params->eps, adv, n_valid_seq, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (launch_diag(lp_train, lp_roll, mask, seq_offsets, adv, shape->T, S, *params, reinterpret_cast<double*>(ws + L.off_diag),
                    n_valid_seq, seq_level ? reinterpret_cast<float*>(ws + L.off_seqw) : nullptr, rho, w_tilde, diag, s) !=
        cudaSuccess)
        return AIS_ERR_DEVICE;
    return AIS_OK;
}

int ais_diag_moments(const ais_shape* shape, const ais_params* params, const float* lp_train, const float* lp_roll,
                     const uint8_t* mask, const int32_t* seq_offsets, const float* rewards, float* adv, int32_t* n_valid_seq,
                     double* moments, float* seq_logw, void* workspace, size_t workspace_bytes, void* stream) {
    int st = check_shape(shape);
    if (st != AIS_OK) return st;
    st = check_params(params);
    if (st != AIS_OK) return st;
    if (!lp_train || !lp_roll || !mask || !seq_offsets || !rewards || !adv || !moments) return AIS_ERR_NULL;
    if (params->seq_level_weights != 0 && !seq_logw) return AIS_ERR_NULL;
    if (!aligned(moments, 8)) return AIS_ERR_ALIGN;
    const Layout L = make_layout(shape, params);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < L.off_coef) return AIS_ERR_WORKSPACE;
    st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int S = shape->P * shape->G;
    if (launch_advantages(rewards, S, shape->G, params->adv_std_norm, params->eps, adv, n_valid_seq, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (launch_moments(lp_train, lp_roll, mask, seq_offsets, adv, shape->T, S, *params, reinterpret_cast<double*>(ws + L.off_diag),
                       n_valid_seq, params->seq_level_weights != 0 ? seq_logw : nullptr, moments, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    return AIS_OK;
}

int ais_diag_finalize(const ais_shape* shape, const ais_params* params, const double* moments, const float* lp_train,
                      const float* lp_roll, const uint8_t* mask, float* rho, float* w_tilde, ais_diag* diag,
                      const int32_t* seq_offsets, const float* seq_logw, void* stream) {
    int st = check_shape(shape);
    if (st != AIS_OK) return st;
    st = check_params(params);
    if (st != AIS_OK) return st;
    if (!moments || !lp_train || !lp_roll || !mask || !w_tilde || !diag) return AIS_ERR_NULL;
    const bool seq_level = params->seq_level_weights != 0;
    if (seq_level && (!seq_offsets || !seq_logw)) return AIS_ERR_NULL;
    if (!aligned(moments, 8) || !aligned(diag, 8)) return AIS_ERR_ALIGN;
    st = device_setup(nullptr);
    if (st != AIS_OK) return st;
    if (launch_finalize(moments, lp_train, lp_roll, mask, shape->T, *params, rho, w_tilde, diag, seq_offsets,
                        shape->P * shape->G, seq_level ? seq_logw : nullptr, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return AIS_ERR_DEVICE;
    return AIS_OK;
}

int ais_loss_bwd(const ais_shape* shape, const ais_params* params, const void* H, const void* W, const int32_t* tokens,
                 const uint8_t* mask, const int32_t* seq_offsets, const float* lse_train, const float* lp_train,
                 const float* lp_old, const float* lp_ref, const float* adv, const float* w_tilde, void* dH, float* loss,
                 ais_diag* diag, float* dW, int64_t lddw, int dw_accumulate,
                 uint32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream) {
    int st = check_shape(shape);
    if (st != AIS_OK) return st;
    st = check_params(params);
    if (st != AIS_OK) return st;
    if (!H || !W || !tokens || !mask || !seq_offsets || !lse_train || !lp_train || !adv || !w_tilde || !dH) return AIS_ERR_NULL;
    if (!aligned(H, 16) || !aligned(W, 16) || !aligned(dH, 16)) return AIS_ERR_ALIGN;
    if (dW && (!aligned(dW, 16) || lddw % 4 != 0)) return AIS_ERR_ALIGN;
    if (dW && lddw < (shape->w_layout == AIS_W_DV ? shape->V : shape->d)) return AIS_ERR_SHAPE;
    const Layout L = make_layout(shape, params);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < L.fixed_bytes + static_cast<size_t>(kBM) * L.u_row_bytes)
        return AIS_ERR_WORKSPACE;
    int num_sms = 0;
    st = device_setup(&num_sms);
    if (st != AIS_OK) return st;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int S = shape->P * shape->G;
    float* coef = reinterpret_cast<float*>(ws + L.off_coef);
    int32_t* nseq = reinterpret_cast<int32_t*>(ws + L.off_nseq);
    if (launch_seq_counts(mask, seq_offsets, S, nseq, s) != cudaSuccess) return AIS_ERR_DEVICE;
    const int P_norm = shape->P_total > 0 ? shape->P_total : shape->P;
    if (launch_loss_coef(lp_train, lp_old, lp_ref, params->beta_kl, mask, seq_offsets, adv, w_tilde, nseq, shape->T, S, P_norm * shape->G, params->clip_eps,
                         reinterpret_cast<double*>(ws + L.off_diag), coef, loss, diag, lse_train, s) != cudaSuccess)
        return AIS_ERR_DEVICE;
    if (shape->T == 0) return AIS_OK;
    // row tiles whose gradient factors are all zero (masked rows, zero advantage) are skipped by the recompute and dH passes
    if (launch_tile_flags_coef(coef, shape->T, ws + L.off_flags, s) != cudaSuccess) return AIS_ERR_DEVICE;

    // rows of scratch the workspace can hold (whole row tiles)
    int64_t blk_rows = static_cast<int64_t>((workspace_bytes - L.fixed_bytes) / L.u_row_bytes) / kBM * kBM;
    const int64_t t_pad = static_cast<int64_t>(align_up(static_cast<size_t>(shape->T), kBM));
    if (blk_rows > t_pad) blk_rows = t_pad;
    __nv_bfloat16* U = reinterpret_cast<__nv_bfloat16*>(ws + L.off_u);
    const uint64_t V = static_cast<uint64_t>(shape->V), d = static_cast<uint64_t>(shape->d);

    // tmW_k: W for the recompute pass (contraction over d), tmW_n: W for the dH pass (contraction over V).  With W [V, d]
    // the first is K-major (boxes of 64 hidden units x 256 vocabulary rows) and the second MN-major (64 x 64 boxes);
    // with W [d, V] it is the other way round (64 x 64 boxes of vocabulary columns x hidden units; boxes of 64 vocabulary
    // columns x 256 hidden units).
    const bool dv = shape->w_layout == AIS_W_DV;
    CUtensorMap tmW_k, tmW_n, tmU;
    if (!(dv ? make_tmap(&tmW_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, V, d, shape->ldw * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)
             : make_tmap(&tmW_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, d, V, shape->ldw * 2, 64, kBN, CU_TENSOR_MAP_SWIZZLE_128B)) ||
        !(dv ? make_tmap(&tmW_n, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, V, d, shape->ldw * 2, 64, kBN, CU_TENSOR_MAP_SWIZZLE_128B)
             : make_tmap(&tmW_n, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, W, d, V, shape->ldw * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) ||
        !make_tmap(&tmU, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, U, V, static_cast<uint64_t>(blk_rows), L.ldU * 2, 64, kBM,
                   CU_TENSOR_MAP_SWIZZLE_128B))
        return AIS_ERR_DEVICE;

    for (int64_t r0 = 0; r0 < shape->T; r0 += blk_rows) {
        const int64_t rows = (shape->T - r0) < blk_rows ? (shape->T - r0) : blk_rows;
        CUtensorMap tmH;
        const __nv_bfloat16* Hc = static_cast<const __nv_bfloat16*>(H) + r0 * shape->ldh;
        if (!make_tmap(&tmH, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Hc, d, static_cast<uint64_t>(rows), shape->ldh * 2, 64, kBM,
                       CU_TENSOR_MAP_SWIZZLE_128B))
            return AIS_ERR_DEVICE;
        LmheadArgs a;
        memset(&a, 0, sizeof(a));
        a.wait_cycles = wait_cycles();
        a.rows = rows;
        a.row0 = r0;
        a.n_row_tiles = static_cast<int32_t>((rows + kBM - 1) / kBM);
        a.tokens = tokens;
        a.mask = mask;
        a.lse = lse_train;
        a.U = U;
        a.ldU = L.ldU;
        a.coef = coef;
        a.dH = static_cast<__nv_bfloat16*>(dH);
        a.lddh = shape->ldh;
        a.status = dev_status;
        a.tile_active = ws + L.off_flags;
        a.sgroups = 1;
        // recompute softmax - onehot into the scratch
        a.ncols = shape->V;
        a.n_col_tiles = (shape->V + kBN - 1) / kBN;
        a.nsplit = L.nsplit;
        a.ksteps = shape->d / 64;
        int units = a.n_row_tiles * a.nsplit;
        if (arm_pace(a, ws, L, (a.n_col_tiles + a.nsplit - 1) / a.nsplit, units < num_sms ? units : num_sms, s) != cudaSuccess)
            return AIS_ERR_DEVICE;
        if (launch_lmhead(dv ? kBwdPDv : kBwdP, tmH, tmW_k, tmH, tmW_k, a, units < num_sms ? units : num_sms, s) != cudaSuccess)
            return AIS_ERR_DEVICE;
        // dH = c (.) (U W)
        a.ncols = shape->d;
        a.n_col_tiles = (shape->d + kBN - 1) / kBN;
        a.n_row_tiles = static_cast<int32_t>((rows + kDhRows - 1) / kDhRows);
        a.nsplit = 1;
        a.ksteps = (shape->V + 63) / 64;
        units = a.n_row_tiles * a.n_col_tiles;
        if (arm_pace(a, ws, L, 1, units < num_sms ? units : num_sms, s) != cudaSuccess) return AIS_ERR_DEVICE;
        if (launch_lmhead(dv ? kBwdDhDv : kBwdDh, tmU, tmW_n, tmU, tmW_n, a, units < num_sms ? units : num_sms, s) != cudaSuccess)
            return AIS_ERR_DEVICE;
        if (dW) {
            // dW (+)= U^T H over the rows of this pass: both operands are read with the rows as contraction axis;
            // the maps end at `rows`, so rows the scratch still holds from an earlier pass read as zeros
            CUtensorMap tmU_t, tmH_t;
            if (!make_tmap(&tmU_t, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, U, V, static_cast<uint64_t>(rows), L.ldU * 2, 64, 64,
                           CU_TENSOR_MAP_SWIZZLE_128B) ||
                !make_tmap(&tmH_t, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Hc, d, static_cast<uint64_t>(rows), shape->ldh * 2, 64, 64,
                           CU_TENSOR_MAP_SWIZZLE_128B))
                return AIS_ERR_DEVICE;
            // output in W's layout: [V, d] = U^T H, or [d, V] = H^T U with the two operands changing places
            const int out_rows = dv ? shape->d : shape->V, out_cols = dv ? shape->V : shape->d;
            LmheadArgs w = a;
            w.rows = out_rows;
            w.row0 = 0;
            w.n_row_tiles = static_cast<int32_t>((out_rows + kDhRows - 1) / kDhRows);
            w.ncols = out_cols;
            w.n_col_tiles = (out_cols + kBN - 1) / kBN;
            w.ksteps = static_cast<int32_t>((rows + 63) / 64);
            w.dW = dW;
            w.lddw = lddw;
            w.dw_accumulate = (dw_accumulate || r0 > 0) ? 1 : 0;
            units = w.n_row_tiles * w.n_col_tiles;
            const CUtensorMap& tmRow = dv ? tmH_t : tmU_t;
            const CUtensorMap& tmCol = dv ? tmU_t : tmH_t;
            if (arm_pace(w, ws, L, 1, units < num_sms ? units : num_sms, s) != cudaSuccess) return AIS_ERR_DEVICE;
            if (launch_lmhead(kBwdDw, tmRow, tmCol, tmRow, tmCol, w, units < num_sms ? units : num_sms, s) != cudaSuccess)
                return AIS_ERR_DEVICE;
        }
    }
    return AIS_OK;
}

}  // extern "C"

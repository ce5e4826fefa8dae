// Host-callable launchers of the streaming (HBM / latency bound) kernels: FP8 block quantisation, merge of
// the per-split log-sum-exp partials, segmented and whole-batch reductions, per-token loss coefficients.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ais.h"

namespace ais {

constexpr int kDiagBlocks = 592;      // fixed grid of the batch reductions (keeps the summation order fixed)
constexpr int kDiagThreads = 256;
constexpr int kNumMoments = 12;

// Raises the dynamic shared-memory limit of the kernels here that need it (once per device).
cudaError_t stream_prepare();

cudaError_t launch_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int block, uint8_t* codes,
                            int64_t ldq, float* scales, int64_t lds, cudaStream_t stream);

// Blocks running down the columns of x [K, ld] (K a multiple of 128): codes transposed [N, ldq], scales [K / block, lds].
cudaError_t launch_quantize_cols(const void* x, int64_t K, int64_t N, int64_t ld, int block, uint8_t* codes, int64_t ldq,
                                 float* scales, int64_t lds, cudaStream_t stream);

// Microscaling: E8M0 scale per 32 elements, packed in 512-byte chunks of 128 rows x 4 blocks; `scale_bytes` is the
// size of the whole packed array (rows padded to a multiple of 256), filled with the neutral code first.
cudaError_t launch_quantize_mx(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq,
                               uint8_t* scales, size_t scale_bytes, bool fp4 /* E2M1 elements, two per byte */,
                               cudaStream_t stream);

// One scale for the whole matrix (written to *scale on the device), then the codes.
cudaError_t launch_quantize_tensor(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, int64_t ldq,
                                   float* scale, cudaStream_t stream);

// lp[t] = z_y - lse, lse[t] from nparts partial triples laid out [nparts][part_ld].
cudaError_t launch_combine(const float* part_m, const float* part_s, const float* part_z, int nparts, int64_t part_ld,
                           const uint8_t* mask, int64_t T, float* lp, float* lse, uint32_t* status, cudaStream_t stream);

// flags[i] = 1 when rows 128 i .. 128 i + 127 contain a row with mask != 0 (resp. a non-zero gradient factor).
cudaError_t launch_tile_flags_mask(const uint8_t* mask, int64_t T, uint8_t* flags, cudaStream_t stream);
cudaError_t launch_tile_flags_coef(const float* coef, int64_t T, uint8_t* flags, cudaStream_t stream);

// n_valid_seq[s] = valid rows of sequence s.
cudaError_t launch_seq_counts(const uint8_t* mask, const int32_t* seq_offsets, int S, int32_t* n_valid_seq, cudaStream_t stream);
// adv[s] (group-relative advantages); zero_counts [S] (may be NULL) is cleared for the moments kernel to count into.
cudaError_t launch_advantages(const float* rewards, int S, int G, int adv_std_norm, float eps, float* adv, int32_t* zero_counts,
                              cudaStream_t stream);

// n_valid_seq (may be NULL) must have been cleared: the moments kernel adds every sequence's valid rows to it.
cudaError_t launch_diag(const float* lp_train, const float* lp_roll, const uint8_t* mask, const int32_t* seq_offsets,
                        const float* adv, int64_t T, int S, const ais_params& p, double* partials /*[kDiagBlocks][kNumMoments]*/,
                        int32_t* n_valid_seq, float* seq_logw /* [S] scratch: non-NULL selects sequence-level weights */,
                        float* rho, float* w_tilde, ais_diag* diag, cudaStream_t stream);

// The two halves of launch_diag: partial moments summed into `moments` [kNumMoments], and everything that follows
// from a (possibly all-reduced) moment vector.
cudaError_t launch_moments(const float* lp_train, const float* lp_roll, const uint8_t* mask, const int32_t* seq_offsets,
                           const float* adv, int64_t T, int S, const ais_params& p, double* partials, int32_t* n_valid_seq,
                           float* seq_logw, double* moments, cudaStream_t stream);
cudaError_t launch_finalize(const double* moments, const float* lp_train, const float* lp_roll, const uint8_t* mask, int64_t T,
                            const ais_params& p, float* rho, float* w_tilde, ais_diag* diag, const int32_t* seq_offsets, int S,
                            const float* seq_logw, cudaStream_t stream);

// coef[t] and the loss; n_valid_seq must already hold the valid counts.  S_norm is the number of sequences the
// objective averages over (all data-parallel ranks together).  Rows whose lse is not finite (marked by the forward
// pass) contribute nothing.
cudaError_t launch_loss_coef(const float* lp_train, const float* lp_old, const float* lp_ref, float beta_kl, const uint8_t* mask,
                             const int32_t* seq_offsets,
                             const float* adv, const float* w_tilde, const int32_t* n_valid_seq, int64_t T, int S, int S_norm,
                             float clip_eps, double* partials /*[kDiagBlocks][2]*/, float* coef, float* loss, ais_diag* diag,
                             const float* lse, cudaStream_t stream);

}  // namespace ais

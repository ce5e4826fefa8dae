/*
 * ais.h - C ABI of the B200 (sm_100a) library for the LM-head step of an AIS-GRPO update.
 *
 * The path: hidden states H [T,d] meet the LM head W twice - once with bf16 operands (the trainer's
 * policy pi_train) and once with block-scaled FP8-E4M3 operands (the rollout policy pi_rollout) - each
 * pass fused with a streaming log-sum-exp over the vocabulary and a pick of the sampled token's logit,
 * so the [T,V] logits never reach global memory.  The two log-probability vectors feed the three AIS
 * diagnostics and the per-batch mixing coefficient alpha (Section 3.1, Algorithm 1); the last call gives
 * the AIS-GRPO surrogate loss (Section 3.2, Eq. ais-grpo, without the KL term) and its gradient with
 * respect to H.
 *
 * Conventions
 * -----------
 *  - Every data pointer is a DEVICE pointer owned by the caller unless it says "host".  The library
 *    never allocates or frees device memory; scratch comes from the caller's `workspace`
 *    (256-byte aligned, at least ais_workspace_bytes() bytes).  The one exception is
 *    ais_logprob_train_static at the end of this header: it takes no workspace, keeps its scratch in an
 *    array inside the library image, has its own (looser) size and alignment rules, a row limit, and
 *    calls to it must not overlap on the GPU.
 *  - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it; they never
 *    synchronise the device.  Calls on one stream are ordered; calls that share a workspace must not
 *    overlap on the GPU.
 *  - Return value: AIS_OK or a negative AIS_ERR_* code.  On a host-detected error nothing has been
 *    enqueued.  Conditions only the device can see (token id outside [0,V), a bounded wait that ran
 *    out, no valid token) are OR-ed into the caller's `dev_status` word / ais_diag.status_flags and the
 *    affected outputs take their documented neutral values; the kernels never trap.
 *  - Layouts: H is row-major [T, ldh] bf16 (ldh >= d).  W is row-major [V, ldw] bf16, one row per
 *    vocabulary entry (the layout of a torch lm_head.weight), so logits are z = H W^T; with
 *    ais_shape.w_layout = AIS_W_DV it is row-major [d, ldw] instead (z = H W).
 *    FP8 codes keep the layout of their source matrix ([rows, cols] uint8).  Scales are "block-major":
 *    scales[kb * ld_scales + row] is the scale of block kb (elements kb*B .. kb*B+B-1 along d) of `row`.
 *  - Rows with mask[t] == 0 yield lp = 0, lse = 0, rho = 1, w_tilde = 1 and a zero row of dH.
 *  - Alignment: H, W, codes, scales and dH 16 bytes, the workspace 256 bytes; ldh and ldw multiples
 *    of 16; d a multiple of 128 (one shared-memory stage is 128 bytes of FP8 along d) and of
 *    fp8_block; V a multiple of 8; ld of scale arrays a multiple of 4.
 */
#ifndef AIS_H_
#define AIS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AIS_VERSION 110

/* status codes */
#define AIS_OK                 0
#define AIS_ERR_NULL          -1   /* a required pointer is NULL                            */
#define AIS_ERR_SHAPE         -2   /* a size is out of range or inconsistent (S != P*G ...) */
#define AIS_ERR_ALIGN         -3   /* pointer or leading dimension not aligned as required  */
#define AIS_ERR_WORKSPACE     -4   /* workspace missing, misaligned or too small            */
#define AIS_ERR_DEVICE        -5   /* current device is not sm_100, or a CUDA call failed   */
#define AIS_ERR_PARAM         -6   /* a hyper-parameter is out of range                     */
#define AIS_ERR_LIMIT         -7   /* size beyond a fixed limit of an entry point           */

/* bits of a device status word / ais_diag.status_flags */
#define AIS_FLAG_EMPTY        1u   /* no valid token in the batch: alpha = 0, loss = 0      */
#define AIS_FLAG_TOKEN_RANGE  2u   /* a valid row has a token id outside [0, V): lp = 0     */
#define AIS_FLAG_NONFINITE    4u   /* a log-prob of a valid row is not finite (a NaN or an infinity
                                      in its hidden state or in W): that row gets lp = 0 and
                                      lse = NaN, which makes ais_loss_bwd leave it out of the loss
                                      and give it a zero row of dH; the batch statistics count it
                                      as a row with lp_train = lp_roll                        */
#define AIS_FLAG_TIMEOUT      8u   /* a bounded device-side wait ran out; outputs undefined */

#define AIS_W_VD 0                /* ais_shape.w_layout: W is row-major [V, ldw], one row per vocabulary entry     */
#define AIS_W_DV 1                /* ais_shape.w_layout: W is row-major [d, ldw], one row per hidden unit          */

#define AIS_FP8_MX32 (-32)        /* ais_shape.fp8_block: microscaling FP8, E8M0 scale per 32 elements */
#define AIS_FP4_MX32 (-4)         /* ais_shape.fp8_block: microscaling FP4 (E2M1 elements), E8M0 scale per 32    */

typedef struct ais_shape {
    int64_t T;            /* token rows                                                      */
    int32_t d;            /* hidden size                                                     */
    int32_t V;            /* vocabulary size                                                 */
    int32_t P;            /* prompts in the batch                                            */
    int32_t G;            /* responses per prompt; sequence s belongs to prompt s / G        */
    int32_t fp8_block;    /* elements along d sharing one FP8 scale: 32, 64 or 128;
                             0 = one scale per tensor (ais_quantize_fp8_tensor);
                             AIS_FP8_MX32 = power-of-two scale per 32 (ais_quantize_mxfp8);
                             AIS_FP4_MX32 = the same with 4-bit elements (ais_quantize_mxfp4)*/
    int32_t P_total;      /* prompts over all data-parallel ranks (loss normaliser); 0 = P    */
    int32_t w_layout;     /* AIS_W_VD (0): W [V, ldw] as a torch lm_head.weight; AIS_W_DV: W [d, ldw], the form in
                             which the paper writes the head.  Both give the same log-probs bit for bit (the
                             tensor cores read either storage order; nothing is transposed in memory).  AIS_W_DV:
                             ldw >= V, a multiple of 8; V a multiple of 8; fp8_block 32, 64 or 128 only; W's codes
                             are [V, d] with row stride d (ais_quantize_fp8_cols); dW comes out [d, lddw].  */
    int64_t ldh;          /* row stride of H (and of its codes) in elements                  */
    int64_t ldw;          /* row stride of W in elements (AIS_W_VD: also of its codes)       */
} ais_shape;

/* Hyper-parameters (Algorithm 1 'Require' line; Appendix 'AIS hyperparameters'; PPO clipping of the
 * hyper-parameter table).  The paper prints no value for beta_var; 1 is this library's default. */
typedef struct ais_params {
    float C;              /* truncation of the importance ratio, >= 1          (5)           */
    float delta;          /* saturation threshold of the divergence gate, > 0  (0.02)        */
    float gamma;          /* tolerance of the variance-amplification ratio, >0 (1.2)         */
    float eps;            /* stabiliser in that ratio                          (1e-6)        */
    float beta_var;       /* weight of the variance penalty                    (1.0)         */
    float clip_eps;       /* PPO clip range of rho_on                          (0.2)         */
    float alpha_override; /* NaN: adaptive alpha.  Otherwise alpha is forced to this value in
                             [0,1] (0 = plain GRPO, 1 = truncated importance sampling); the
                             diagnostics are still reported.                                 */
    int32_t adv_std_norm; /* 0: A = r - mean(group) (the paper's form).  1: also divide by
                             (population std of the group + eps).                            */
    int32_t vocab_chunk;  /* 0: library default.  Otherwise the vocabulary is streamed in
                             independent chunks of about this many columns whose partial
                             (max, sum-exp, target logit) triples are merged afterwards.     */
    float beta_kl;        /* weight of the KL(pi_theta || pi_ref) term of the objective (0: no term;
                             the paper gives no value).  Used only when ais_loss_bwd gets lp_ref.  */
    int32_t seq_level_weights; /* 0: per-token truncated ratios min(rho_t, C) (Algorithm 1).  1: every valid row of a
                             sequence carries the sequence's weight min(prod_t rho_t, C) of Eq. is-weight /
                             Eq. ais-components instead; d_bar and rho stay per token.                  */
} ais_params;

/* Everything the reductions produce; lives in DEVICE memory, the caller copies it back.
 * The three variances (cv2, std_A, std_Aw) are E[x^2] - E[x]^2 in fp64 over sums that are accurate relative to the
 * spread of the data (short runs are summed about one of their own values), so weights that differ by 1e-4 of their
 * size still give the right variance; what is left is the rounding of the fp64 additions, and a variance below
 * 2^-44 of the mean square is reported as exactly 0.
 * status_flags carries AIS_FLAG_EMPTY for N = 0 and AIS_FLAG_TIMEOUT if a bounded wait of the moments kernel ran out. */
typedef struct ais_diag {
    double n_valid;       /* N = number of rows with mask 1                                  */
    double mean_w;        /* mean of w_bar = min(rho, C)                                     */
    double cv2;           /* squared coefficient of variation of w_bar (population moments)  */
    double ess;           /* (sum w_bar)^2 / sum w_bar^2                                     */
    double ess_ratio;     /* ess / N                                                         */
    double alpha_ess;     /* (1 + cv2)^(-1/2)                         Eq. alpha-ess          */
    double d_bar;         /* mean |lp_train - lp_roll|                Eq. discrepancy        */
    double alpha_mis;     /* min(1, d_bar / delta)                    Eq. alpha-mis          */
    double std_A;         /* population std of the token-level advantage                     */
    double std_Aw;        /* population std of A * w_bar                                     */
    double delta_sigma;   /* std_Aw / (std_A + eps)                                          */
    double alpha_var;     /* max(0, (delta_sigma - gamma) / gamma)    Eq. alpha-var          */
    double alpha_adaptive;/* clip(alpha_ess - beta_var alpha_var, 0, 1) * alpha_mis          */
    double alpha;         /* the coefficient in force (alpha_adaptive or the override)       */
    double loss;          /* written by ais_loss_bwd                                         */
    double kl_k1;         /* monitor: mean(lp_roll - lp_train)                               */
    double mean_abs_dp;   /* monitor: mean |exp(lp_train) - exp(lp_roll)|                    */
    double kl_ref;        /* written by ais_loss_bwd: value of the KL term (without beta_kl) */
    uint32_t status_flags;
    uint32_t reserved;
} ais_diag;

int ais_version(void);
const char* ais_strerror(int status);

/* Bound of every device-side wait of the tensor-core passes, in SM clock ticks (a producer waiting for a free stage,
 * the MMA issuer for operands, an epilogue warp for an accumulator).  0 restores the default of 4e9 ticks, about two
 * seconds; a wait that runs out ends its kernel in an orderly way (copies in flight are awaited, tensor memory is
 * freed) with AIS_FLAG_TIMEOUT in the call's dev_status and undefined outputs, and the next call works normally.
 * Process-wide, read by every later call; meant for watchdog tuning and for testing the time-out path (a bound of a
 * few ticks makes the first wait of a pass run out).  Returns AIS_ERR_PARAM for a negative value. */
int ais_set_wait_cycles(int64_t cycles);

/* Fills *p with the defaults listed above (alpha_override = NaN). `p` is a host pointer. */
void ais_default_params(ais_params* p);

/* Recommended workspace size in bytes for all entry points on this shape (host pointers in).
 * Any 256-byte aligned workspace of at least ais_workspace_min_bytes() is accepted; a larger one
 * lets ais_loss_bwd process more rows per pass.  Returns 0 for an invalid shape. */
size_t ais_workspace_bytes(const ais_shape* shape, const ais_params* params);
size_t ais_workspace_min_bytes(const ais_shape* shape, const ais_params* params);

/*
 * FP8-E4M3 block quantisation (Section 2.1, quantisation equation, with the E4M3 grid in place of the
 * integer grid): for every run of `block` consecutive elements of a row,
 *     s = fl32(max|x| / 448)   (s = 1 for an all-zero block)
 *     q = E4M3_rne_saturating( fl32(fl32(x) / s) )
 * x       [rows, ld]  bf16, row-major
 * codes   [rows, ldq] uint8                       (written)
 * scales  [cols/block, lds] float, block-major    (written; lds >= rows)
 * cols must be a multiple of `block`; block is 32, 64 or 128.  Used for H (rows = T) and W (rows = V).
 */
int ais_quantize_fp8(const void* x, int64_t rows, int64_t cols, int64_t ld, int block,
                     uint8_t* codes, int64_t ldq, float* scales, int64_t lds, void* stream);

/*
 * The same quantisation for a matrix whose blocks run down its columns: an LM head stored [d, V] (AIS_W_DV).
 * x       [rows, ld] bf16, row-major; rows (= d) a multiple of 128; cols (= V) a multiple of 8
 * codes   [cols, ldq] uint8: TRANSPOSED, codes[v, k] belongs to x[k, v]; ldq >= rows, a multiple of 16   (written)
 * scales  [rows/block, lds] float: scales[kb, v] is the scale of x[kb*block .. kb*block+block-1, v]       (written)
 * The result is element for element what ais_quantize_fp8 gives for the transposed matrix.
 */
int ais_quantize_fp8_cols(const void* x, int64_t rows, int64_t cols, int64_t ld, int block,
                          uint8_t* codes, int64_t ldq, float* scales, int64_t lds, void* stream);

/*
 * Per-tensor dynamic scaling, the setting of the paper's own rollouts (Appendix "FP8 rollout"): one scale
 * s = fl32(max|x| / 448) for the whole matrix (s = 1 for an all-zero matrix), same code rule.  `scale` is one
 * float on the device (written).  With shape->fp8_block == 0, ais_logprob_fwd takes such codes and reads sH / sW
 * as pointers to one float each (ldsH / ldsW are ignored); the contraction then accumulates entirely in tensor
 * memory and the two scales are applied once per logit.
 */
int ais_quantize_fp8_tensor(const void* x, int64_t rows, int64_t cols, int64_t ld,
                            uint8_t* codes, int64_t ldq, float* scale, void* stream);

/*
 * Microscaling FP8 (the lower-precision block-scaled formats that the paper's Limitations section names for future
 * rollouts; format rule from the published OCP microscaling specification): every 32 consecutive elements of a row
 * share the power-of-two scale 2^X, X = floor(log2 max|x|) - 8, stored as the byte X + 127 (clamped to 0..254; 127
 * for an all-zero block), and the elements are E4M3_rne_saturating(x / 2^X).
 * x       [rows, ld]  bf16, row-major; cols a multiple of 128
 * codes   [rows, ldq] uint8                                   (written)
 * scales  ais_mx_scale_bytes(rows, cols) bytes, 16-byte aligned (written): chunks of 128 rows x 4 blocks, chunk
 *         (r / 128, kb / 4) at ((r / 256) * (cols / 128) + kb / 4) * 1024 + ((r % 256) / 128) * 512, byte
 *         (r % 32) * 16 + ((r % 128) / 32) * 4 + kb % 4 inside it -- the order in which the block-scaled
 *         tensor-core instruction reads one K-step's scales; rows are padded to a multiple of 256 with the
 *         neutral byte 127.
 * With shape->fp8_block == AIS_FP8_MX32, ais_logprob_fwd takes such codes, reads sH / sW as these packed arrays
 * (ldsH / ldsW are ignored) and lets tcgen05's block-scaled MMA apply the scales, so the whole contraction stays in
 * tensor memory.
 */
size_t ais_mx_scale_bytes(int64_t rows, int64_t cols);
int ais_quantize_mxfp8(const void* x, int64_t rows, int64_t cols, int64_t ld,
                       uint8_t* codes, int64_t ldq, uint8_t* scales, void* stream);

/*
 * Microscaling FP4, the FP4 rollouts the paper names as future work (Introduction, Limitations): the same rule with
 * E2M1 elements (magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6; X = floor(log2 max|x|) - 2; scaled magnitudes in (6, 8)
 * saturate).  codes [rows, ldq] bytes hold two 4-bit codes each, the element with the lower index in the low nibble
 * (ldq >= cols / 2, a multiple of 4); scales as for ais_quantize_mxfp8.  With shape->fp8_block == AIS_FP4_MX32
 * (d a multiple of 256, ldh and ldw multiples of 32; the codes' row strides are ldh / 2 and ldw / 2 bytes)
 * ais_logprob_fwd runs the rollout pass on tcgen05's packed-FP4 block-scaled MMA.
 */
int ais_quantize_mxfp4(const void* x, int64_t rows, int64_t cols, int64_t ld,
                       uint8_t* codes, int64_t ldq, uint8_t* scales, void* stream);

/*
 * Trainer and rollout log-probabilities (Algorithm 1: "full-precision log-probs" and the sampler's
 * log-probs entering rho_rt; Eq. logit-mismatch).  For every row t with mask[t] = 1:
 *     lse_train[t] = log sum_v exp(z[t,v]),  z = H W^T  (bf16 operands, fp32 accumulation)
 *     lp_train[t]  = z[t, tokens[t]] - lse_train[t]
 *     lp_roll[t], lse_roll[t]: the same with z^[t,v] = sum_kb sH[kb,t] sW[kb,v] sum_{k in kb} qH[t,k] qW[v,k]
 * The train pass is skipped when lp_train is NULL; the rollout pass when lp_roll is NULL.
 * lse_train / lse_roll may be NULL when not wanted (lse_train is needed later by ais_loss_bwd).
 * sH is [d/B, ldsH] and sW is [d/B, ldsW] floats (block-major, as ais_quantize_fp8 writes them); one float each with
 * fp8_block == 0; packed scale bytes with fp8_block == AIS_FP8_MX32.
 * tokens [T] int32, mask [T] uint8, dev_status: one uint32 on the device (OR-ed into; may be NULL).
 */
int ais_logprob_fwd(const ais_shape* shape, const ais_params* params,
                    const void* H, const void* W,
                    const uint8_t* qH, const void* sH, int64_t ldsH,
                    const uint8_t* qW, const void* sW, int64_t ldsW,
                    const int32_t* tokens, const uint8_t* mask,
                    float* lp_train, float* lse_train, float* lp_roll, float* lse_roll,
                    uint32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Ratios, advantages, diagnostics, alpha and the rectification weight (Algorithm 1, "Adaptive
 * Coefficient Estimation" and "Advantage Rectification"; Eqs. grpo_adv, alpha-ess, discrepancy,
 * alpha-mis, alpha-var, alpha-final, adjusted-advantage).
 * seq_offsets [S+1] int32 row offsets of the S = P*G sequences (seq_offsets[S] == T), rewards [S].
 * Outputs: adv [S] (A_s), n_valid_seq [S] int32 (valid rows per sequence; may be NULL),
 * rho [T] = exp(lp_train - lp_roll) (may be NULL), w_tilde [T] = 1 + alpha (min(rho, C) - 1),
 * diag (one ais_diag on the device).  All moments are population moments over the valid rows.
 */
int ais_diagnostics(const ais_shape* shape, const ais_params* params,
                    const float* lp_train, const float* lp_roll, const uint8_t* mask,
                    const int32_t* seq_offsets, const float* rewards,
                    float* adv, int32_t* n_valid_seq, float* rho, float* w_tilde, ais_diag* diag,
                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same step in two halves, for data-parallel use (each rank holds whole prompts; alpha is one number
 * per global batch, Eq. alpha-final).  ais_diag_moments writes adv, n_valid_seq and this rank's AIS_NUM_MOMENTS
 * masked sums (double, on the device):
 *   0 N   1 sum w_bar   2 sum w_bar^2   3 sum |lp_train - lp_roll|   4 sum A   5 sum A^2   6 sum A w_bar
 *   7 sum (A w_bar)^2   8 sum (lp_roll - lp_train)   9 sum |exp(lp_train) - exp(lp_roll)|   10, 11 unused (zero)
 * The caller sums the vectors of all ranks (one all-reduce of 12 doubles) and hands the result to
 * ais_diag_finalize, which derives the diagnostics, alpha, rho and w_tilde from it.  With one rank the two
 * calls give bit-identical results to ais_diagnostics.
 */
#define AIS_NUM_MOMENTS 12
int ais_diag_moments(const ais_shape* shape, const ais_params* params,
                     const float* lp_train, const float* lp_roll, const uint8_t* mask,
                     const int32_t* seq_offsets, const float* rewards,
                     float* adv, int32_t* n_valid_seq, double* moments,
                     float* seq_logw /* [S], written when params->seq_level_weights; else may be NULL */,
                     void* workspace, size_t workspace_bytes, void* stream);
int ais_diag_finalize(const ais_shape* shape, const ais_params* params, const double* moments,
                      const float* lp_train, const float* lp_roll, const uint8_t* mask,
                      float* rho, float* w_tilde, ais_diag* diag,
                      const int32_t* seq_offsets, const float* seq_logw /* both read only with seq_level_weights */,
                      void* stream);

/*
 * AIS-GRPO loss and its gradient with respect to H (Eq. ais-grpo; the objective is maximised, so
 * loss = -J).  With rho_on = exp(lp_train - lp_old)
 * (lp_old == NULL means rho_on = 1) and n_s the valid rows of sequence s:
 *     loss  = - sum_s 1/(P G n_s) sum_{t in s, mask} w_tilde[t] min(rho_on A_s, clip(rho_on, 1 +- clip_eps) A_s)
 *     c_t   = mask[t] w_tilde[t] A_s rho_on [unclipped branch active] / (P G n_s)
 * (P is shape->P_total when that is set, so that the losses of all data-parallel ranks add up to the global one)
 *     dH[t,:] = c_t (softmax(z[t,:]) - onehot(tokens[t])) W
 * With lp_ref != NULL and beta_kl != 0 the KL term is included.  The paper does not name its estimator; this
 * library uses the one of the GRPO paper it builds on, per token kl_t = r - log r - 1 with
 * r = exp(lp_ref[t] - lp_train[t]) (lp_ref: log-probs of the sampled tokens under the reference policy, e.g.
 * from another ais_logprob_fwd call with the reference LM head):
 *     loss += beta_kl sum_s 1/(P G n_s) sum_t kl_t ,   c_t -= mask[t] beta_kl (1 - r) / (P G n_s)
 * The softmax is recomputed from H, W and lse_train; w_tilde, A, lp_old and lp_ref are constants.
 * dH [T, ldh] bf16 (written, zero rows where mask = 0), loss: one float on the device (may be NULL),
 * diag: if not NULL its `loss` and `kl_ref` fields are written too.
 * dW (may be NULL): gradient with respect to the LM head in W's layout, [V, lddw] fp32 ([d, lddw] with AIS_W_DV),
 *     dW[v,:] = sum_t c_t (softmax(z[t,:])[v] - [v == tokens[t]]) H[t,:]
 * overwritten when dw_accumulate == 0, added to otherwise (micro-batch accumulation); costs one more
 * T x d x V tensor-core pass over the scratch that dH uses.
 */
int ais_loss_bwd(const ais_shape* shape, const ais_params* params,
                 const void* H, const void* W, const int32_t* tokens, const uint8_t* mask,
                 const int32_t* seq_offsets, const float* lse_train, const float* lp_train,
                 const float* lp_old, const float* lp_ref, const float* adv, const float* w_tilde,
                 void* dH, float* loss, ais_diag* diag,
                 float* dW, int64_t lddw, int dw_accumulate,
                 uint32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Row compaction for batches whose valid rows are scattered (masked-diffusion log-probabilities: only the masked
 * positions of a response take part, Appendix "LLaDA Experiments").  The tensor-core passes work on tiles of 128
 * consecutive rows, so scattered invalid rows cost as much as valid ones; packing the valid rows first makes the
 * passes proportional to the number of valid rows.
 *   ais_compact_index : n_valid_seq [S] (valid rows per sequence), packed_offsets [S+1] (their exclusive scan: row
 *                       offsets of the packed batch) and row_index [>= N] (original row of packed row i, increasing
 *                       inside every sequence; N = packed_offsets[S]).
 *   ais_gather_rows   : dst[i,:] = src[row_index[i],:] for rows of row_bytes bytes (multiple of 16; strides in bytes).
 *   ais_scatter_rows  : the row_bytes of each of dst's dst_rows rows are zero-filled (padding between rows is left
 *                       alone), then dst[row_index[i],:] = src[i,:].
 *   ais_gather_words / ais_scatter_words : the same for vectors of 32-bit elements (tokens, log-probs, rho, w_tilde);
 *                       the scatter first fills dst[0 .. dst_rows) with fill_bits (0 for log-probs, the bits of 1.0f
 *                       for rho and w_tilde).
 * The caller runs the path on the packed batch (T = N, mask all ones, seq_offsets = packed_offsets) and scatters
 * what it needs back.  N is data dependent: the caller either knows it (it made the mask) or reads packed_offsets[S].
 */
int ais_compact_index(const uint8_t* mask, const int32_t* seq_offsets, int32_t S, int32_t* n_valid_seq,
                      int32_t* packed_offsets, int32_t* row_index, void* stream);
int ais_gather_rows(const void* src, int64_t src_stride_bytes, const int32_t* row_index, int64_t n, int64_t row_bytes,
                    void* dst, int64_t dst_stride_bytes, void* stream);
int ais_scatter_rows(const void* src, int64_t src_stride_bytes, const int32_t* row_index, int64_t n, int64_t row_bytes,
                     void* dst, int64_t dst_stride_bytes, int64_t dst_rows, void* stream);
int ais_gather_words(const void* src, const int32_t* row_index, int64_t n, void* dst, void* stream);
int ais_scatter_words(const void* src, const int32_t* row_index, int64_t n, void* dst, int64_t dst_rows,
                      uint32_t fill_bits, void* stream);

/*
 * Trainer log-probabilities for callers that cannot hand over a workspace (the paper has no counterpart;
 * this is a packaging variant of the trainer pass of ais_logprob_fwd, same kernels, same results).
 *
 * Who needs it: code that runs where device memory cannot be obtained at call time - a plug-in or
 * callback that receives only its input and output buffers, a process whose HBM has been handed in
 * full to another pool (a serving engine's KV cache, a training framework's caching allocator), or a
 * latency-critical loop that must avoid cudaMalloc because it stalls the whole device.  Such a caller
 * has nowhere to get the workspace that ais_logprob_fwd asks for.
 *
 * The partial (max, sum-exp, target-logit) triples of the vocabulary ranges are kept in a fixed array of
 * 3 x 8 x AIS_STATIC_MAX_ROWS floats (1.5 MiB) that is part of the library image; every GPU on which
 * the library is loaded holds it until the process exits.  The call allocates and frees nothing.
 *   - T must not exceed AIS_STATIC_MAX_ROWS; a larger T returns AIS_ERR_LIMIT and enqueues nothing.
 *   - shape->d must be a multiple of 64 and V of 8; P, G and fp8_block are not read.  The vocabulary
 *     is always streamed in 4 ranges.
 *   - The first call on each device resolves the array's device address and prepares the kernels; that is
 *     also the moment at which the CUDA runtime may load this part of the library onto the device, and the
 *     1.5 MiB array comes with it.  So the device does take that memory once, at the first call, not at a
 *     later one: make the first call at start-up, with the device current and before any stream capture
 *     begins.  If that first call fails for lack of resources it can simply be repeated; only a device of
 *     the wrong architecture is remembered as unusable.
 *   - All calls on a device share the one array, which keeps what the last call left in it.  Each call
 *     overwrites every slot it later reads, so nothing has to be cleared; but two calls that overlap on
 *     the GPU (different streams, no ordering between them) race on it and give undefined results.
 * Inputs and outputs as in ais_logprob_fwd: H [T, ldh] bf16, W [V, ldw] bf16, tokens [T], mask [T],
 * lp_train [T] (written), lse_train [T] (written, may be NULL), dev_status (OR-ed into, may be NULL).
 */
#define AIS_STATIC_MAX_ROWS 16384
int ais_logprob_train_static(const ais_shape* shape, const void* H, const void* W, const int32_t* tokens,
                             const uint8_t* mask, float* lp_train, float* lse_train, uint32_t* dev_status,
                             void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AIS_H_ */

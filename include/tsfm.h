/*
 * tsfm.h -- C ABI of the B200 (sm_100a) speculative decoder for continuous patch
 * autoregression.
 *
 * The library decodes a batch of univariate series patch by patch with a decoder-only
 * patch transformer ("target"), optionally accelerated by a cheap draft model under the
 * Gaussian speculative-decoding rule:
 *
 *   - patch-autoregressive decoding, T = ceil(H / P) patches per series   (paper Eq. 1)
 *   - Gaussian surrogate heads N(mu, sigma^2 I) with a supplied shared
 *     scale sigma, here called `tau`                                      (Sec. 3.1, Eq. 4)
 *   - acceptance statistic l_i = (1/d) log p(x_i)/q(x_i), accept with
 *     probability min{1, exp(l_i)}, evaluated in the log domain           (Sec. 3.2, Eq. 5)
 *   - mean proposals x_i = mu_q^(i), target-mean fallback, bonus patch    (Sec. 3.3, Eq. 6)
 *   - single causal verification pass over [h, x_1..x_K], read at the
 *     K+1 prefix boundaries; instance statistics frozen on the context    (Sec. 3.4)
 *   - one round = Algorithm 1 (appendix B), looped until T patches are committed.
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers on the current device; "host" pointers are
 *     ordinary host memory.  Nothing in this ABI is a torch type.
 *   - All work is enqueued on the stream given at creation (a cudaStream_t passed as void*,
 *     NULL = the legacy default stream).  Calls that return data to host memory (stats,
 *     traces) synchronise that stream before returning; the others are asynchronous.
 *   - Every function returns 0 on success or a negative TSFM_ERR_* code.  Nothing aborts,
 *     traps, or throws across this boundary.  Device-side waits are bounded; if one expires
 *     the call returns TSFM_ERR_TIMEOUT and the CUDA context stays usable.
 *   - There is no CPU fallback: on a machine without an sm_100 device every compute entry
 *     point returns TSFM_ERR_ARCH / TSFM_ERR_CUDA.
 */
#ifndef TSFM_H_
#define TSFM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TSFM_OK            0
#define TSFM_ERR_ARG      (-1)  /* null pointer, B < 1, K < 1, tau not finite or <= 0, H < 1           */
#define TSFM_ERR_SHAPE    (-2)  /* ctx_len % P != 0, fewer than 2 context patches, capacity exceeded
                                   (B, N, T or K beyond the handle's max_*), d_model % n_heads != 0,
                                   unsupported head size, bad weight blob                           */
#define TSFM_ERR_ARCH     (-3)  /* current device is not compute capability 10.x                   */
#define TSFM_ERR_CUDA     (-4)  /* a CUDA runtime/driver call failed (see tsfm_last_cuda_error)     */
#define TSFM_ERR_TIMEOUT  (-5)  /* a bounded device-side wait expired                               */
#define TSFM_ERR_INTERNAL (-6)

#define TSFM_F32   0            /* weights, activations and KV cache in fp32 (SIMT FMA path)        */
#define TSFM_BF16  1            /* bf16 weights / MMA operands / KV cache, fp32 accumulate+residual */

#define TSFM_DRAFT_SEPARATE   0 /* draft has its own weight blob                                    */
#define TSFM_DRAFT_LAYER_SKIP 1 /* draft = first draft.n_layers layers of the target + its final
                                   norm and head; draft_w must be NULL                              */

#define TSFM_GEMM_AUTO  0       /* bf16 contractions on tcgen05 tensor cores where shapes allow     */
#define TSFM_GEMM_SIMT  1       /* force the plain FMA kernels everywhere (differential reference)  */
#define TSFM_GEMM_WS    2       /* tsfm_gemm_bf16 only: the small-batch kernel that keeps its weight
                                   tile in shared memory (TSFM_ERR_SHAPE outside its domain: at most
                                   256 tokens, K a multiple of 64 up to 2048, grid within one wave);
                                   a decoder picks it by itself where it applies                   */

#define TSFM_EXEC_GRAPH   0       /* a forecast is one CUDA-graph launch: prologue, a device-side WHILE
                                   over the rounds, de-normalisation; no host round trip             */
#define TSFM_EXEC_STREAM  1       /* kernels are launched one by one and the host checks for completion
                                   after every round (reference behaviour; also used while profiling) */

#define TSFM_EXEC_NO_PDL  2       /* flag, may be OR-ed in: launch without programmatic dependent launch,
                                   i.e. every kernel starts only after its predecessor has finished   */

#define TSFM_EXEC_NO_COMPACT 4     /* flag, may be OR-ed in: every round runs its passes over all B series, finished
                                   or not (by default only the series that still have patches to commit take
                                   part: the batch desynchronises as per-series first rejections differ, the
                                   paper's "Batch Size" sensitivity paragraph); same results either way  */

#define TSFM_EXEC_CHECK_BOUNDS 8   /* flag, may be OR-ed in: bounds-checking mode.  Every device buffer of the handle
                                   gets guard bytes behind it, every (layer, series, head) block of the KV
                                   caches and every series' history one spare token that nothing may write;
                                   after each call a kernel inspects them all, and a damaged guard makes a
                                   call that reads its status (stats != NULL) return TSFM_ERR_INTERNAL with
                                   the buffer's name in tsfm_last_cuda_error().  Costs memory and a launch
                                   per call; for test runs                                               */

#define TSFM_MAX_K 32           /* hard upper bound on the block size K                             */

typedef struct tsfm_spec tsfm_spec;   /* opaque decoder handle */

/* Decoder-only pre-norm patch transformer: n_layers x {RMSNorm, RoPE causal attention with
 * n_heads heads, RMSNorm, GELU MLP d_model -> d_ff -> d_model}, linear patch embedding and
 * linear mean head.  d_model % n_heads == 0; head size d_model / n_heads in {32, 64, 128};
 * d_model and d_ff multiples of 64; patch_len a multiple of 16, at most 256. */
typedef struct {
  int32_t n_layers, d_model, n_heads, d_ff;
} tsfm_arch;

typedef struct {
  tsfm_arch target, draft;
  int32_t patch_len;            /* P: input and output patch length (one channel)               */
  int32_t dtype;                /* TSFM_F32 | TSFM_BF16                                          */
  int32_t draft_mode;           /* TSFM_DRAFT_*                                                  */
  int32_t max_batch;            /* capacity: series per call                                     */
  int32_t max_ctx_tokens;       /* capacity: context tokens N = ctx_len / P_in (>= 2 patches' worth) */
  int32_t max_horizon_patches;  /* capacity: T = ceil(H / P)                                     */
  int32_t max_K;                /* capacity: block size, <= TSFM_MAX_K                           */
  int32_t gemm_backend;         /* TSFM_GEMM_*                                                   */
  float   rms_eps;              /* RMSNorm epsilon (1e-6)                                        */
  float   norm_eps;             /* instance-norm variance epsilon (1e-5)                         */
  float   rope_base;            /* RoPE base (1e4)                                               */
  int32_t exec_mode;            /* TSFM_EXEC_GRAPH or TSFM_EXEC_STREAM, optionally | TSFM_EXEC_NO_PDL | TSFM_EXEC_NO_COMPACT */
  int32_t patch_in;             /* P_in: steps per INPUT token; 0 = patch_len (a token is a whole patch).
                                   Must divide patch_len.  With P_in < P (the point-token family of the
                                   paper's appendix B: P_in = 1, a horizon head of P steps) a committed
                                   patch is P / P_in tokens, the embedding is [d, P_in], and the target's
                                   prediction after prefix i is read at token N - 1 + i (P / P_in) of the
                                   verification pass (appendix B, "Per-Family Boundary Indexing")        */
  void   *stream;               /* cudaStream_t, borrowed for the handle's lifetime              */
} tsfm_cfg;

/* A weight blob in DEVICE memory, borrowed for the handle's lifetime (never copied, never
 * written).  Layout: a 256-byte header of int32 words
 *     [0] magic 0x4D465354 ("TSFM")  [1] version 1  [2] dtype  [3] n_layers  [4] d_model
 *     [5] n_heads  [6] d_ff  [7] patch_len  [8] patch_in (0 = patch_len)   (remaining words zero)
 * followed by the tensors, each starting on a 256-byte boundary, every linear stored
 * [out_features, in_features] row-major in `dtype`, gains in fp32, in this order:
 *     W_emb[d,P_in];  per layer: g1[d], Wq[d,d], Wk[d,d], Wv[d,d], Wo[d,d], g2[d],
 *     W1[d_ff,d], W2[d,d_ff];  g_f[d];  W_head[P,d].
 * tsfm_weights_bytes() gives the total size. */
typedef struct {
  const void *blob;             /* dev */
  size_t      bytes;
} tsfm_weights;

/* Counters of one forecast call (host memory).  "tested" counts proposals whose accept/reject
 * decision was taken (accepted ones plus the first rejected one of each round): accepted/tested
 * estimates the conditional acceptance rate of the capped-geometric law (Eq. 7). */
typedef struct {
  int64_t rounds;                       /* speculative rounds executed (max over series)        */
  int64_t proposals_drafted;            /* K per active series per round                        */
  int64_t proposals_tested;
  int64_t proposals_accepted;
  int64_t patches_committed;            /* after truncation to T; equals B * T on success       */
  int64_t near_margin_decisions;        /* tested decisions with |l_i - log u_i| < margin       */
  int64_t tested_by_pos[TSFM_MAX_K];
  int64_t accepted_by_pos[TSFM_MAX_K];
  int64_t L_hist[TSFM_MAX_K + 2];       /* untruncated round yield L = n_accept + 1, index L    */
  float   ms_total, ms_prefill, ms_draft, ms_verify, ms_accept;   /* CUDA-event times           */
  int32_t device_status;                /* 0, or the code a kernel's bounded wait reported      */
  int32_t reserved0;
} tsfm_stats;

/* Size in bytes of the weight blob of a model of this shape. Returns 0 on invalid arguments. */
size_t tsfm_weights_bytes(const tsfm_arch *arch, int32_t patch_len, int32_t dtype);

/* Byte offset of a tensor inside the blob; `layer` is ignored for W_emb (-1), g_f, W_head.
 * `name` is one of "W_emb","g1","Wq","Wk","Wv","Wo","g2","W1","W2","g_f","W_head".
 * Returns 0 on invalid arguments (no tensor lives at offset 0: the header does). */
size_t tsfm_weights_offset(const tsfm_arch *arch, int32_t patch_len, int32_t dtype,
                           int32_t layer, const char *name);

/* The same two queries for a model whose input tokens are patch_in steps long (0 = patch_len):
 * only W_emb [d, patch_in] differs.  Return 0 if patch_in does not divide patch_len. */
size_t tsfm_weights_bytes_io(const tsfm_arch *arch, int32_t patch_in, int32_t patch_len, int32_t dtype);
size_t tsfm_weights_offset_io(const tsfm_arch *arch, int32_t patch_in, int32_t patch_len, int32_t dtype,
                              int32_t layer, const char *name);

/* Create a decoder (Algorithm 1's inputs "target p, draft q").  Validates shapes and blob
 * headers, allocates both KV caches ([layer][series][head][token][d_head], capacity
 * max_ctx_tokens + (max_horizon_patches + max_K + 1) * (P / P_in) tokens per series), activation workspaces
 * and TMA descriptors.  target_w, cfg, out_h: host pointers to structs; blobs: dev.
 * draft_w may be NULL only with TSFM_DRAFT_LAYER_SKIP.  *out_h is owned by the caller and
 * released with tsfm_spec_destroy. */
int tsfm_spec_create(const tsfm_weights *target_w, const tsfm_weights *draft_w,
                     const tsfm_cfg *cfg, tsfm_spec **out_h);

/* Speculative forecast (Algorithm 1 looped; Sec. 3.1-3.4).
 *   series  dev  [B, ctx_len] fp32 row-major, raw (un-normalised) context values
 *   out     dev  [B, H] fp32 row-major, forecast in the series' own scale
 *   stats   host, nullable; when non-NULL the call synchronises the stream and fills it
 * ctx_len must be a multiple of P (hence of P_in) with at least 2 patches; T = ceil(H / P) patches are
 * committed per series, the last one truncated to H on output.  Each round drafts K patches
 * with the draft model, verifies them in one causal target pass, accepts left to right with
 * uniforms Philox4x32-10(key = seed, counter = (series, round, position, 0)), commits the
 * accepted proposals plus the target's correction or bonus patch, and rolls both KV caches
 * back to the committed length.  tau is the acceptance temperature (the paper's sigma). */
int tsfm_spec_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                       int32_t H, int32_t K, float tau, uint64_t seed,
                       float *out, tsfm_stats *stats);

/* The general form of the rule (Sec. 3.3 "Fallback Correction and Sampled Variants", Algorithm 1
 * with r > 0; component ablation of Table 2).  The deployed scheme is tsfm_spec_forecast: mean
 * proposals, r = 0, sigma_q = sigma_p = tau, 1/d tempering.
 *   sigma_q           draft surrogate scale of Eq. 5; 0 = same as tau (determinant term vanishes)
 *   fallback_noise    r >= 0: correction and bonus patches are mu_p + r eps
 *   sample_proposals  nonzero: x_i = mu_q^(i) + sigma_q eps, the draft continues from the sampled x_i
 *   no_tempering      nonzero: drop the 1/d factor of the statistic
 * eps are standard normals from the same Philox key: Box-Muller on the words of counter
 * (series, round, position, stream | element / 2), stream 0x10000000 for proposals and 0x20000000
 * for the fallback, cosine branch for even elements, sine for odd.  variant == NULL is the deployed
 * scheme. */
typedef struct {
  float   sigma_q;
  float   fallback_noise;
  int32_t sample_proposals;
  int32_t no_tempering;
} tsfm_variant;
int tsfm_spec_forecast_variant(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                               int32_t H, int32_t K, float tau, uint64_t seed,
                               const tsfm_variant *variant, float *out, tsfm_stats *stats);

/* Target-only decoding (Eq. 1): T sequential one-token target passes.  Same argument
 * meaning as above; only the timing fields, rounds (= T) and patches_committed of `stats`
 * are filled. */
int tsfm_target_only_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                              int32_t H, float *out, tsfm_stats *stats);

/* Draft-only decoding: the same loop as tsfm_target_only_forecast run with the draft model alone
 * (the third arm of the paper's matched three-way protocol, Sec. 4.1 "Evaluation Protocol").
 * Timing goes to ms_prefill / ms_draft. */
int tsfm_draft_only_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                             int32_t H, float *out, tsfm_stats *stats);

/* The two forecasts with HOST buffers: series host [B, ctx_len], out host [B, H] (pinned
 * memory makes the copies asynchronous; pageable memory works too).  The input is copied to
 * a device staging buffer owned by the handle, the forecast runs as above, the result is
 * copied back, and the stream is synchronised before returning. */
int tsfm_spec_forecast_host(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                            int32_t H, int32_t K, float tau, uint64_t seed,
                            float *out, tsfm_stats *stats);
int tsfm_target_only_forecast_host(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len,
                                   int32_t H, float *out, tsfm_stats *stats);

/* Per-round decisions of the last tsfm_spec_forecast on this handle, copied to HOST arrays
 * (any may be NULL).  R = rounds of that call, B and K as in that call.
 *   n_accept [R, B] int32: leading accepted proposals, or -1 if the series had finished
 *   ell      [R, B, K] fp32: l_i of Eq. 5 for every position (tested or not)
 *   log_u    [R, B, K] fp32: log of the uniform drawn for that position
 * *rounds receives R.  cap_rounds is the first dimension of the arrays the caller provided;
 * returns TSFM_ERR_ARG if it is smaller than R.  Synchronises the stream. */
int tsfm_spec_last_trace(tsfm_spec *h, int32_t cap_rounds, int32_t *rounds,
                         int32_t *n_accept, float *ell, float *log_u);

/* One fused accept step (Eq. 5 + first rejection + correction/bonus) on caller buffers, the
 * same kernel the round uses.  All pointers dev.
 *   x     [B, K, P]   proposals x_i            mu_q [B, K, P] draft means (may alias x)
 *   mu_p  [B, K+1, P] boundary predictions
 *   done  [B] int32   in/out: patches committed so far; series with done >= T are skipped
 *   commit[B, K+1, P] out: x_1..x_n then mu_p^(n+1)          n_accept [B] int32 out
 *   ell, log_u [B, K] out (nullable)
 * sigma_p, sigma_q: the two surrogate scales (equal in the deployed scheme); round_idx and
 * series0 enter the Philox counter; forced_u (dev [B, K], nullable) replaces the drawn
 * uniforms, for scripted tests. */
int tsfm_accept_round(void *stream, const float *x, const float *mu_q, const float *mu_p,
                      int32_t B, int32_t K, int32_t P, int32_t T, float sigma_p, float sigma_q,
                      uint64_t seed, int32_t round_idx, int32_t series0, const float *forced_u,
                      int32_t *done, float *commit, int32_t *n_accept, float *ell, float *log_u);

/* Full causal forward of one of the handle's models over fresh sequences (positions
 * 0..n-1), for numerics checks: tokens dev [B, n, P_in] fp32 (already normalised), out dev
 * [B, n, P] fp32 = next-patch mean at every position.  which: 0 target, 1 draft.
 * n <= max_ctx_tokens (TSFM_ERR_SHAPE beyond it).  Overwrites the KV cache; synchronises the stream. */
int tsfm_model_forward(tsfm_spec *h, int32_t which, const float *tokens, int32_t B, int32_t n,
                       float *out);

/* C[M, N] = A[M, Kd] * W[N, Kd]^T with bf16 operands and fp32 accumulation, through the
 * tensor-memory kernel (backend TSFM_GEMM_AUTO), the FMA kernel (TSFM_GEMM_SIMT) or the small-batch
 * kernel (TSFM_GEMM_WS); for differential tests of the contraction.  A, W dev bf16 row-major; C dev fp32 row-major. */
int tsfm_gemm_bf16(void *stream, const void *A, const void *W, float *C,
                   int32_t M, int32_t N, int32_t Kd, int32_t backend);

/* The same contraction as tsfm_gemm_bf16 (tensor-core kernel, K split across CTAs with fp32
 * atomic accumulation) for callers that must not allocate device memory.  The paper has no
 * counterpart to this entry point; it exists for the library's users.  Who they are: a
 * serving loop that checks the contraction while forecasts are in flight on other streams
 * (cudaMalloc and cudaFree synchronise the whole device and would stall those forecasts), and
 * a process that has handed all device memory to a pooling allocator, where a raw cudaMalloc
 * can simply fail.  This call makes no cudaMalloc, cudaFree or other allocating call.
 *   - Scratch (the split-K accumulator and a status word) is a fixed array of
 *     256 + 4 * TSFM_STATIC_GEMM_MAX_ELEMS bytes (4 MiB + 256 B) inside the library image; every
 *     GPU that loads the library holds it until the process exits.
 *   - M * N must not exceed TSFM_STATIC_GEMM_MAX_ELEMS: larger outputs are rejected with
 *     TSFM_ERR_SHAPE and a message available from tsfm_last_cuda_error().
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside of any stream capture.
 *   - Every call on a device shares the one array, which still holds the previous call's
 *     contents: the call clears the part it uses before accumulating.  Two calls that overlap
 *     on the GPU (different streams, or threads) race on it; serialise them.
 * A, W dev bf16 row-major, C dev fp32 [M, N] row-major (written last, by a device-to-device
 * copy); synchronises `stream` before returning. */
#define TSFM_STATIC_GEMM_MAX_ELEMS (1 << 20)
int tsfm_gemm_bf16_static(void *stream, const void *A, const void *W, float *C,
                          int32_t M, int32_t N, int32_t Kd);

/* Bounds-checking mode only (TSFM_EXEC_CHECK_BOUNDS): *n_regions (nullable) receives the number of
 * guard regions of the handle.  region >= 0 additionally overwrites (damage != 0) or restores
 * (damage == 0) one byte of that guard region -- a write inside the library's own allocation --
 * so that a test can see the checker report it.  region < 0: query only. */
int tsfm_spec_debug_guard(tsfm_spec *h, int32_t region, int32_t damage, int32_t *n_regions);

/* Per-launch timing, for roofline accounting.  While enabled, every kernel launch of the handle
 * is bracketed by two CUDA events on the handle's stream (this perturbs end-to-end time: do not
 * quote throughput from a profiled call).  tsfm_spec_set_profiling clears the records.
 * tsfm_spec_kernel_profile synchronises and aggregates them per kernel: launches, total device
 * milliseconds, and the algorithmic bytes and flops of those launches (what the operation must
 * move / compute: operands read once, results written once).  out: host array of `cap` entries;
 * *n receives the number of kernels with at least one launch. */
typedef struct {
  char    name[24];
  int64_t launches;
  double  ms_total;
  double  bytes;
  double  flops;
} tsfm_kernel_stat;
int tsfm_spec_set_profiling(tsfm_spec *h, int32_t enable);
int tsfm_spec_kernel_profile(tsfm_spec *h, int32_t cap, int32_t *n, tsfm_kernel_stat *out);

/* Block-size advice from measured quantities (host arithmetic only).  alpha = conditional
 * acceptance rate, c = draft step cost and v = verification pass cost in units of one target step.
 * Expected yield E[L_K] = sum_{j=0..K} alpha^j (Eq. 7), predicted speedup S(K) = E[L_K] / (c K + v)
 * (Eq. 8).  Steps K up from 1 while the marginal-gain condition alpha^(K+1) (c K + v) >= c E[L_K]
 * of the block-size proposition holds (it is equivalent to S(K+1) >= S(K)) and returns the K reached,
 * at most max_K; *speedup (nullable) receives S at that K.  Returns 0 on invalid arguments
 * (alpha outside [0, 1], c <= 0, v <= 0, max_K < 1). */
int32_t tsfm_advise_block_size(double alpha, double c, double v, int32_t max_K, double *speedup);

int tsfm_spec_destroy(tsfm_spec *h);

/* Number of kernels this library has launched in this process (all handles, all streams).  The
 * rounds of a graph-mode forecast count their launches on the device: the call waits for the
 * streams of all live handles to read those counters. */
int64_t tsfm_launch_count(void);

const char *tsfm_strerror(int code);
/* Text of the last CUDA error that produced TSFM_ERR_CUDA on this thread ("" if none). */
const char *tsfm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TSFM_H_ */

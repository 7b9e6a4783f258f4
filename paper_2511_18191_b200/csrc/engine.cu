// Host side of the decoder library: handle, weight-blob layout, forward-pass assembly,
// the speculative round loop (Algorithm 1 looped), target-only decoding (Eq. 1) and the
// C ABI declared in include/tsfm.h.
#include "../../include/tsfm.h"

#include <cuda_runtime.h>
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <tuple>
#include <vector>

#include "common.cuh"
#include "kernels_simt.cuh"
#include "attn_flash.cuh"
#include "accept.cuh"
#include "gemm_tc.cuh"
#include "gemm_sk.cuh"
#include "gemm_ws.cuh"

using namespace tsfm;

namespace {

std::atomic<long long> g_launches{0};
thread_local std::string g_cuda_err;
std::mutex g_handles_mu;
std::vector<tsfm_spec *> g_handles;           // live handles (their replayed rounds count launches on the device)
constexpr int kMaxGraphs = 16;                // captured forecast geometries kept per handle

#define CU_TRY(expr)                                                            \
  do {                                                                          \
    cudaError_t e_ = (expr);                                                    \
    if (e_ != cudaSuccess) {                                                    \
      g_cuda_err = std::string(#expr) + ": " + cudaGetErrorString(e_);          \
      return TSFM_ERR_CUDA;                                                     \
    }                                                                           \
  } while (0)

#define LAUNCHED() (g_launches.fetch_add(1, std::memory_order_relaxed))

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }
inline size_t elt_bytes(int dtype) { return dtype == TSFM_BF16 ? 2 : 4; }

bool arch_ok(const tsfm_arch &a, int P) {
  if (a.n_layers < 1 || a.d_model < 64 || a.n_heads < 1 || a.d_ff < 64) return false;
  if (a.d_model % a.n_heads) return false;
  const int dh = a.d_model / a.n_heads;
  if (dh != 32 && dh != 64 && dh != 128) return false;
  if (a.d_model % 64 || a.d_ff % 64) return false;
  if (P < 16 || P > 256 || P % 16) return false;
  return true;
}
// Input token length P_in (0 = P): it divides the patch length P (a patch is P / P_in tokens).
inline int token_len(int P_in, int P) { return P_in > 0 ? P_in : P; }
bool io_ok(int P_in, int P) { return P_in >= 0 && P % token_len(P_in, P) == 0; }

// Offsets of the tensors of one model inside its blob (canonical order, 256-byte aligned).
struct BlobLayout {
  size_t W_emb = 0, g_f = 0, W_head = 0, total = 0;
  struct L { size_t g1, Wq, Wk, Wv, Wo, g2, W1, W2; };
  std::vector<L> layers;
};

BlobLayout blob_layout(const tsfm_arch &a, int P, int dtype, int P_in = 0) {
  BlobLayout b;
  const size_t e = elt_bytes(dtype), d = a.d_model, f = a.d_ff;
  size_t off = 256;
  auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
  b.W_emb = take(d * token_len(P_in, P) * e);
  for (int l = 0; l < a.n_layers; ++l) {
    BlobLayout::L x;
    x.g1 = take(d * 4);
    x.Wq = take(d * d * e);
    x.Wk = take(d * d * e);
    x.Wv = take(d * d * e);
    x.Wo = take(d * d * e);
    x.g2 = take(d * 4);
    x.W1 = take(f * d * e);
    x.W2 = take(d * f * e);
    b.layers.push_back(x);
  }
  b.g_f = take(d * 4);
  b.W_head = take((size_t)P * d * e);
  b.total = off;
  return b;
}

struct LayerDev {
  const float *g1, *g2;
  const void *Wqkv, *Wo, *W1, *W2;
  GemmSkPlan tc_qkv, tc_o, tc_1, tc_2;
};

struct ModelDev {
  tsfm_arch arch{};
  int dh = 0;
  const void *W_emb = nullptr, *W_head = nullptr;
  const float *g_f = nullptr;
  std::vector<LayerDev> layers;
  void *Kc = nullptr, *Vc = nullptr;     // [L][B][heads][cap][dh]
  size_t kv_layer_elems = 0;
  float2 *rope = nullptr;                // [cap][dh/2] (cos, sin)
};

}  // namespace

struct GraphKey {
  int mode, B, N, H, K;
  bool operator<(const GraphKey &o) const {
    return std::tie(mode, B, N, H, K) < std::tie(o.mode, o.B, o.N, o.H, o.K);
  }
};
struct GraphInfo {
  cudaGraphExec_t exec = nullptr;
  long long n_fixed = 0;                 // kernel launches outside the round loop, per replay
};

struct tsfm_spec {
  tsfm_cfg cfg{};
  cudaStream_t stream = nullptr;         // the caller's stream: all work is ordered on it
  cudaStream_t ls = nullptr;             // stream the launches go to (== stream, or a capturing stream)
  cudaStream_t cap_stream = nullptr, cap_stream2 = nullptr;   // capture-only streams
  std::map<GraphKey, GraphInfo> graphs;
  unsigned long long *dev_launches = nullptr;   // launches made by replayed round bodies
  int *dev_body_launches = nullptr;             // [kMaxGraphs] launches of one round body, per cached graph
  DevState *st = nullptr;
  int P_in = 0, tpp = 1;                 // steps per input token; tokens per patch (P / P_in)
  int cap = 0;                           // token capacity per series of history and KV caches
  bool use_tc = false;
  bool pdl = false;                      // launches carry the programmatic-serialization attribute
  ModelDev tgt, drf;
  // activations (sized for M_max rows)
  int M_max = 0;
  float *x = nullptr, *qkv = nullptr, *ssq = nullptr;   // ssq: [M_max][d / 16] slice sums of squares
  void *a = nullptr, *ao = nullptr, *hbuf = nullptr;
  // decoding state
  float *hist = nullptr, *vout = nullptr, *mean = nullptr, *sd = nullptr;
  float *muq = nullptr;                  // [B][max_K][P] draft means of the round (sampled proposals)
  int *done = nullptr;
  int *live = nullptr, *n_live = nullptr;   // [B] slot -> unfinished series, and their number (round_end_kernel)
  bool compact = true;                   // rounds run over the unfinished series only
  AcceptCounters *ctr = nullptr;
  int *unfinished = nullptr;             // [max_T + 1]
  int *h_unfinished = nullptr;           // pinned
  int *dev_status = nullptr;
  int *tr_nacc = nullptr;                // [max_T][B]
  float *tr_ell = nullptr, *tr_logu = nullptr;   // [max_T][B][K]
  float *stage_in = nullptr, *stage_out = nullptr;   // device staging for the *_host entry points
  int last_B = 0, last_K = 0;
  int enqueue_err = TSFM_OK;             // first failure while enqueuing work (a launch that was refused)
  // optional per-launch timing (tsfm_spec_set_profiling)
  bool profiling = false;
  struct ProfRec { int cls; cudaEvent_t e0, e1; double bytes, flops; };
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> prof_pool;
  size_t prof_pool_used = 0;
  std::vector<cudaEvent_t> ev;
  std::vector<void *> owned;
  // bounds-checking mode (TSFM_EXEC_CHECK_BOUNDS): guard regions, their names, the device copy
  bool check = false;
  std::vector<GuardRegion> guards;
  std::vector<std::string> guard_names;
  GuardRegion *dev_guards = nullptr;
};

namespace {

// Kernel classes for per-launch timing.
// The tensor-core contraction is one kernel in three regimes: up to 512 tokens it streams weights
// (HBM / latency bound), from 4096 tokens it is tensor bound, between them it is one wave of tiles.
enum { KC_INSTNORM = 0, KC_EMBED, KC_RMSNORM, KC_GEMM_WS, KC_GEMM_TC_SMALL, KC_GEMM_TC_MID, KC_GEMM_TC_LARGE, KC_GEMM_SIMT,
       KC_ATTN, KC_HEAD, KC_ACCEPT, KC_DENORM, KC_COUNT };
const char *const kKernelNames[KC_COUNT] = {"instnorm", "embed", "rmsnorm", "gemm_ws_small_M", "gemm_sk_small_M",
                                            "gemm_sk_mid_M", "gemm_sk_large_M", "gemm_simt", "attn", "head", "accept",
                                            "denorm"};

// Brackets one launch with two events when profiling is on (no-op otherwise).
struct KTimer {
  tsfm_spec *h;
  size_t idx = 0;
  bool on = false;
  KTimer(tsfm_spec *h_, int cls, double bytes, double flops) : h(h_) {
    if (!h->profiling || cls < 0) return;
    auto get = [&]() -> cudaEvent_t {
      if (h->prof_pool_used == h->prof_pool.size()) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        h->prof_pool.push_back(e);
      }
      return h->prof_pool[h->prof_pool_used++];
    };
    tsfm_spec::ProfRec r{cls, get(), get(), bytes, flops};
    if (!r.e0 || !r.e1) return;
    cudaEventRecord(r.e0, h->ls);
    h->prof.push_back(r);
    idx = h->prof.size() - 1;
    on = true;
  }
  ~KTimer() {
    if (on) cudaEventRecord(h->prof[idx].e1, h->ls);
  }
};

constexpr size_t kGuardTail = 256;       // guard bytes behind every allocation in bounds-checking mode

// Registers (and fills) a guard region: n_blocks runs of len bytes, stride bytes apart.
int add_guard(tsfm_spec *h, const char *name, void *base, size_t stride, size_t n_blocks, size_t len) {
  if (n_blocks == 1) CU_TRY(cudaMemsetAsync(base, GUARD_BYTE, len, h->stream));
  else CU_TRY(cudaMemset2DAsync(base, stride, GUARD_BYTE, len, n_blocks, h->stream));
  h->guards.push_back(GuardRegion{(const unsigned char *)base, (unsigned long long)stride, (unsigned)n_blocks, (unsigned)len});
  h->guard_names.push_back(name);
  return TSFM_OK;
}

template <typename T>
int dev_alloc(tsfm_spec *h, T **p, size_t count, const char *name = "buffer") {
  void *q = nullptr;
  const size_t bytes = count * sizeof(T) ? count * sizeof(T) : 256;
  CU_TRY(cudaMalloc(&q, bytes + (h->check ? kGuardTail : 0)));
  h->owned.push_back(q);
  *p = (T *)q;
  if (h->check) return add_guard(h, name, (char *)q + bytes, 0, 1, kGuardTail);
  return TSFM_OK;
}

int read_header(const tsfm_weights *w, const tsfm_arch &a, int P, int P_in, int dtype, cudaStream_t s) {
  if (!w || !w->blob) return TSFM_ERR_ARG;
  int32_t hd[9];
  CU_TRY(cudaMemcpyAsync(hd, w->blob, sizeof(hd), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  if (hd[0] != 0x4D465354 || hd[1] != 1 || hd[2] != dtype || hd[3] < a.n_layers ||
      hd[4] != a.d_model || hd[5] != a.n_heads || hd[6] != a.d_ff || hd[7] != P ||
      token_len(hd[8], P) != token_len(P_in, P))
    return TSFM_ERR_SHAPE;
  return TSFM_OK;
}

// Wire a model's tensor pointers.  `blob_arch` is the shape the blob was written for (a
// layer-skip draft reads the first layers of the target's blob).
void wire_model(ModelDev &m, const tsfm_arch &arch, const tsfm_arch &blob_arch, const void *blob,
                int P, int dtype, int P_in) {
  const BlobLayout lay = blob_layout(blob_arch, P, dtype, P_in);
  const char *base = (const char *)blob;
  m.arch = arch;
  m.dh = arch.d_model / arch.n_heads;
  m.W_emb = base + lay.W_emb;
  m.g_f = (const float *)(base + lay.g_f);
  m.W_head = base + lay.W_head;
  m.layers.clear();
  for (int l = 0; l < arch.n_layers; ++l) {
    LayerDev L{};
    L.g1 = (const float *)(base + lay.layers[l].g1);
    L.g2 = (const float *)(base + lay.layers[l].g2);
    L.Wqkv = base + lay.layers[l].Wq;    // Wq, Wk, Wv are adjacent: one [3d, d] matrix
    L.Wo = base + lay.layers[l].Wo;
    L.W1 = base + lay.layers[l].W1;
    L.W2 = base + lay.layers[l].W2;
    m.layers.push_back(L);
  }
}

int make_rope(tsfm_spec *h, ModelDev &m) {
  const int half = m.dh / 2;
  std::vector<float2> t((size_t)h->cap * half);
  for (int p = 0; p < h->cap; ++p)
    for (int i = 0; i < half; ++i) {
      const double theta = std::pow((double)h->cfg.rope_base, -2.0 * i / m.dh);
      t[(size_t)p * half + i] = make_float2((float)std::cos(p * theta), (float)std::sin(p * theta));
    }
  if (int rc = dev_alloc(h, &m.rope, t.size(), "rope")) return rc;
  CU_TRY(cudaMemcpyAsync(m.rope, t.data(), t.size() * sizeof(float2), cudaMemcpyHostToDevice, h->stream));
  CU_TRY(cudaStreamSynchronize(h->stream));
  return TSFM_OK;
}

template <typename T> size_t attn_smem_bytes(int dh, int nk) {
  const int vw = AttnWords<T>::per_row(dh);
  return (size_t)nk * (2 * vw + 1) * 4 + (size_t)ATTN_QT * nk * sizeof(float) + (size_t)5 * ATTN_QT * dh * sizeof(float) +
         2 * ATTN_QT * sizeof(float);
}

// fp32 caches: number of CTAs (one cluster) that share the keys of one (series, head, query
// tile): long rows are split so that each CTA stages a quarter of the cache and more CTAs fit
// on an SM.
inline int attn_key_split(int cap) { return cap >= 192 ? 4 : 1; }
// key rows one CTA must hold: its share of the longest row, in whole 16-key MMA blocks
inline int attn_rows_per_cta(int cap, int skv) { return ((cap + skv - 1) / skv + 15) & ~15; }

template <typename T, int DH>
int attn_set_attr(size_t bytes) {
  CU_TRY(cudaFuncSetAttribute(attn_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  return TSFM_OK;
}
// bf16 caches take the running-softmax kernel (attn_flash_kernel), fp32 caches attn_kernel.
// Short rows with at least this many (series, head) pairs: one warp per pair instead of four
// (measured: C2's draft, 1024 pairs, 15 % faster that way; no difference at 256 pairs).
constexpr int kFlashWarpMaxCap = 64, kFlashWarpMinPairs = 512;
// Long rows with at least this many pairs take one warp per pair too: split four ways, a CTA's life
// is one pipeline fill (positions -> copies -> scores -> merge) and 1280 CTAs at three per SM need
// three such fills in a row; 1280 warps at twelve per SM are one wave, each streaming its whole row
// through its ring (measured on C4's verification pass and decode step: attention 51.7 -> 47.2 ms
// per forecast).
constexpr int kFlashWarpLongMinPairs = 1024;
// one-tile passes: a two-stage ring (each warp has a few chunks only, and a third CTA fits on the SM)
constexpr int kFlashStShort = 2;
template <int DH> int flash_set_attr() {
  CU_TRY(cudaFuncSetAttribute(attn_flash_kernel<DH, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, FlashGeom<DH, 3>::SMEM_BYTES));
  CU_TRY(cudaFuncSetAttribute(attn_flash_kernel<DH, kFlashStShort>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              FlashGeom<DH, kFlashStShort>::SMEM_BYTES));
  CU_TRY(cudaFuncSetAttribute(attn_flash_single_kernel<DH, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, FlashGeom<DH>::single_bytes(1)));
  CU_TRY(cudaFuncSetAttribute(attn_flash_single_kernel<DH, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, FlashGeom<DH>::single_bytes(2)));
  return TSFM_OK;
}
template <typename T>
int attn_prepare(int dh, int cap) {
  if constexpr (sizeof(T) == 2) {
    return dh == 32 ? flash_set_attr<32>() : dh == 64 ? flash_set_attr<64>() : flash_set_attr<128>();
  } else {
    const size_t bytes = attn_smem_bytes<T>(dh, attn_rows_per_cta(cap, attn_key_split(cap)));
    if (bytes > 227 * 1024) return TSFM_ERR_SHAPE;
    const size_t optin = 227 * 1024;        // opt in once to the per-CTA maximum; launches size themselves
    if (dh == 32) return attn_set_attr<T, 32>(optin);
    if (dh == 64) return attn_set_attr<T, 64>(optin);
    return attn_set_attr<T, 128>(optin);
  }
}

// Every kernel of the library asks for the same (maximum) shared-memory carve-out, so that the
// SMs never have to re-partition L1 / shared memory between two consecutive launches of a pass.
template <typename F> void prefer_max_smem(F *fn) {
  cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}
template <typename T> void prefer_max_smem_typed() {
  prefer_max_smem(embed_kernel<T>);
  prefer_max_smem(rmsnorm_kernel<T, false>);
  prefer_max_smem(rmsnorm_kernel<T, true>);
  prefer_max_smem(head_kernel<T>);
  prefer_max_smem(embed_rows_kernel<T>);
  prefer_max_smem(head_rows_kernel<T>);
  cudaFuncSetAttribute(head_rows_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  prefer_max_smem(gemm_simt_kernel<T, EPI_F32>);
  prefer_max_smem(gemm_simt_kernel<T, EPI_T>);
  prefer_max_smem(gemm_simt_kernel<T, EPI_GELU_T>);
  prefer_max_smem(gemm_simt_kernel<T, EPI_RESID>);
  if constexpr (sizeof(T) == 4) {
    prefer_max_smem(attn_kernel<T, 32>);
    prefer_max_smem(attn_kernel<T, 64>);
    prefer_max_smem(attn_kernel<T, 128>);
  }
  prefer_max_smem(kv_append_kernel<T, 32>);
  prefer_max_smem(kv_append_kernel<T, 64>);
  prefer_max_smem(kv_append_kernel<T, 128>);
}
void prefer_max_smem_all() {
  prefer_max_smem_typed<float>();
  prefer_max_smem_typed<bf16>();
  prefer_max_smem(instnorm_kernel);
  prefer_max_smem(denorm_kernel);
  prefer_max_smem(accept_kernel);
  prefer_max_smem(round_end_kernel);
  prefer_max_smem(gemm_sk_kernel<1, false>);
  prefer_max_smem(gemm_sk_kernel<1, true>);
  prefer_max_smem(gemm_sk_kernel<2, false>);
  prefer_max_smem(gemm_ws_kernel<false>);
  prefer_max_smem(gemm_ws_kernel<true>);
  prefer_max_smem(attn_flash_kernel<32, 3>);
  prefer_max_smem(attn_flash_kernel<32, kFlashStShort>);
  prefer_max_smem(attn_flash_kernel<64, 3>);
  prefer_max_smem(attn_flash_kernel<64, kFlashStShort>);
  prefer_max_smem(attn_flash_kernel<128, 3>);
  prefer_max_smem(attn_flash_kernel<128, kFlashStShort>);
  prefer_max_smem(attn_flash_single_kernel<32, 1>);
  prefer_max_smem(attn_flash_single_kernel<32, 2>);
  prefer_max_smem(attn_flash_single_kernel<64, 1>);
  prefer_max_smem(attn_flash_single_kernel<64, 2>);
  prefer_max_smem(attn_flash_single_kernel<128, 1>);
  prefer_max_smem(attn_flash_single_kernel<128, 2>);
  cudaGetLastError();
}

// One kernel launch; with pdl the launch carries the programmatic-serialization attribute, so
// the kernel may be scheduled while its predecessor drains (its pdl_wait() restores the order).
template <typename... KArgs, typename... Args>
void launch_ex(cudaStream_t s, bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
               Args &&...args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
  LAUNCHED();
}

// The same with a thread-block cluster of cluster_z CTAs along z (grid.z a multiple of it).
template <typename... KArgs, typename... Args>
void launch_ex_cluster(cudaStream_t s, bool pdl, int cluster_z, void (*kernel)(KArgs...), dim3 grid, dim3 block,
                       size_t smem, Args &&...args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = (unsigned)cluster_z;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
  LAUNCHED();
}

template <typename T>
void launch_gemm_simt(cudaStream_t s, bool pdl, const T *A, const T *W, void *C, int M, int N, int K, int epi) {
  dim3 grid((N + 63) / 64, (M + 63) / 64), block(256);
  switch (epi) {
    case EPI_F32: launch_ex(s, pdl, gemm_simt_kernel<T, EPI_F32>, grid, block, 0, A, W, C, M, N, K); break;
    case EPI_T: launch_ex(s, pdl, gemm_simt_kernel<T, EPI_T>, grid, block, 0, A, W, C, M, N, K); break;
    case EPI_GELU_T: launch_ex(s, pdl, gemm_simt_kernel<T, EPI_GELU_T>, grid, block, 0, A, W, C, M, N, K); break;
    default: launch_ex(s, pdl, gemm_simt_kernel<T, EPI_RESID>, grid, block, 0, A, W, C, M, N, K); break;
  }
}

// C (op)= A . W^T through the tensor-core kernel when a plan exists, else the FMA kernel.
template <typename T>
void gemm(tsfm_spec *h, GemmSkPlan *plan, const void *A, const void *W, void *C, int M, int N,
          int K, int epi, const SkNorm *norm = nullptr, LiveRows lr = LiveRows{nullptr, 0}) {
  const double e = sizeof(T);
  const double out_b = (epi == EPI_F32 || epi == EPI_ATOMIC) ? 4.0 : epi == EPI_RESID ? 8.0 : e;
  const double bytes = ((double)N * K + (double)M * K) * e + (double)M * N * out_b;
  const double flops = 2.0 * M * N * K;
  if (sizeof(T) == 2 && h->use_tc && plan && plan->valid && gemm_ws_eligible(A, W, M, N, K)) {
    // few tokens, short K: the shared-memory-resident weight tile kernel has the shorter chain
    KTimer kt(h, KC_GEMM_WS, bytes, flops);
    if (gemm_ws_launch(h->ls, h->pdl, A, W, C, M, N, K, epi, norm, lr)) {
      LAUNCHED();
    } else if (h->enqueue_err == TSFM_OK) {
      h->enqueue_err = TSFM_ERR_CUDA;
      g_cuda_err = std::string("small-batch contraction could not be launched: ") + cudaGetErrorString(cudaGetLastError());
    }
    return;
  }
  if (sizeof(T) == 2 && h->use_tc && plan && plan->valid) {
    KTimer kt(h, M <= 512 ? KC_GEMM_TC_SMALL : M < 4096 ? KC_GEMM_TC_MID : KC_GEMM_TC_LARGE, bytes, flops);
    if (gemm_sk_launch(h->ls, h->pdl, *plan, C, M, epi, h->dev_status, norm, lr)) {
      LAUNCHED();
    } else if (h->enqueue_err == TSFM_OK) {
      // No silent fallback: the FMA kernel knows nothing of a folded norm, and a pass that mixes
      // the two would be wrong without saying so.  The call that enqueued this reports the error.
      h->enqueue_err = TSFM_ERR_CUDA;
      g_cuda_err = std::string("tensor-core contraction could not be launched: ") + cudaGetErrorString(cudaGetLastError());
    }
    return;
  }
  KTimer kt(h, KC_GEMM_SIMT, bytes, flops);
  launch_gemm_simt<T>(h->ls, h->pdl, (const T *)A, (const T *)W, C, M, N, K, epi);
}

template <typename T, int DH>
void launch_attn(tsfm_spec *h, ModelDev &m, int l, int B, const PassGeom &g) {
  T *Kc = (T *)m.Kc + (size_t)l * m.kv_layer_elems;
  T *Vc = (T *)m.Vc + (size_t)l * m.kv_layer_elems;
  // algorithmic bytes: q/k/v of the pass + the cached keys and values (lower bound: done = 0)
  const double kv = (double)B * std::max(g.base, 0) * 2.0 * m.arch.d_model * sizeof(T);
  const double Mr = (double)B * g.q_len;
  KTimer kt(h, KC_ATTN, Mr * 3 * m.arch.d_model * 4 + kv + Mr * m.arch.d_model * (2.0 * sizeof(T) + sizeof(T)),
            4.0 * Mr * (std::max(g.base, 0) + 0.5 * g.q_len) * m.arch.d_model);
  // several query tiles: the pass's keys and values go to the cache first, once
  const int pre = g.q_len > ATTN_QT ? 1 : 0;
  if (pre)
    launch_ex(h->ls, h->pdl, kv_append_kernel<T, DH>, dim3(m.arch.n_heads, B, (g.q_len + 15) / 16), dim3(128), 0,
              h->qkv, Kc, Vc, m.rope, g, m.arch.n_heads);
  if constexpr (sizeof(T) == 2) {
    const int pairs = B * m.arch.n_heads;
    const int mode = pre ? FLASH_TILES
                         : ((h->cap <= kFlashWarpMaxCap && pairs >= kFlashWarpMinPairs) || pairs >= kFlashWarpLongMinPairs)
                               ? FLASH_WARP : FLASH_SPLIT;
    const dim3 grid = mode == FLASH_WARP ? dim3((pairs + 3) / 4)
                                         : dim3(m.arch.n_heads, B, pre ? (g.q_len + 4 * ATTN_QT - 1) / (4 * ATTN_QT) : 1);
    // short caches: one stage of 32 or 64 rows per warp instead of the ring, more warps per SM
    const int nb = pre ? 0 : h->cap <= FlashGeom<DH>::CHUNK ? 1 : h->cap <= 2 * FlashGeom<DH>::CHUNK ? 2 : 0;
    if (nb == 1)
      launch_ex(h->ls, h->pdl, attn_flash_single_kernel<DH, 1>, grid, dim3(128), (size_t)FlashGeom<DH>::single_bytes(1),
                h->qkv, (bf16 *)Kc, (bf16 *)Vc, m.rope, g, m.arch.n_heads, pairs, mode, (bf16 *)h->ao);
    else if (nb == 2)
      launch_ex(h->ls, h->pdl, attn_flash_single_kernel<DH, 2>, grid, dim3(128), (size_t)FlashGeom<DH>::single_bytes(2),
                h->qkv, (bf16 *)Kc, (bf16 *)Vc, m.rope, g, m.arch.n_heads, pairs, mode, (bf16 *)h->ao);
    else if (pre)
      launch_ex(h->ls, h->pdl, attn_flash_kernel<DH, 3>, grid, dim3(128), (size_t)FlashGeom<DH, 3>::SMEM_BYTES, h->qkv,
                (bf16 *)Kc, (bf16 *)Vc, m.rope, g, m.arch.n_heads, pairs, mode, (bf16 *)h->ao);
    else      // one query tile: each warp has a few chunks only, a two-stage ring lets a third CTA onto the SM
      launch_ex(h->ls, h->pdl, attn_flash_kernel<DH, kFlashStShort>, grid, dim3(128),
                (size_t)FlashGeom<DH, kFlashStShort>::SMEM_BYTES, h->qkv, (bf16 *)Kc, (bf16 *)Vc, m.rope, g,
                m.arch.n_heads, pairs, mode, (bf16 *)h->ao);
  } else {
    const int QT = g.q_len <= ATTN_QT ? g.q_len : ATTN_QT;
    const int skv = attn_key_split(h->cap);
    const dim3 grid(m.arch.n_heads, B, ((g.q_len + QT - 1) / QT) * skv);
    const int nk_max = attn_rows_per_cta(h->cap, skv);   // regions stay 16-byte aligned
    const size_t smem = attn_smem_bytes<T>(DH, nk_max);
    if (skv > 1)
      launch_ex_cluster(h->ls, h->pdl, skv, attn_kernel<T, DH>, grid, dim3(128), smem, h->qkv, Kc, Vc, m.rope, g,
                        m.arch.n_heads, QT, nk_max, skv, pre, (T *)h->ao);
    else
      launch_ex(h->ls, h->pdl, attn_kernel<T, DH>, grid, dim3(128), smem, h->qkv, Kc, Vc, m.rope, g, m.arch.n_heads,
                QT, nk_max, skv, pre, (T *)h->ao);
  }
}

enum { HEAD_NONE = 0, HEAD_LAST_TO_HIST = 1, HEAD_ALL_TO_VOUT = 2 };
// Passes of at least this many rows take the embedding and head kernels that share each weight
// load between 8 rows; below it there are too few rows to fill the SMs that way.
constexpr int kManyRows = 1024;
// Up to this many rows the separate RMSNorm kernel fetches its constants before the dependency wait.
constexpr int kNormEarlyMaxRows = 2048;

// Draft step i of a round (k_pos = i - 1): lets the head kernel turn its mean into a sampled
// proposal when the call asks for one (Sec. 3.3); target and prefill passes carry none.
struct DraftStep { int k_pos = -1, K = 0; };

// One causal pass of a model over q_len new tokens per series (appends to its KV cache).
template <typename T>
void run_pass(tsfm_spec *h, ModelDev &m, int B, const PassGeom &g, int head_mode, float *vout,
              unsigned long long *stamp, DraftStep ds, bool opens_round) {
  const int M = B * g.q_len, d = m.arch.d_model, f = m.arch.d_ff, P = h->cfg.patch_len, Pi = h->P_in;
  cudaStream_t s = h->ls;
  const float eps = h->cfg.rms_eps;
  // On the tensor-core path the RMSNorms are folded into the contractions around them (SkNorm):
  // whoever produces the residual stream also writes the next operand a' = bf16(gain * x) and the
  // rows' slice sums of squares; whoever consumes a' scales its result rows by rstd.
  // (Only for passes of few tokens, where a launch costs more than the extra epilogue work: with
  // large tiles the epilogue is the bottleneck and the separate RMSNorm kernel is the cheaper way.)
  // On the bf16 path the RMSNorms of passes of up to 512 tokens are folded into the contractions
  // around them (SkNorm): whoever produces the residual stream also writes the next operand
  // a' = bf16(gain * x) and the rows' sums of squares over 16-feature slices; whoever consumes a'
  // scales its result rows by rstd.  (Only for few tokens, where a launch costs more than the extra
  // epilogue work.  With the large tiles' TMA epilogues a producer would have to load its block of x
  // back after the reduction: measured on C2-C4, that costs what the RMSNorm kernel costs.)
  const bool fold = sizeof(T) == 2 && h->use_tc && m.layers[0].tc_qkv.valid && M <= 512;
  const int L = m.arch.n_layers;
  const LiveRows lr{g.n_live, g.q_len};
  // the RMSNorm of passes of a few thousand rows is a link in a chain: constants before the wait
  auto *norm_kernel = M <= kNormEarlyMaxRows && d <= 1280 ? rmsnorm_kernel<T, true> : rmsnorm_kernel<T, false>;
  {
    KTimer kt(h, KC_EMBED, (double)M * Pi * 4 + (double)d * Pi * sizeof(T) + (double)M * d * 4, 2.0 * M * Pi * d);
    if (!fold && M >= kManyRows)
      launch_ex(s, h->pdl, embed_rows_kernel<T>, dim3((M + 7) / 8, (d + 127) / 128), dim3(128), 8 * Pi * sizeof(float),
                h->hist, g, M, Pi, d, (const T *)m.W_emb, h->x, stamp);
    else
      launch_ex(s, h->pdl, embed_kernel<T>, dim3(M, (d + 127) / 128), dim3(128), Pi * sizeof(float), h->hist, g, Pi, d,
                (const T *)m.W_emb, h->x, stamp, fold ? m.layers[0].g1 : (const float *)nullptr,
                fold ? (T *)h->a : (T *)nullptr, fold ? h->ssq : (float *)nullptr, opens_round ? 1 : 0);
  }
  const double norm_bytes = (double)M * d * (4 + sizeof(T)) + d * 4.0;
  SkNorm consume{};                 // scale the result rows by rstd of the input rows
  consume.ssq_in = h->ssq;
  consume.n_part = d / 16;
  consume.inv_d = 1.f / d;
  consume.eps = eps;
  for (int l = 0; l < L; ++l) {
    LayerDev &ly = m.layers[l];
    if (!fold) {
      KTimer kt(h, KC_RMSNORM, norm_bytes, 3.0 * M * d);
      launch_ex(s, h->pdl, norm_kernel, dim3((M + 7) / 8), dim3(256), 0, h->x, ly.g1, M, d, eps, (T *)h->a, lr);
    }
    gemm<T>(h, &ly.tc_qkv, h->a, ly.Wqkv, h->qkv, M, 3 * d, d, EPI_F32, fold ? &consume : nullptr, lr);
    if (m.dh == 32) launch_attn<T, 32>(h, m, l, B, g);
    else if (m.dh == 64) launch_attn<T, 64>(h, m, l, B, g);
    else launch_attn<T, 128>(h, m, l, B, g);
    if (l == L - 1 && head_mode == HEAD_NONE) break;   // prefill: only the cache is needed
    SkNorm produce{};               // residual epilogue also emits the next operand and its statistics
    produce.ssq_out = h->ssq;
    produce.a_out = (bf16 *)h->a;
    produce.gain = ly.g2;
    gemm<T>(h, &ly.tc_o, h->ao, ly.Wo, h->x, M, d, d, EPI_RESID, fold ? &produce : nullptr, lr);
    if (!fold) {
      KTimer kt(h, KC_RMSNORM, norm_bytes, 3.0 * M * d);
      launch_ex(s, h->pdl, norm_kernel, dim3((M + 7) / 8), dim3(256), 0, h->x, ly.g2, M, d, eps, (T *)h->a, lr);
    }
    gemm<T>(h, &ly.tc_1, h->a, ly.W1, h->hbuf, M, f, d, EPI_GELU_T, fold ? &consume : nullptr, lr);
    produce.gain = l + 1 < L ? m.layers[l + 1].g1 : nullptr;
    if (l + 1 == L) produce.a_out = nullptr, produce.ssq_out = nullptr;   // the head kernel norms the final rows itself
    gemm<T>(h, &ly.tc_2, h->hbuf, ly.W2, h->x, M, d, f, EPI_RESID, fold && l + 1 < L ? &produce : nullptr, lr);
  }
  const int Mb = B * (g.q_len / g.head_step);          // boundary rows the head reads (verification)
  const double rows = head_mode == HEAD_LAST_TO_HIST ? B : Mb;
  KTimer kt(h, head_mode == HEAD_NONE ? -1 : KC_HEAD, rows * d * 4 + (double)P * d * sizeof(T) + rows * P * 4,
            2.0 * rows * P * d);
  const bool rows_fit = (size_t)8 * d * sizeof(float) <= 200 * 1024;
  // (The last-token head keeps one CTA per series and eight outputs also with a thousand series:
  // sharing each weight load between 8 series, as the verification head does, measured slower --
  // C3 target-only decode 15.98 vs 15.13 ms.)
  if (head_mode == HEAD_LAST_TO_HIST) {
    launch_ex(s, h->pdl, head_kernel<T>, dim3(B, (P + 7) / 8), dim3(256), d * sizeof(float), h->x, m.g_f,
              (const T *)m.W_head, d, P, eps, g, 1, h->hist, (float *)nullptr,
              ds.k_pos >= 0 ? (const DevState *)h->st : (const DevState *)nullptr, h->muq, ds.k_pos, ds.K, Pi);
  } else if (head_mode == HEAD_ALL_TO_VOUT && Mb >= kManyRows && rows_fit) {
    launch_ex(s, h->pdl, head_rows_kernel<T>, dim3((Mb + 7) / 8, (P + 31) / 32), dim3(256), (size_t)8 * d * sizeof(float),
              h->x, m.g_f, (const T *)m.W_head, Mb, d, P, eps, vout, g);
  } else if (head_mode == HEAD_ALL_TO_VOUT) {
    launch_ex(s, h->pdl, head_kernel<T>, dim3(Mb, (P + 7) / 8), dim3(256), d * sizeof(float), h->x, m.g_f,
              (const T *)m.W_head, d, P, eps, g, 0, (float *)nullptr, vout, (const DevState *)nullptr, (float *)nullptr, 0, 0,
              Pi);
  }
}

// opens_round: the pass is the first of a round, i.e. its first kernel directly follows the kernel
// that closed the previous one (and wrote the live list); it then looks its slots up after its wait.
void pass(tsfm_spec *h, ModelDev &m, int B, const PassGeom &g, int head_mode, float *vout = nullptr,
          unsigned long long *stamp = nullptr, DraftStep ds = DraftStep{}, bool opens_round = false) {
  if (g.q_len < 1) return;
  if (h->cfg.dtype == TSFM_BF16) run_pass<bf16>(h, m, B, g, head_mode, vout, stamp, ds, opens_round);
  else run_pass<float>(h, m, B, g, head_mode, vout, stamp, ds, opens_round);
}

int check_call(tsfm_spec *h, const float *series, int B, int ctx_len, int H, float *out, int K) {
  if (!h || !series || !out) return TSFM_ERR_ARG;
  if (B < 1 || H < 1 || ctx_len < 1) return TSFM_ERR_ARG;
  const int P = h->cfg.patch_len;
  if (ctx_len % P) return TSFM_ERR_SHAPE;                       // the context is a whole number of patches
  const int N = ctx_len / h->P_in, T = (H + P - 1) / P;         // N counts input tokens
  if (ctx_len / P < 2) return TSFM_ERR_SHAPE;
  if (B > h->cfg.max_batch || N > h->cfg.max_ctx_tokens || T > h->cfg.max_horizon_patches ||
      K > h->cfg.max_K)
    return TSFM_ERR_SHAPE;
  return TSFM_OK;
}

// ---------------------------------------------------------------- enqueue helpers
// Each of these only enqueues work on h->ls; none synchronises, so that they can run under
// stream capture.

void enqueue_begin(tsfm_spec *h, int B, int ctx_len) {
  const int hist_stride = h->cap * h->P_in;             // values per series in the history buffer
  const int hist_len = hist_stride - (h->check ? h->P_in : 0);   // (the spare token stays untouched)
  cudaMemsetAsync(h->dev_status, 0, sizeof(int), h->ls);
  KTimer kt(h, KC_INSTNORM, (double)B * (ctx_len + (double)hist_len) * 4, 4.0 * B * ctx_len);
  launch_ex(h->ls, h->pdl, instnorm_kernel, dim3(B), dim3(256), 0, h->st, ctx_len, hist_stride, hist_len, h->cfg.norm_eps, h->hist,
            h->mean, h->sd, h->done, h->live, h->n_live);
}

// Bounds-checking mode: after the work of a call, look at every guard region.
void enqueue_guard_check(tsfm_spec *h) {
  if (!h->check || h->guards.empty()) return;
  launch_ex(h->ls, h->pdl, guard_check_kernel, dim3(64, (unsigned)std::min<size_t>(h->guards.size(), 1024)), dim3(256), 0,
            (const GuardRegion *)h->dev_guards, (int)h->guards.size(), h->dev_status);
}

// N = context tokens.
void enqueue_denorm(tsfm_spec *h, int B, int N, int H) {
  KTimer kt(h, KC_DENORM, 8.0 * B * H, 2.0 * B * H);
  launch_ex(h->ls, h->pdl, denorm_kernel, dim3(B), dim3(256), 0, h->hist, N * h->P_in, h->cap * h->P_in, H, h->mean, h->sd,
            h->st);
  enqueue_guard_check(h);
}

// Everything of a speculative forecast that precedes the round loop: counters, traces,
// instance norm, and the prefill of both caches (the target ingests the context except its
// last patch, the draft except its last two: those are re-read by the first round).
// N counts context tokens; a patch is tpp = P / P_in of them.
void enqueue_spec_prologue(tsfm_spec *h, int B, int N, int T, int K) {
  cudaStream_t s = h->ls;
  cudaMemsetAsync(h->ctr, 0, sizeof(AcceptCounters), s);
  cudaMemsetAsync(h->unfinished, 0, sizeof(int) * (T + 1), s);
  cudaMemsetAsync(h->tr_nacc, 0xff, sizeof(int) * (size_t)T * B, s);
  cudaMemsetAsync(h->tr_ell, 0, sizeof(float) * (size_t)T * B * K, s);
  cudaMemsetAsync(h->tr_logu, 0, sizeof(float) * (size_t)T * B * K, s);
  const int tpp = h->tpp;
  enqueue_begin(h, B, N * h->P_in);
  pass(h, h->tgt, B, PassGeom{nullptr, 0, N - tpp, h->cap}, HEAD_NONE);
  pass(h, h->drf, B, PassGeom{nullptr, 0, N - 2 * tpp, h->cap}, HEAD_NONE);
}

// One round of Algorithm 1 for the whole batch: K draft steps, one verification pass over
// [pending, x_1..x_K], the fused accept, and the round bookkeeping.  The round index, tau and
// the Philox key are read from device state, so the same enqueued work serves every round.
void enqueue_round(tsfm_spec *h, int B, int N, int T, int K, cudaGraphConditionalHandle handle, int use_handle,
                   const int *body_launches = nullptr) {
  const int P = h->cfg.patch_len, tpp = h->tpp;
  // the passes of a round run over the unfinished series only (see PassGeom)
  const int *live = h->compact ? h->live : nullptr, *n_live = h->compact ? h->n_live : nullptr;
  // step 1 re-ingests the last two committed patches (the draft cache may lack the last
  // accepted proposal), steps 2..K ingest the previous proposal; a patch is tpp tokens
  pass(h, h->drf, B, PassGeom{h->done, N - 2 * tpp, 2 * tpp, h->cap, live, n_live, tpp, tpp}, HEAD_LAST_TO_HIST, nullptr,
       &h->st->t_phase[0], DraftStep{0, K}, true);
  for (int i = 2; i <= K; ++i)
    pass(h, h->drf, B, PassGeom{h->done, N - tpp + (i - 1) * tpp, tpp, h->cap, live, n_live, tpp, tpp}, HEAD_LAST_TO_HIST,
         nullptr, nullptr, DraftStep{i - 1, K});
  // single-pass verification over [pending, x_1..x_K], read at the last token of each patch: the
  // prefix boundaries N - 1 + i (P / P_in), i = 0..K (appendix B, "Per-Family Boundary Indexing")
  pass(h, h->tgt, B, PassGeom{h->done, N - tpp, (K + 1) * tpp, h->cap, live, n_live, tpp, tpp}, HEAD_ALL_TO_VOUT, h->vout,
       &h->st->t_phase[1]);

  AcceptArgs a{};
  a.x = a.mu_q = h->hist + (size_t)N * h->P_in;   // patch done[b] behind the context holds x_1
  a.x_stride_b = (long long)h->cap * h->P_in;
  a.mu_q_alt = h->muq;                          // used only when the call samples its proposals
  a.mu_p = h->vout;
  a.commit = h->hist + (size_t)N * h->P_in;
  a.commit_stride_b = a.x_stride_b;
  a.commit_accepted = 0;
  a.commit_follows_done = 1;
  a.done = h->done;
  a.B = B; a.K = K; a.P = P; a.T = T;
  a.margin = h->cfg.dtype == TSFM_BF16 ? 5e-2f : 1e-3f;
  a.series0 = 0;
  a.forced_u = nullptr;
  a.ctr = h->ctr;
  a.n_accept = h->tr_nacc;
  a.ell = h->tr_ell;
  a.log_u = h->tr_logu;
  a.unfinished = h->unfinished;
  a.st = h->st;
  {
    KTimer kt(h, KC_ACCEPT, (double)B * (2 * K + 2) * P * 4, 4.0 * B * K * P);
    launch_ex(h->ls, h->pdl, accept_kernel, dim3((B + 3) / 4), dim3(128), 0, a);
  }
  launch_ex(h->ls, h->pdl, round_end_kernel, dim3(1), dim3(256), 0, h->st, (const int *)h->unfinished, T, handle,
            use_handle, body_launches, h->dev_launches, (const int *)h->done, B, h->live, h->n_live);
}

// Plain patch-autoregressive decoding with one model (the target, or the draft on its own).
void enqueue_single_model(tsfm_spec *h, ModelDev &m, int B, int N, int T, int H) {
  const int tpp = h->tpp;
  enqueue_begin(h, B, N * h->P_in);
  pass(h, m, B, PassGeom{nullptr, 0, N - tpp, h->cap}, HEAD_NONE);
  for (int t = 0; t < T; ++t)       // Eq. 1: one pass per committed patch (its tpp tokens)
    pass(h, m, B, PassGeom{nullptr, N - tpp + t * tpp, tpp, h->cap}, HEAD_LAST_TO_HIST, nullptr,
         t == 0 ? &h->st->t_phase[0] : nullptr);
  enqueue_denorm(h, B, N, H);
}

// The first error met while enqueuing (and clears it).
int take_enqueue_err(tsfm_spec *h) {
  const int rc = h->enqueue_err;
  h->enqueue_err = TSFM_OK;
  return rc;
}

// ---------------------------------------------------------------- graph capture
// A forecast of a given geometry is captured once into a CUDA graph and replayed: the
// prologue, a WHILE node whose body is one round (the round-end kernel sets the condition),
// and the de-normalisation.  Capture runs on the handle's own streams (the caller's stream
// may be the legacy default stream, which cannot capture); the graph is launched on the
// caller's stream.
int capture_graph(tsfm_spec *h, const GraphKey &k, int slot, GraphInfo *out) {
  const int P = h->cfg.patch_len, T = (k.H + P - 1) / P;
  cudaStream_t cs = h->cap_stream, cs2 = h->cap_stream2;
  cudaGraph_t graph = nullptr;
  const cudaStreamCaptureMode mode = cudaStreamCaptureModeThreadLocal;
  const long long launches0 = g_launches.load();
  long long n_body = 0;
  CU_TRY(cudaStreamBeginCapture(cs, mode));
  int rc = TSFM_OK;
  auto step = [&](cudaError_t e, const char *what) {
    if (rc == TSFM_OK && e != cudaSuccess) {
      g_cuda_err = std::string(what) + ": " + cudaGetErrorString(e);
      rc = TSFM_ERR_CUDA;
    }
    return rc == TSFM_OK;
  };
  h->ls = cs;
  if (k.mode != 0) {
    enqueue_single_model(h, k.mode == 1 ? h->tgt : h->drf, k.B, k.N, T, k.H);
  } else {
    enqueue_spec_prologue(h, k.B, k.N, T, k.K);
    cudaStreamCaptureStatus status;
    cudaGraph_t g = nullptr;
    const cudaGraphNode_t *deps = nullptr;
    size_t ndeps = 0;
    cudaGraphConditionalHandle handle{};
    cudaGraphNode_t node = nullptr;
    cudaGraphNodeParams np{};
    np.type = cudaGraphNodeTypeConditional;
    if (step(cudaStreamGetCaptureInfo(cs, &status, nullptr, &g, &deps, &ndeps), "cudaStreamGetCaptureInfo") &&
        step(cudaGraphConditionalHandleCreate(&handle, g, 1, cudaGraphCondAssignDefault),
             "cudaGraphConditionalHandleCreate")) {
      np.conditional.handle = handle;
      np.conditional.type = cudaGraphCondTypeWhile;
      np.conditional.size = 1;
      if (step(cudaGraphAddNode(&node, g, deps, ndeps, &np), "cudaGraphAddNode(conditional)") &&
          step(cudaStreamUpdateCaptureDependencies(cs, &node, 1, cudaStreamSetCaptureDependencies),
               "cudaStreamUpdateCaptureDependencies")) {
        cudaGraph_t body = np.conditional.phGraph_out[0];
        if (step(cudaStreamBeginCaptureToGraph(cs2, body, nullptr, nullptr, 0, mode), "cudaStreamBeginCaptureToGraph")) {
          h->ls = cs2;
          const long long before = g_launches.load();
          enqueue_round(h, k.B, k.N, T, k.K, handle, 1, h->dev_body_launches + slot);
          n_body = g_launches.load() - before;
          cudaGraph_t same = nullptr;
          step(cudaStreamEndCapture(cs2, &same), "cudaStreamEndCapture(body)");
          h->ls = cs;
        }
      }
    }
    if (rc == TSFM_OK) enqueue_denorm(h, k.B, k.N, k.H);
  }
  h->ls = h->stream;
  step(cudaStreamEndCapture(cs, &graph), "cudaStreamEndCapture");
  out->n_fixed = g_launches.load() - launches0 - n_body;
  g_launches.store(launches0);                     // captured launches have not run
  if (rc == TSFM_OK) step(cudaGetLastError(), "capture");
  if (rc == TSFM_OK) rc = take_enqueue_err(h);
  if (rc == TSFM_OK) step(cudaGraphInstantiate(&out->exec, graph, 0), "cudaGraphInstantiate");
  if (graph) cudaGraphDestroy(graph);
  if (rc == TSFM_OK) {
    // the round body reports its own launch count to the device-side launch counter
    const int nb = (int)n_body;
    step(cudaMemcpyAsync(h->dev_body_launches + slot, &nb, sizeof(int), cudaMemcpyHostToDevice, h->stream),
         "cudaMemcpyAsync(body launches)");
  }
  return rc;
}

int get_graph(tsfm_spec *h, const GraphKey &k, GraphInfo *info) {
  auto it = h->graphs.find(k);
  if (it != h->graphs.end()) { *info = it->second; return TSFM_OK; }
  if ((int)h->graphs.size() >= kMaxGraphs) {       // bounded cache: drop everything and start over
    CU_TRY(cudaStreamSynchronize(h->stream));
    for (auto &kv : h->graphs) cudaGraphExecDestroy(kv.second.exec);
    h->graphs.clear();
  }
  GraphInfo gi;
  if (int rc = capture_graph(h, k, (int)h->graphs.size(), &gi)) {
    if (gi.exec) cudaGraphExecDestroy(gi.exec);
    return rc;
  }
  h->graphs[k] = gi;
  *info = gi;
  return TSFM_OK;
}

// Writes the call parameters and clears the loop state.  The source is an ordinary host
// struct: for pageable memory the copy is staged before the call returns.
int write_call_state(tsfm_spec *h, const float *series, float *out, float tau, uint64_t seed,
                     const tsfm_variant *v = nullptr) {
  DevState st{};
  st.series = series;
  st.out = out;
  st.tau = tau;
  st.sigma_q = v && v->sigma_q > 0.f ? v->sigma_q : tau;
  st.fallback_r = v ? v->fallback_noise : 0.f;
  st.flags = v ? (v->sample_proposals ? VAR_SAMPLE_PROPOSALS : 0) | (v->no_tempering ? VAR_NO_TEMPERING : 0) : 0;
  st.key0 = (uint32_t)(seed & 0xffffffffu);
  st.key1 = (uint32_t)(seed >> 32);
  CU_TRY(cudaMemcpyAsync(h->st, &st, sizeof(st), cudaMemcpyHostToDevice, h->stream));
  return TSFM_OK;
}

// Launches made so far by this handle's replayed round bodies (waits for its stream).
long long device_launches(tsfm_spec *h) {
  unsigned long long v = 0;
  if (!h->dev_launches) return 0;
  if (cudaMemcpyAsync(&v, h->dev_launches, sizeof(v), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return 0;
  return (long long)v;
}

bool use_graph(const tsfm_spec *h) { return !(h->cfg.exec_mode & TSFM_EXEC_STREAM) && !h->profiling; }

// What a non-zero device status word means for the caller.
int status_code(tsfm_spec *h, int status) {
  if (status == 0) return TSFM_OK;
  if (status < DEV_GUARD_BASE) return TSFM_ERR_TIMEOUT;
  const size_t k = (size_t)(status - DEV_GUARD_BASE);
  g_cuda_err = "bounds check: a kernel wrote past the end of '" +
               (k < h->guard_names.size() ? h->guard_names[k] : std::string("?")) + "' (guard region " + std::to_string(k) + ")";
  return TSFM_ERR_INTERNAL;
}

// Reads status and phase clocks back (synchronises) and fills ms_total.
int finish_stats(tsfm_spec *h, tsfm_stats *stats, DevState *st_out) {
  cudaStream_t s = h->stream;
  CU_TRY(cudaEventRecord(h->ev[1], s));
  CU_TRY(cudaMemcpyAsync(st_out, h->st, sizeof(DevState), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaMemcpyAsync(&stats->device_status, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  CU_TRY(cudaEventElapsedTime(&stats->ms_total, h->ev[0], h->ev[1]));
  return TSFM_OK;
}

}  // namespace

// ====================================================================================
// C ABI
// ====================================================================================
extern "C" {

size_t tsfm_weights_bytes(const tsfm_arch *arch, int32_t patch_len, int32_t dtype) {
  return tsfm_weights_bytes_io(arch, 0, patch_len, dtype);
}

size_t tsfm_weights_offset(const tsfm_arch *arch, int32_t patch_len, int32_t dtype, int32_t layer,
                           const char *name) {
  return tsfm_weights_offset_io(arch, 0, patch_len, dtype, layer, name);
}

size_t tsfm_weights_bytes_io(const tsfm_arch *arch, int32_t patch_in, int32_t patch_len, int32_t dtype) {
  if (!arch || !arch_ok(*arch, patch_len) || !io_ok(patch_in, patch_len) || (dtype != TSFM_F32 && dtype != TSFM_BF16))
    return 0;
  return blob_layout(*arch, patch_len, dtype, patch_in).total;
}

size_t tsfm_weights_offset_io(const tsfm_arch *arch, int32_t patch_in, int32_t patch_len, int32_t dtype, int32_t layer,
                              const char *name) {
  if (!arch || !name || !arch_ok(*arch, patch_len) || !io_ok(patch_in, patch_len) ||
      (dtype != TSFM_F32 && dtype != TSFM_BF16))
    return 0;
  const BlobLayout b = blob_layout(*arch, patch_len, dtype, patch_in);
  const std::string n(name);
  if (n == "W_emb") return b.W_emb;
  if (n == "g_f") return b.g_f;
  if (n == "W_head") return b.W_head;
  if (layer < 0 || layer >= arch->n_layers) return 0;
  const BlobLayout::L &l = b.layers[layer];
  if (n == "g1") return l.g1;
  if (n == "Wq") return l.Wq;
  if (n == "Wk") return l.Wk;
  if (n == "Wv") return l.Wv;
  if (n == "Wo") return l.Wo;
  if (n == "g2") return l.g2;
  if (n == "W1") return l.W1;
  if (n == "W2") return l.W2;
  return 0;
}

int tsfm_spec_destroy(tsfm_spec *h) {
  if (!h) return TSFM_ERR_ARG;
  cudaStreamSynchronize(h->stream);
  {
    std::lock_guard<std::mutex> lock(g_handles_mu);
    for (size_t i = 0; i < g_handles.size(); ++i)
      if (g_handles[i] == h) {
        g_launches.fetch_add(device_launches(h));      // keep what its replayed rounds launched
        g_handles.erase(g_handles.begin() + i);
        break;
      }
  }
  for (auto &kv : h->graphs) cudaGraphExecDestroy(kv.second.exec);
  if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
  if (h->cap_stream2) cudaStreamDestroy(h->cap_stream2);
  for (cudaEvent_t e : h->prof_pool) cudaEventDestroy(e);
  for (void *p : h->owned) cudaFree(p);
  if (h->h_unfinished) cudaFreeHost(h->h_unfinished);
  for (cudaEvent_t e : h->ev) cudaEventDestroy(e);
  delete h;
  return TSFM_OK;
}

int tsfm_spec_create(const tsfm_weights *target_w, const tsfm_weights *draft_w, const tsfm_cfg *cfg,
                     tsfm_spec **out_h) {
  if (!target_w || !cfg || !out_h) return TSFM_ERR_ARG;
  *out_h = nullptr;
  const int P = cfg->patch_len;
  if (cfg->dtype != TSFM_F32 && cfg->dtype != TSFM_BF16) return TSFM_ERR_ARG;
  if (cfg->exec_mode & ~(TSFM_EXEC_STREAM | TSFM_EXEC_NO_PDL | TSFM_EXEC_NO_COMPACT | TSFM_EXEC_CHECK_BOUNDS))
    return TSFM_ERR_ARG;
  if (cfg->gemm_backend != TSFM_GEMM_AUTO && cfg->gemm_backend != TSFM_GEMM_SIMT) return TSFM_ERR_ARG;
  if (cfg->draft_mode != TSFM_DRAFT_SEPARATE && cfg->draft_mode != TSFM_DRAFT_LAYER_SKIP) return TSFM_ERR_ARG;
  if (cfg->max_batch < 1 || cfg->max_ctx_tokens < 2 || cfg->max_horizon_patches < 1 || cfg->max_K < 1 ||
      cfg->max_K > TSFM_MAX_K)
    return TSFM_ERR_ARG;
  if (!(cfg->rms_eps > 0.f) || !(cfg->norm_eps > 0.f) || !(cfg->rope_base > 1.f)) return TSFM_ERR_ARG;
  if (!arch_ok(cfg->target, P) || !arch_ok(cfg->draft, P) || !io_ok(cfg->patch_in, P)) return TSFM_ERR_SHAPE;
  if (cfg->draft_mode == TSFM_DRAFT_LAYER_SKIP) {
    if (draft_w && draft_w->blob) return TSFM_ERR_ARG;
    if (cfg->draft.d_model != cfg->target.d_model || cfg->draft.n_heads != cfg->target.n_heads ||
        cfg->draft.d_ff != cfg->target.d_ff || cfg->draft.n_layers > cfg->target.n_layers)
      return TSFM_ERR_SHAPE;
  } else if (!draft_w || !draft_w->blob) {
    return TSFM_ERR_ARG;
  }
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CU_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return TSFM_ERR_ARCH;

  tsfm_spec *h = new (std::nothrow) tsfm_spec();
  if (!h) return TSFM_ERR_INTERNAL;
  h->cfg = *cfg;
  h->stream = h->ls = (cudaStream_t)cfg->stream;
  h->P_in = token_len(cfg->patch_in, P);
  h->tpp = P / h->P_in;
  if (cfg->max_ctx_tokens < 2 * h->tpp) { delete h; return TSFM_ERR_ARG; }   // at least two context patches
  h->check = (cfg->exec_mode & TSFM_EXEC_CHECK_BOUNDS) != 0;
  // token capacity per series; bounds-checking mode adds one spare token that nothing may write
  h->cap = cfg->max_ctx_tokens + (cfg->max_horizon_patches + cfg->max_K + 1) * h->tpp + (h->check ? 1 : 0);
  h->use_tc = cfg->dtype == TSFM_BF16 && cfg->gemm_backend != TSFM_GEMM_SIMT;
  h->pdl = (cfg->exec_mode & TSFM_EXEC_NO_PDL) == 0;
  h->compact = (cfg->exec_mode & TSFM_EXEC_NO_COMPACT) == 0;
  int rc = TSFM_OK;
  auto fail = [&](int code) { tsfm_spec_destroy(h); return code; };

  const int Pi = cfg->patch_in;
  if (target_w->bytes < blob_layout(cfg->target, P, cfg->dtype, Pi).total) return fail(TSFM_ERR_SHAPE);
  if ((rc = read_header(target_w, cfg->target, P, Pi, cfg->dtype, h->stream))) return fail(rc);
  wire_model(h->tgt, cfg->target, cfg->target, target_w->blob, P, cfg->dtype, Pi);
  if (cfg->draft_mode == TSFM_DRAFT_LAYER_SKIP) {
    wire_model(h->drf, cfg->draft, cfg->target, target_w->blob, P, cfg->dtype, Pi);
  } else {
    if (draft_w->bytes < blob_layout(cfg->draft, P, cfg->dtype, Pi).total) return fail(TSFM_ERR_SHAPE);
    if ((rc = read_header(draft_w, cfg->draft, P, Pi, cfg->dtype, h->stream))) return fail(rc);
    wire_model(h->drf, cfg->draft, cfg->draft, draft_w->blob, P, cfg->dtype, Pi);
  }

  const size_t e = elt_bytes(cfg->dtype);
  const int Bm = cfg->max_batch;
  for (ModelDev *m : {&h->tgt, &h->drf}) {
    m->kv_layer_elems = (size_t)Bm * m->arch.d_model * h->cap;
    const size_t bytes = m->kv_layer_elems * m->arch.n_layers * e;
    if ((rc = dev_alloc(h, (char **)&m->Kc, bytes, "K cache"))) return fail(rc);
    if ((rc = dev_alloc(h, (char **)&m->Vc, bytes, "V cache"))) return fail(rc);
    if (h->check) {                       // the spare last row of every (layer, series, head) block
      const size_t row = (size_t)m->dh * e, blk = (size_t)h->cap * row;
      const size_t n_blk = (size_t)m->arch.n_layers * Bm * m->arch.n_heads;
      if ((rc = add_guard(h, "K cache row past a series' capacity", (char *)m->Kc + blk - row, blk, n_blk, row))) return fail(rc);
      if ((rc = add_guard(h, "V cache row past a series' capacity", (char *)m->Vc + blk - row, blk, n_blk, row))) return fail(rc);
    }
    if ((rc = make_rope(h, *m))) return fail(rc);
    rc = cfg->dtype == TSFM_BF16 ? attn_prepare<bf16>(m->dh, h->cap) : attn_prepare<float>(m->dh, h->cap);
    if (rc) return fail(rc);
  }
  h->M_max = Bm * std::max(std::max(cfg->max_ctx_tokens, (cfg->max_K + 1) * h->tpp), 2 * h->tpp);
  const int dmax = std::max(cfg->target.d_model, cfg->draft.d_model);
  const int fmax = std::max(cfg->target.d_ff, cfg->draft.d_ff);
  const size_t Mx = h->M_max;
  if ((rc = dev_alloc(h, &h->x, Mx * dmax, "x"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->qkv, Mx * 3 * dmax, "qkv"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->ssq, Mx * (dmax / 16 + 1), "ssq"))) return fail(rc);
  if ((rc = dev_alloc(h, (char **)&h->a, Mx * dmax * e, "a"))) return fail(rc);
  if ((rc = dev_alloc(h, (char **)&h->ao, Mx * dmax * e, "ao"))) return fail(rc);
  if ((rc = dev_alloc(h, (char **)&h->hbuf, Mx * fmax * e, "hbuf"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->hist, (size_t)Bm * h->cap * h->P_in, "hist"))) return fail(rc);
  if (h->check) {                         // the spare last token of every series' history
    const size_t tok = (size_t)h->P_in * sizeof(float), blk = (size_t)h->cap * tok;
    if ((rc = add_guard(h, "history token past a series' capacity", (char *)h->hist + blk - tok, blk, Bm, tok))) return fail(rc);
  }
  if ((rc = dev_alloc(h, &h->vout, (size_t)Bm * (cfg->max_K + 1) * P, "vout"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->muq, (size_t)Bm * cfg->max_K * P, "muq"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->mean, Bm, "mean"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->sd, Bm, "sd"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->done, Bm, "done"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->live, Bm, "live"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->n_live, 1))) return fail(rc);
  if ((rc = dev_alloc(h, &h->ctr, 1))) return fail(rc);
  if ((rc = dev_alloc(h, &h->unfinished, cfg->max_horizon_patches + 1, "unfinished"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->dev_status, 1))) return fail(rc);
  if ((rc = dev_alloc(h, &h->st, 1))) return fail(rc);
  if ((rc = dev_alloc(h, &h->dev_launches, 1))) return fail(rc);
  if ((rc = dev_alloc(h, &h->dev_body_launches, kMaxGraphs))) return fail(rc);
  if (cudaMemsetAsync(h->st, 0, sizeof(DevState), h->stream) != cudaSuccess ||
      cudaMemsetAsync(h->dev_launches, 0, sizeof(unsigned long long), h->stream) != cudaSuccess)
    return fail(TSFM_ERR_CUDA);
  if (cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&h->cap_stream2, cudaStreamNonBlocking) != cudaSuccess)
    return fail(TSFM_ERR_CUDA);
  const size_t tr = (size_t)cfg->max_horizon_patches * Bm;
  if ((rc = dev_alloc(h, &h->tr_nacc, tr, "trace n_accept"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->tr_ell, tr * cfg->max_K, "trace ell"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->tr_logu, tr * cfg->max_K, "trace log_u"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->stage_in, (size_t)Bm * cfg->max_ctx_tokens * h->P_in, "stage_in"))) return fail(rc);
  if ((rc = dev_alloc(h, &h->stage_out, (size_t)Bm * cfg->max_horizon_patches * P, "stage_out"))) return fail(rc);
  if (cudaMallocHost((void **)&h->h_unfinished, sizeof(int)) != cudaSuccess) return fail(TSFM_ERR_CUDA);
  h->ev.resize(2 + 4 * (size_t)cfg->max_horizon_patches + 4);
  for (auto &ev : h->ev)
    if (cudaEventCreate(&ev) != cudaSuccess) { ev = nullptr; return fail(TSFM_ERR_CUDA); }
  if (cudaMemsetAsync(h->dev_status, 0, sizeof(int), h->stream) != cudaSuccess) return fail(TSFM_ERR_CUDA);

  if (h->check) {
    if ((rc = dev_alloc(h, &h->dev_guards, h->guards.size() + 1, "guard table"))) return fail(rc);
    if (cudaMemcpyAsync(h->dev_guards, h->guards.data(), sizeof(GuardRegion) * h->guards.size(), cudaMemcpyHostToDevice,
                        h->stream) != cudaSuccess)
      return fail(TSFM_ERR_CUDA);
  }
  prefer_max_smem_all();
  if (h->use_tc) {
    if ((rc = gemm_sk_init())) return fail(rc);
    if ((rc = gemm_ws_init())) return fail(rc);
    for (ModelDev *m : {&h->tgt, &h->drf}) {
      const int d = m->arch.d_model, f = m->arch.d_ff;
      for (LayerDev &ly : m->layers) {
        if ((rc = gemm_sk_plan(&ly.tc_qkv, ly.Wqkv, 3 * d, d, h->a, h->M_max))) return fail(rc);
        if ((rc = gemm_sk_plan(&ly.tc_o, ly.Wo, d, d, h->ao, h->M_max))) return fail(rc);
        if ((rc = gemm_sk_plan(&ly.tc_1, ly.W1, f, d, h->a, h->M_max))) return fail(rc);
        if ((rc = gemm_sk_plan(&ly.tc_2, ly.W2, d, f, h->hbuf, h->M_max))) return fail(rc);
      }
    }
  }
  if (cudaStreamSynchronize(h->stream) != cudaSuccess) return fail(TSFM_ERR_CUDA);
  {
    std::lock_guard<std::mutex> lock(g_handles_mu);
    g_handles.push_back(h);
  }
  *out_h = h;
  return TSFM_OK;
}

static int single_model_forecast(tsfm_spec *h, int mode, const float *series, int32_t B, int32_t ctx_len, int32_t H,
                                 float *out, tsfm_stats *stats) {
  if (int rc = check_call(h, series, B, ctx_len, H, out, 1)) return rc;
  const int P = h->cfg.patch_len, N = ctx_len / h->P_in, T = (H + P - 1) / P;
  cudaStream_t s = h->stream;
  if (stats) CU_TRY(cudaEventRecord(h->ev[0], s));
  if (int rc = write_call_state(h, series, out, 1.f, 0)) return rc;
  if (use_graph(h)) {
    GraphInfo gi;
    if (int rc = get_graph(h, GraphKey{mode, B, N, H, 0}, &gi)) return rc;
    CU_TRY(cudaGraphLaunch(gi.exec, s));
    g_launches.fetch_add(gi.n_fixed, std::memory_order_relaxed);
  } else {
    h->ls = s;
    enqueue_single_model(h, mode == 1 ? h->tgt : h->drf, B, N, T, H);
  }
  CU_TRY(cudaGetLastError());
  if (int rc = take_enqueue_err(h)) return rc;
  if (stats) {
    std::memset(stats, 0, sizeof(*stats));
    DevState st;
    if (int rc = finish_stats(h, stats, &st)) return rc;
    stats->ms_prefill = (float)((st.t_phase[0] - st.t_call) * 1e-6);
    (mode == 1 ? stats->ms_verify : stats->ms_draft) = (float)((st.t_end - st.t_phase[0]) * 1e-6);
    stats->rounds = T;
    stats->patches_committed = (int64_t)B * T;
    if (stats->device_status) return status_code(h, stats->device_status);
  }
  return TSFM_OK;
}

int tsfm_target_only_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H,
                              float *out, tsfm_stats *stats) {
  return single_model_forecast(h, 1, series, B, ctx_len, H, out, stats);
}

int tsfm_draft_only_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H,
                             float *out, tsfm_stats *stats) {
  return single_model_forecast(h, 2, series, B, ctx_len, H, out, stats);
}

int tsfm_spec_forecast(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H, int32_t K,
                       float tau, uint64_t seed, float *out, tsfm_stats *stats) {
  return tsfm_spec_forecast_variant(h, series, B, ctx_len, H, K, tau, seed, nullptr, out, stats);
}

int tsfm_spec_forecast_variant(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H, int32_t K,
                               float tau, uint64_t seed, const tsfm_variant *variant, float *out,
                               tsfm_stats *stats) {
  if (K < 1) return TSFM_ERR_ARG;
  if (!(tau > 0.f) || !std::isfinite(tau)) return TSFM_ERR_ARG;
  if (variant) {
    if (!std::isfinite(variant->sigma_q) || variant->sigma_q < 0.f || !std::isfinite(variant->fallback_noise) ||
        variant->fallback_noise < 0.f)
      return TSFM_ERR_ARG;
  }
  if (int rc = check_call(h, series, B, ctx_len, H, out, K)) return rc;
  const int P = h->cfg.patch_len, N = ctx_len / h->P_in, T = (H + P - 1) / P;
  cudaStream_t s = h->stream;
  if (stats) CU_TRY(cudaEventRecord(h->ev[0], s));
  if (int rc = write_call_state(h, series, out, tau, seed, variant)) return rc;
  if (use_graph(h)) {
    // one launch: prologue, WHILE(rounds), de-normalisation; no host round trip
    GraphInfo gi;
    if (int rc = get_graph(h, GraphKey{0, B, N, H, K}, &gi)) return rc;
    CU_TRY(cudaGraphLaunch(gi.exec, s));
    g_launches.fetch_add(gi.n_fixed, std::memory_order_relaxed);   // the rounds count themselves on the device
  } else {
    h->ls = s;
    enqueue_spec_prologue(h, B, N, T, K);
    for (int r = 0; r < T; ++r) {
      enqueue_round(h, B, N, T, K, cudaGraphConditionalHandle{}, 0);
      CU_TRY(cudaMemcpyAsync(h->h_unfinished, h->unfinished + r, sizeof(int), cudaMemcpyDeviceToHost, s));
      CU_TRY(cudaStreamSynchronize(s));
      if (*h->h_unfinished == 0) break;
    }
    enqueue_denorm(h, B, N, H);
  }
  h->last_B = B; h->last_K = K;
  CU_TRY(cudaGetLastError());
  if (int rc = take_enqueue_err(h)) return rc;
  if (stats) {
    std::memset(stats, 0, sizeof(*stats));
    AcceptCounters c;
    DevState st;
    CU_TRY(cudaMemcpyAsync(&c, h->ctr, sizeof(c), cudaMemcpyDeviceToHost, s));
    if (int rc = finish_stats(h, stats, &st)) return rc;
    stats->rounds = st.round;
    stats->proposals_drafted = (int64_t)c.drafted;
    stats->proposals_tested = (int64_t)c.tested;
    stats->proposals_accepted = (int64_t)c.accepted;
    stats->patches_committed = (int64_t)c.committed;
    stats->near_margin_decisions = (int64_t)c.near_margin;
    for (int i = 0; i < TSFM_MAX_K; ++i) {
      stats->tested_by_pos[i] = (int64_t)c.tested_by_pos[i];
      stats->accepted_by_pos[i] = (int64_t)c.accepted_by_pos[i];
    }
    for (int i = 0; i < TSFM_MAX_K + 2; ++i) stats->L_hist[i] = (int64_t)c.L_hist[i];
    stats->ms_prefill = (float)(st.ns_prefill * 1e-6);
    stats->ms_draft = (float)(st.ns_draft * 1e-6);
    stats->ms_verify = (float)(st.ns_verify * 1e-6);
    stats->ms_accept = (float)(st.ns_accept * 1e-6);
    if (stats->device_status) return status_code(h, stats->device_status);
  }
  return TSFM_OK;
}

int tsfm_spec_forecast_host(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H,
                            int32_t K, float tau, uint64_t seed, float *out, tsfm_stats *stats) {
  if (K < 1) return TSFM_ERR_ARG;
  if (int rc = check_call(h, series, B, ctx_len, H, out, K)) return rc;
  CU_TRY(cudaMemcpyAsync(h->stage_in, series, sizeof(float) * (size_t)B * ctx_len, cudaMemcpyHostToDevice, h->stream));
  if (int rc = tsfm_spec_forecast(h, h->stage_in, B, ctx_len, H, K, tau, seed, h->stage_out, stats)) return rc;
  CU_TRY(cudaMemcpyAsync(out, h->stage_out, sizeof(float) * (size_t)B * H, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(cudaStreamSynchronize(h->stream));
  return TSFM_OK;
}

int tsfm_target_only_forecast_host(tsfm_spec *h, const float *series, int32_t B, int32_t ctx_len, int32_t H,
                                   float *out, tsfm_stats *stats) {
  if (int rc = check_call(h, series, B, ctx_len, H, out, 1)) return rc;
  CU_TRY(cudaMemcpyAsync(h->stage_in, series, sizeof(float) * (size_t)B * ctx_len, cudaMemcpyHostToDevice, h->stream));
  if (int rc = tsfm_target_only_forecast(h, h->stage_in, B, ctx_len, H, h->stage_out, stats)) return rc;
  CU_TRY(cudaMemcpyAsync(out, h->stage_out, sizeof(float) * (size_t)B * H, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(cudaStreamSynchronize(h->stream));
  return TSFM_OK;
}

int tsfm_spec_last_trace(tsfm_spec *h, int32_t cap_rounds, int32_t *rounds, int32_t *n_accept, float *ell,
                         float *log_u) {
  if (!h || !rounds) return TSFM_ERR_ARG;
  cudaStream_t s = h->stream;
  int R = 0;
  CU_TRY(cudaMemcpyAsync(&R, &h->st->round, sizeof(int), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  *rounds = R;
  if (cap_rounds < R) return TSFM_ERR_ARG;
  const size_t nb = (size_t)R * h->last_B, nk = nb * h->last_K;
  if (n_accept && nb) CU_TRY(cudaMemcpyAsync(n_accept, h->tr_nacc, nb * sizeof(int), cudaMemcpyDeviceToHost, s));
  if (ell && nk) CU_TRY(cudaMemcpyAsync(ell, h->tr_ell, nk * sizeof(float), cudaMemcpyDeviceToHost, s));
  if (log_u && nk) CU_TRY(cudaMemcpyAsync(log_u, h->tr_logu, nk * sizeof(float), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  return TSFM_OK;
}

int tsfm_accept_round(void *stream, const float *x, const float *mu_q, const float *mu_p, int32_t B,
                      int32_t K, int32_t P, int32_t T, float sigma_p, float sigma_q, uint64_t seed,
                      int32_t round_idx, int32_t series0, const float *forced_u, int32_t *done,
                      float *commit, int32_t *n_accept, float *ell, float *log_u) {
  if (!x || !mu_q || !mu_p || !done || !commit) return TSFM_ERR_ARG;
  if (B < 1 || K < 1 || K > TSFM_MAX_K || P < 1 || T < 1) return TSFM_ERR_ARG;
  if (!(sigma_p > 0.f) || !(sigma_q > 0.f) || !std::isfinite(sigma_p) || !std::isfinite(sigma_q))
    return TSFM_ERR_ARG;
  AcceptArgs a{};
  a.x = x; a.mu_q = mu_q; a.x_stride_b = (long long)K * P;
  a.mu_p = mu_p;
  a.commit = commit; a.commit_stride_b = (long long)(K + 1) * P;
  a.commit_accepted = 1; a.commit_follows_done = 0;
  a.done = done;
  a.B = B; a.K = K; a.P = P; a.T = T;
  a.sigma_p = sigma_p; a.sigma_q = sigma_q; a.margin = 0.f;
  a.key = make_uint2((uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32));
  a.round_idx = round_idx; a.series0 = series0;
  a.forced_u = forced_u;
  a.n_accept = n_accept; a.ell = ell; a.log_u = log_u;
  accept_kernel<<<(B + 3) / 4, 128, 0, (cudaStream_t)stream>>>(a);
  LAUNCHED();
  CU_TRY(cudaGetLastError());
  return TSFM_OK;
}

int tsfm_model_forward(tsfm_spec *h, int32_t which, const float *tokens, int32_t B, int32_t n, float *out) {
  if (!h || !tokens || !out || (which != 0 && which != 1)) return TSFM_ERR_ARG;
  if (B < 1 || n < 1) return TSFM_ERR_ARG;
  if (B > h->cfg.max_batch || n > h->cfg.max_ctx_tokens || B * n > h->M_max) return TSFM_ERR_SHAPE;
  const int Pi = h->P_in;
  CU_TRY(cudaMemcpy2DAsync(h->hist, (size_t)h->cap * Pi * sizeof(float), tokens, (size_t)n * Pi * sizeof(float),
                           (size_t)n * Pi * sizeof(float), B, cudaMemcpyDeviceToDevice, h->stream));
  CU_TRY(cudaMemsetAsync(h->dev_status, 0, sizeof(int), h->stream));
  h->ls = h->stream;
  pass(h, which == 0 ? h->tgt : h->drf, B, PassGeom{nullptr, 0, n, h->cap}, HEAD_ALL_TO_VOUT, out);
  enqueue_guard_check(h);
  CU_TRY(cudaGetLastError());
  if (int rc = take_enqueue_err(h)) return rc;
  int status = 0;
  CU_TRY(cudaMemcpyAsync(&status, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(cudaStreamSynchronize(h->stream));
  return status_code(h, status);
}

int tsfm_gemm_bf16(void *stream, const void *A, const void *W, float *C, int32_t M, int32_t N, int32_t Kd,
                   int32_t backend) {
  if (!A || !W || !C) return TSFM_ERR_ARG;
  if (M < 1 || N < 1 || Kd < 16 || Kd % 16) return TSFM_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (backend == TSFM_GEMM_SIMT) {
    launch_gemm_simt<bf16>(s, false, (const bf16 *)A, (const bf16 *)W, C, M, N, Kd, EPI_F32);
    CU_TRY(cudaGetLastError());
    return TSFM_OK;
  }
  if (backend == TSFM_GEMM_WS) {
    if (!gemm_ws_eligible(A, W, M, N, Kd)) return TSFM_ERR_SHAPE;
    if (int rc = gemm_ws_init()) return rc;
    if (!gemm_ws_launch(s, false, A, W, C, M, N, Kd, EPI_F32, nullptr, LiveRows{nullptr, 0})) CU_TRY(cudaGetLastError());
    LAUNCHED();
    CU_TRY(cudaGetLastError());
    return TSFM_OK;
  }
  if (Kd % 8) return TSFM_ERR_SHAPE;
  if (int rc = gemm_sk_init()) return rc;
  GemmSkPlan plan;
  if (int rc = gemm_sk_plan(&plan, W, N, Kd, A, M)) return rc;
  if (!plan.valid) return TSFM_ERR_SHAPE;
  int *status = nullptr;
  CU_TRY(cudaMalloc((void **)&status, sizeof(int)));
  if (cudaError_t e0 = cudaMemsetAsync(status, 0, sizeof(int), s)) {
    cudaFree(status);
    CU_TRY(e0);
  }
  const bool ok = gemm_sk_launch(s, false, plan, C, M, EPI_F32, status);
  if (ok) LAUNCHED();
  int hs = 0;
  cudaError_t e1 = cudaMemcpyAsync(&hs, status, sizeof(int), cudaMemcpyDeviceToHost, s);
  cudaError_t e2 = cudaStreamSynchronize(s);
  cudaFree(status);
  CU_TRY(e1);
  CU_TRY(e2);
  CU_TRY(cudaGetLastError());
  if (!ok) return TSFM_ERR_INTERNAL;
  return hs ? TSFM_ERR_TIMEOUT : TSFM_OK;
}

// ------------------------------------------------------------------------------------
// Allocation-free variant of the tensor-core contraction (see include/tsfm.h).
// The accumulator of the K-split partial sums and the kernel's status word live in a
// file-scope device array instead of cudaMalloc'd memory.  The array's name is only a
// host-side handle for the symbol: its device address is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
// ------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[256 + sizeof(float) * TSFM_STATIC_GEMM_MAX_ELEMS];

static int static_scratch_ptr(unsigned char **out) {
  static std::mutex mu;
  static unsigned char *per_device[64] = {nullptr};
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return TSFM_ERR_INTERNAL;
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    unsigned char *p = nullptr;
    CU_TRY(cudaGetSymbolAddress((void **)&p, g_static_scratch));
    if (!p) return TSFM_ERR_INTERNAL;
    per_device[dev] = p;
  }
  *out = per_device[dev];
  return TSFM_OK;
}

int tsfm_gemm_bf16_static(void *stream, const void *A, const void *W, float *C, int32_t M, int32_t N,
                          int32_t Kd) {
  if (!A || !W || !C) return TSFM_ERR_ARG;
  if (M < 1 || N < 1 || Kd < 16 || Kd % 16) return TSFM_ERR_ARG;
  if ((long long)M * N > (long long)TSFM_STATIC_GEMM_MAX_ELEMS) {
    g_cuda_err = "tsfm_gemm_bf16_static: M * N = " + std::to_string((long long)M * N) +
                 " output elements exceed the static scratch capacity of " +
                 std::to_string((long long)TSFM_STATIC_GEMM_MAX_ELEMS);
    return TSFM_ERR_SHAPE;
  }
  cudaStream_t s = (cudaStream_t)stream;
  unsigned char *scratch = nullptr;
  if (int rc = static_scratch_ptr(&scratch)) return rc;
  if (int rc = gemm_tc_init()) return rc;
  GemmTcPlan plan;
  if (int rc = gemm_tc_plan(&plan, W, N, Kd, A, M)) return rc;
  if (!plan.valid) return TSFM_ERR_SHAPE;
  int *status = (int *)scratch;
  float *acc = (float *)(scratch + 256);
  const size_t out_bytes = sizeof(float) * (size_t)M * N;
  // the array keeps whatever the previous call left: the status word and the part of the
  // accumulator this call adds into must start at zero
  CU_TRY(cudaMemsetAsync(status, 0, 256, s));
  CU_TRY(cudaMemsetAsync(acc, 0, out_bytes, s));
  if (!gemm_tc_launch(s, plan, A, acc, M, EPI_ATOMIC, status)) return TSFM_ERR_INTERNAL;
  CU_TRY(cudaGetLastError());            // a refused launch: C is left untouched
  LAUNCHED();
  int hs = 0;
  CU_TRY(cudaMemcpyAsync(C, acc, out_bytes, cudaMemcpyDeviceToDevice, s));
  CU_TRY(cudaMemcpyAsync(&hs, status, sizeof(int), cudaMemcpyDeviceToHost, s));
  CU_TRY(cudaStreamSynchronize(s));
  CU_TRY(cudaGetLastError());
  return hs ? TSFM_ERR_TIMEOUT : TSFM_OK;
}

int tsfm_spec_debug_guard(tsfm_spec *h, int32_t region, int32_t damage, int32_t *n_regions) {
  if (!h) return TSFM_ERR_ARG;
  if (n_regions) *n_regions = (int32_t)h->guards.size();
  if (region < 0) return TSFM_OK;
  if (!h->check || (size_t)region >= h->guards.size()) return TSFM_ERR_ARG;
  // one byte of the library's own guard region: an ordinary in-bounds write
  const GuardRegion &g = h->guards[region];
  unsigned char *p = const_cast<unsigned char *>(g.base) + (size_t)(g.n_blocks - 1) * g.stride + g.len - 1;
  CU_TRY(cudaMemsetAsync(p, damage ? 0x00 : GUARD_BYTE, 1, h->stream));
  CU_TRY(cudaStreamSynchronize(h->stream));
  return TSFM_OK;
}

int tsfm_spec_set_profiling(tsfm_spec *h, int32_t enable) {
  if (!h) return TSFM_ERR_ARG;
  CU_TRY(cudaStreamSynchronize(h->stream));
  h->profiling = enable != 0;
  h->prof.clear();
  h->prof_pool_used = 0;
  return TSFM_OK;
}

int tsfm_spec_kernel_profile(tsfm_spec *h, int32_t cap, int32_t *n, tsfm_kernel_stat *out) {
  if (!h || !n || (cap > 0 && !out)) return TSFM_ERR_ARG;
  CU_TRY(cudaStreamSynchronize(h->stream));
  tsfm_kernel_stat acc[KC_COUNT];
  std::memset(acc, 0, sizeof(acc));
  for (int c = 0; c < KC_COUNT; ++c) std::snprintf(acc[c].name, sizeof(acc[c].name), "%s", kKernelNames[c]);
  for (const tsfm_spec::ProfRec &r : h->prof) {
    float ms = 0.f;
    CU_TRY(cudaEventElapsedTime(&ms, r.e0, r.e1));
    acc[r.cls].launches += 1;
    acc[r.cls].ms_total += ms;
    acc[r.cls].bytes += r.bytes;
    acc[r.cls].flops += r.flops;
  }
  int k = 0;
  for (int c = 0; c < KC_COUNT; ++c)
    if (acc[c].launches) {
      if (k < cap) out[k] = acc[c];
      ++k;
    }
  *n = k;
  return k <= cap ? TSFM_OK : TSFM_ERR_ARG;
}

int32_t tsfm_advise_block_size(double alpha, double c, double v, int32_t max_K, double *speedup) {
  if (!(alpha >= 0.0 && alpha <= 1.0) || !(c > 0.0) || !(v > 0.0) || max_K < 1) return 0;
  int K = 1;
  double EL = 1.0 + alpha, pw = alpha * alpha;      // E[L_1], alpha^(K+1) at K = 1
  while (K < max_K && pw * (c * K + v) >= c * EL) {
    EL += pw;                                        // E[L_{K+1}] = E[L_K] + alpha^(K+1)
    pw *= alpha;
    ++K;
  }
  if (speedup) *speedup = EL / (c * K + v);
  return K;
}

int64_t tsfm_launch_count(void) {
  long long n = g_launches.load();
  std::lock_guard<std::mutex> lock(g_handles_mu);
  for (tsfm_spec *h : g_handles) n += device_launches(h);
  return n;
}

const char *tsfm_strerror(int code) {
  switch (code) {
    case TSFM_OK: return "ok";
    case TSFM_ERR_ARG: return "invalid argument";
    case TSFM_ERR_SHAPE: return "unsupported shape or capacity exceeded";
    case TSFM_ERR_ARCH: return "device is not sm_100";
    case TSFM_ERR_CUDA: return "CUDA call failed";
    case TSFM_ERR_TIMEOUT: return "bounded device-side wait expired";
    case TSFM_ERR_INTERNAL: return "internal error";
    default: return "unknown error code";
  }
}

const char *tsfm_last_cuda_error(void) { return g_cuda_err.c_str(); }

}  // extern "C"

// Plain CUDA-core kernels of the forward pass: instance norm, patch embedding, RMSNorm,
// FMA GEMM, RoPE causal attention over the contiguous KV cache, final norm + mean head,
// de-normalisation.  Everything is templated on the storage type T (float | bf16) of
// weights, MMA-operand activations and the KV cache; the residual stream, norms, softmax
// and head output are always fp32.
#pragma once
#include "common.cuh"

namespace tsfm {

// Where the tokens of one pass sit.  Token j of series b is history token
// pos0(b) + j with pos0(b) = done[b] * tpp + base (done may be NULL = 0; tpp = tokens per
// committed patch: 1 when a token is a whole patch, P / P_in for shorter input tokens).
// Activations are stored row-major with row = b * q_len + j.  The mean head reads every
// head_step-th token of a pass (the last token of each patch: the prefix boundaries
// N - 1 + i (P / P_in) of the paper's appendix B, "Per-Family Boundary Indexing").
//
// Active-series compaction: inside the round loop only the series that still have patches to
// commit take part in a pass.  `live` lists them in ascending order and `n_live` counts them (both
// written by round_end_kernel); the pass works on SLOTS 0 .. n_live-1, slot s standing for series
// live[s].  Activation rows are compacted (row = slot * q_len + j); history, KV caches, `done` and
// the verification output stay indexed by series.  Grids are sized for all B series (a captured
// graph cannot change them): blocks of slots >= n_live return at once.  live == NULL: slot = series.
struct PassGeom {
  const int *done;   // [B] patches committed so far, or NULL
  int base;          // pos0 = done[b] + base
  int q_len;         // tokens per series in this pass
  int cap;           // token capacity of history / KV cache per series
  const int *live = nullptr;     // [B] slot -> series, or NULL
  const int *n_live = nullptr;   // number of live slots, or NULL (all)
  int tpp = 1;                   // tokens per committed patch
  int head_step = 1;             // the head reads tokens head_step - 1, 2 head_step - 1, ... of the pass
};
__device__ __forceinline__ int pos0_of(const PassGeom &g, int b) {
  return (g.done ? g.done[b] * g.tpp : 0) + g.base;
}
__device__ __forceinline__ bool slot_dead(const PassGeom &g, int slot) { return g.n_live && slot >= *g.n_live; }
__device__ __forceinline__ int series_of(const PassGeom &g, int slot) { return g.live ? g.live[slot] : slot; }
// Series, first token position and liveness of a slot in one go.  The live count and the slot's series
// are two independent loads (issued together); the committed count follows the series index.  The
// loads are volatile (served by L2) because most kernels do this lookup BEFORE their dependency wait,
// to take its two L2 round trips off the chain of dependent launches: `live` / `n_live` are written
// only by round_end_kernel (and the instance-norm kernel), `done` only by accept_kernel, and every
// kernel of a pass except the embedding that opens a round has at least two kernels between itself
// and those -- a grid starts only after every CTA of its predecessor has passed its own dependency
// wait, i.e. after the predecessor's predecessor has finished.  A dead slot's entry of `live` is a
// stale but valid series index, so the lookup stays in bounds.
struct SlotPos {
  int b, p0;
  bool dead;
};
__device__ __forceinline__ SlotPos slot_lookup(const PassGeom &g, int slot) {
  const int nl = g.n_live ? *reinterpret_cast<const volatile int *>(g.n_live) : 0x7fffffff;
  const int b = g.live ? reinterpret_cast<const volatile int *>(g.live)[slot] : slot;
  SlotPos s;
  s.dead = slot >= nl;
  s.b = b;
  s.p0 = (g.done ? reinterpret_cast<const volatile int *>(g.done)[b] * g.tpp : 0) + g.base;
  return s;
}
// Rows of a pass that are in use: n_live * q_len of the M the launch was sized for.
struct LiveRows {
  const int *n_live;
  int q_len;
};
__device__ __forceinline__ int live_rows(const LiveRows &lr, int M) {
  return lr.n_live ? min(M, *lr.n_live * lr.q_len) : M;
}

// ----------------------------------------------------------------------------------
// Instance statistics frozen on the context (Sec. 3.4) and history initialisation.
// grid = B, block = 256.  hist[b, :ctx_len] = (series - mean) / sd; the rest of the
// series' hist_len values is zeroed.  Sums in fp64 (8 K values, one pass each).
// ----------------------------------------------------------------------------------
__global__ void instnorm_kernel(DevState *__restrict__ st, int ctx_len, int hist_stride, int hist_len,
                                float norm_eps, float *__restrict__ hist,
                                float *__restrict__ mean_out, float *__restrict__ sd_out,
                                int *__restrict__ done, int *__restrict__ live, int *__restrict__ n_live) {
  __shared__ double red[32];
  const int b = blockIdx.x;
  pdl_sync();
  if (b == 0 && threadIdx.x == 0) st->t_call = globaltimer_ns();
  const float *s = st->series + (size_t)b * ctx_len;
  double acc = 0.0;
  for (int i = threadIdx.x; i < ctx_len; i += blockDim.x) acc += (double)s[i];
  const double mean = block_sum_d(acc, red) / ctx_len;
  acc = 0.0;
  for (int i = threadIdx.x; i < ctx_len; i += blockDim.x) {
    const double c = (double)s[i] - mean;
    acc += c * c;
  }
  const double var = block_sum_d(acc, red) / ctx_len;
  const double sd = sqrt(var + (double)norm_eps);
  float *hb = hist + (size_t)b * hist_stride;             // (stride > length only in bounds-checking mode)
  for (int i = threadIdx.x; i < hist_len; i += blockDim.x)
    hb[i] = (i < ctx_len) ? (float)(((double)s[i] - mean) / sd) : 0.f;
  if (threadIdx.x == 0) {
    mean_out[b] = (float)mean;
    sd_out[b] = (float)sd;
    done[b] = 0;
    live[b] = b;                                  // every series starts unfinished
    if (b == 0) *n_live = gridDim.x;
  }
}

// out[b, s] = hist[b, ctx_len + s] * sd + mean, s < H.   grid = B.
__global__ void denorm_kernel(const float *hist, int ctx_len, int hist_len, int H,
                              const float *mean, const float *sd,
                              DevState *__restrict__ st) {
  const int b = blockIdx.x;
  pdl_sync();
  float *out = st->out;
  if (b == 0 && threadIdx.x == 0) st->t_end = globaltimer_ns();
  const float m = mean[b], s = sd[b];
  const float *hb = hist + (size_t)b * hist_len + ctx_len;
  for (int i = threadIdx.x; i < H; i += blockDim.x) out[(size_t)b * H + i] = hb[i] * s + m;
}

// Bounds-checking mode: every guard byte must still hold GUARD_BYTE after a forecast; the first
// region found damaged is reported through the status word.  grid = (64, regions), block = 256.
__global__ void guard_check_kernel(const GuardRegion *__restrict__ regions, int n, int *__restrict__ status) {
  pdl_sync();
  for (int k = blockIdx.y; k < n; k += gridDim.y) {
    const GuardRegion r = regions[k];
    const unsigned long long total = (unsigned long long)r.n_blocks * r.len;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (unsigned long long)gridDim.x * blockDim.x) {
      if (r.base[(i / r.len) * r.stride + (i % r.len)] != GUARD_BYTE) {
        atomicCAS(status, 0, DEV_GUARD_BASE + k);
        break;
      }
    }
  }
}

// 16-byte vector loads of T (8 bf16 or 4 fp32) unpacked to floats.
template <typename T> struct Vec16;
// (raw() / unpack() split the load from its use: kernels fetch constants of the model before their
// dependency wait and unpack them after it.)
template <> struct Vec16<float> {
  static constexpr int N = 4;
  using Raw = float4;
  static __device__ __forceinline__ Raw raw(const float *p) { return *reinterpret_cast<const float4 *>(p); }
  static __device__ __forceinline__ void unpack(const Raw &t, float *v) { v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  static __device__ __forceinline__ void load(const float *p, float *v) { unpack(raw(p), v); }
};
template <> struct Vec16<bf16> {
  static constexpr int N = 8;
  using Raw = uint4;
  static __device__ __forceinline__ Raw raw(const bf16 *p) { return *reinterpret_cast<const uint4 *>(p); }
  static __device__ __forceinline__ void unpack(const Raw &t, float *v) {
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ void load(const bf16 *p, float *v) { unpack(raw(p), v); }
};

// ----------------------------------------------------------------------------------
// Token embedding x[row, f] = sum_i W_emb[f, i] * z[i], z = history token of P values (fp32;
// P here is the input token length P_in).  grid = (M rows, ceil(d / 128)), block = 128: one
// output feature per thread, its weight row read with independent 16-byte loads when P is a
// multiple of the vector width, element by element for short tokens (point tokens: P = 1).
// ----------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128)
embed_kernel(const float *hist, PassGeom g, int P, int d, const T *__restrict__ W,
             float *__restrict__ x, unsigned long long *__restrict__ stamp,
             const float *__restrict__ gain, T *__restrict__ a_out, float *__restrict__ ssq_out, int opens_round) {
  extern __shared__ float zs[];
  constexpr int V = Vec16<T>::N, PRE = 12;                     // weight vectors fetched before the wait
  const int row = blockIdx.x, slot = row / g.q_len, j = row % g.q_len;
  const int f = blockIdx.y * 128 + threadIdx.x;
  // Before the dependency wait: what does not depend on the preceding kernel -- the start of this
  // thread's weight row, its gain, and (unless this pass opens a round, when the kernel that closed
  // the previous round is the predecessor itself) the slot lookup.
  const T *wr = W + (size_t)min(f, d - 1) * P;
  typename Vec16<T>::Raw wpre[PRE];
  if (P % V == 0) {
#pragma unroll
    for (int k = 0; k < PRE; ++k)
      if (k * V < P) wpre[k] = Vec16<T>::raw(wr + k * V);
  }
  const float gf = a_out ? gain[min(f, d - 1)] : 0.f;
  SlotPos sp;
  if (!opens_round) sp = slot_lookup(g, slot);
  pdl_sync();
  if (stamp && row == 0 && blockIdx.y == 0 && threadIdx.x == 0) *stamp = globaltimer_ns();
  if (opens_round) sp = slot_lookup(g, slot);
  if (sp.dead) return;
  const int b = sp.b;
  const float *z = hist + ((size_t)b * g.cap + sp.p0 + j) * P;
  for (int i = threadIdx.x; i < P; i += blockDim.x) zs[i] = z[i];
  __syncthreads();
  if (f >= d) return;
  float acc = 0.f;
  if (P % V == 0) {
#pragma unroll
    for (int k = 0; k < PRE; ++k)
      if (k * V < P) {
        float w[V];
        Vec16<T>::unpack(wpre[k], w);
#pragma unroll
        for (int c = 0; c < V; ++c) acc = fmaf(w[c], zs[k * V + c], acc);
      }
#pragma unroll 4
    for (int i = PRE * V; i < P; i += V) {
      float w[V];
      Vec16<T>::load(wr + i, w);
#pragma unroll
      for (int c = 0; c < V; ++c) acc = fmaf(w[c], zs[i + c], acc);
    }
  } else {
    for (int i = 0; i < P; ++i) acc = fmaf(to_f32(wr[i]), zs[i], acc);
  }
  x[(size_t)row * d + f] = acc;
  if (a_out) {            // operand of the first contraction, normalised later (see SkNorm); d % 64 == 0
    a_out[(size_t)row * d + f] = from_f32<T>(gf * acc);
    float sq = acc * acc;                                       // sums of squares over slices of 16 features
    sq += __shfl_xor_sync(0xffffffffu, sq, 1);
    sq += __shfl_xor_sync(0xffffffffu, sq, 2);
    sq += __shfl_xor_sync(0xffffffffu, sq, 4);
    sq += __shfl_xor_sync(0xffffffffu, sq, 8);
    if ((threadIdx.x & 15) == 0) ssq_out[(size_t)row * (d >> 4) + (f >> 4)] = sq;
  }
}

// The same embedding for passes of many rows: 8 rows per CTA share every weight load.
// grid = (ceil(M / 8), ceil(d / 128)), block = 128, dynamic shared memory 8 * P floats.
template <typename T>
__global__ void __launch_bounds__(128)
embed_rows_kernel(const float *hist, PassGeom g, int M, int P, int d, const T *__restrict__ W,
                  float *__restrict__ x, unsigned long long *__restrict__ stamp) {
  constexpr int R = 8;
  extern __shared__ float zs[];                               // [R][P]
  pdl_sync();
  const int row0 = blockIdx.x * R;
  if (stamp && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *stamp = globaltimer_ns();
  if (slot_dead(g, row0 / g.q_len)) return;                   // every row of this CTA is past the live ones
  for (int i = threadIdx.x; i < R * P; i += blockDim.x) {
    const int row = row0 + i / P;
    float v = 0.f;
    if (row < M && !slot_dead(g, row / g.q_len)) {
      const int b = series_of(g, row / g.q_len), j = row % g.q_len;
      v = hist[((size_t)b * g.cap + pos0_of(g, b) + j) * P + i % P];
    }
    zs[i] = v;
  }
  __syncthreads();
  const int f = blockIdx.y * 128 + threadIdx.x;
  if (f >= d) return;
  const T *wr = W + (size_t)f * P;
  constexpr int V = Vec16<T>::N;
  float acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.f;
  if (P % V == 0) {
#pragma unroll 2
    for (int i = 0; i < P; i += V) {
      float w[V];
      Vec16<T>::load(wr + i, w);
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < V; ++c) acc[r] = fmaf(w[c], zs[r * P + i + c], acc[r]);
    }
  } else {
    for (int i = 0; i < P; ++i) {
      const float w1 = to_f32(wr[i]);
#pragma unroll
      for (int r = 0; r < R; ++r) acc[r] = fmaf(w1, zs[r * P + i], acc[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
    if (row0 + r < M) x[(size_t)(row0 + r) * d + f] = acc[r];
}

// ----------------------------------------------------------------------------------
// RMSNorm: a[row, :] = g * x / sqrt(mean(x^2) + eps), rounded to T.  One warp per row, 8 rows
// per CTA (grid = ceil(M / 8), block = 256): the row is read once with 16-byte loads and kept in
// registers (rows of up to 2048 features; longer rows are read a second time), reduced with
// shuffles only, and written with 16-byte (fp32) or 8-byte (bf16) stores.  d is a multiple of 4.
// ----------------------------------------------------------------------------------
__device__ __forceinline__ void store4(float *o, float a, float b, float c, float d4) {
  *reinterpret_cast<float4 *>(o) = make_float4(a, b, c, d4);
}
__device__ __forceinline__ void store4(bf16 *o, float a, float b, float c, float d4) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d4);
  uint2 pk;
  pk.x = *reinterpret_cast<const uint32_t *>(&lo);
  pk.y = *reinterpret_cast<const uint32_t *>(&hi);
  *reinterpret_cast<uint2 *>(o) = pk;
}

// EARLY (passes of up to a few thousand rows, where the launch is a link in a chain and not a
// stream of bytes): the gain and the live-row count are fetched before the dependency wait, which
// takes two L2 round trips out of the chain at the price of registers (rows of at most 1280
// features, so that two CTAs still fit on an SM).  The count was written by the kernel that closed
// the previous round, at least two kernels back.
template <typename T, bool EARLY>
__global__ void __launch_bounds__(256, 2)
rmsnorm_kernel(const float *x, const float *__restrict__ gain, int M, int d, float eps,
               T *__restrict__ a, LiveRows lr) {
  constexpr int CACHE = EARLY ? 10 : 16;                      // float4 per lane kept in registers
  const int lane = threadIdx.x & 31;
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const float4 *gr = reinterpret_cast<const float4 *>(gain);
  const int nv = d / 4;
  float4 gpre[EARLY ? CACHE : 1];
  if (EARLY) {
    if (lr.n_live) M = min(M, *reinterpret_cast<const volatile int *>(lr.n_live) * lr.q_len);
    if (row >= (size_t)M) return;
#pragma unroll
    for (int k = 0; k < CACHE; ++k)
      if (lane + 32 * k < nv) gpre[EARLY ? k : 0] = gr[lane + 32 * k];
  }
  pdl_sync();
  if (!EARLY && row >= (size_t)live_rows(lr, M)) return;
  const float4 *xr = reinterpret_cast<const float4 *>(x + row * d);
  float4 v[CACHE];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < CACHE; ++k) {
    const int i = lane + 32 * k;
    if (i < nv) {
      v[k] = xr[i];
      ss = fmaf(v[k].x, v[k].x, fmaf(v[k].y, v[k].y, fmaf(v[k].z, v[k].z, fmaf(v[k].w, v[k].w, ss))));
    }
  }
  for (int i = lane + 32 * CACHE; i < nv; i += 32) {
    const float4 u = xr[i];
    ss = fmaf(u.x, u.x, fmaf(u.y, u.y, fmaf(u.z, u.z, fmaf(u.w, u.w, ss))));
  }
  const float rstd = rsqrtf(warp_sum(ss) / d + eps);
  T *ar = a + row * d;
#pragma unroll
  for (int k = 0; k < CACHE; ++k) {
    const int i = lane + 32 * k;
    if (i < nv) {
      const float4 gg = EARLY ? gpre[EARLY ? k : 0] : gr[i];
      store4(ar + 4 * i, gg.x * v[k].x * rstd, gg.y * v[k].y * rstd, gg.z * v[k].z * rstd, gg.w * v[k].w * rstd);
    }
  }
  for (int i = lane + 32 * CACHE; i < nv; i += 32) {
    const float4 u = xr[i], gg = gr[i];
    store4(ar + 4 * i, gg.x * u.x * rstd, gg.y * u.y * rstd, gg.z * u.z * rstd, gg.w * u.w * rstd);
  }
}

// ----------------------------------------------------------------------------------
// FMA GEMM  C[M, N] (op)= A[M, K] . W[N, K]^T, fp32 accumulate.  64x64 tile, BK = 16,
// 256 threads, 4x4 outputs per thread.  K must be a multiple of 16.
// Epilogues: store fp32 | store T | GELU -> T | residual add into fp32.
// ----------------------------------------------------------------------------------
enum { EPI_F32 = 0, EPI_T = 1, EPI_GELU_T = 2, EPI_RESID = 3, EPI_ATOMIC = 4 };   // ATOMIC: fp32 atomic add

template <typename T, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T *A, const T *__restrict__ W, void *Cout,
                 int M, int N, int K) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const int tid = threadIdx.x;
  pdl_sync();
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int lr = tid >> 2;          // 0..63: tile row loaded by this thread
  const int lk = (tid & 3) * 4;     // 0,4,8,12: first of 4 k's loaded
  const int tm = (tid >> 4) * 4;    // output rows tm..tm+3
  const int tn = (tid & 15) * 4;    // output cols tn..tn+3
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += 16) {
    float av[4], wv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      av[i] = (m0 + lr < M) ? to_f32(A[(size_t)(m0 + lr) * K + k0 + lk + i]) : 0.f;
      wv[i] = (n0 + lr < N) ? to_f32(W[(size_t)(n0 + lr) * K + k0 + lk + i]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lr] = av[i];
      Ws[lk + i][lr] = wv[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a4[4], w4[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a4[i] = As[kk][tm + i];
        w4[i] = Ws[kk][tn + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a4[i], w4[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + tm + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tn + j;
      if (n >= N) continue;
      const size_t o = (size_t)m * N + n;
      if (EPI == EPI_F32) ((float *)Cout)[o] = acc[i][j];
      else if (EPI == EPI_T) ((T *)Cout)[o] = from_f32<T>(acc[i][j]);
      else if (EPI == EPI_GELU_T) ((T *)Cout)[o] = from_f32<T>(gelu_erf(acc[i][j]));
      else ((float *)Cout)[o] += acc[i][j];
    }
  }
}

// ----------------------------------------------------------------------------------
// RoPE + KV append + causal attention for one (head, series, query tile): the kernel of the
// fp32 caches (bf16 caches take attn_flash_kernel).
//   qkv   [M, 3 d] fp32: q | k | v of this pass's tokens (row = b * q_len + j)
//   Kc,Vc [B, heads, cap, DH] T: this layer's cache; positions < pos0 are valid
//   rope  [cap, DH/2] float2 (cos, sin), rotate-half pairing (i, i + DH/2)
//   out   [M, d] T
// The CTA loads keys 0..pos0-1 from the cache (16-byte asynchronous copies) and the keys of this
// pass (rotated here, or appended beforehand by kv_append_kernel when the pass has several query
// tiles) up to its last query into shared memory once; all queries of the tile share that read.
// The tile that owns a token writes its rotated key and its value to the cache.
// grid = (heads, B, ceil(q_len / QT) * skv), block = 128; the queries of a tile are processed
// together.  Shared memory is addressed in 32-bit words; key rows are dense with their 16-byte
// chunks rotated by the row index (attn_kword).
//   V tile [nk][VW] words, K tile [nk][KW] words, scores [16][nk] f32, q [16][DH] f32,
//   partial outputs [4][16][DH] f32, row maxima [16] and row sums [16] f32.
// ----------------------------------------------------------------------------------
template <typename T> struct AttnWords;                 // words per DH elements
template <> struct AttnWords<float> {
  static __host__ __device__ constexpr int per_row(int dh) { return dh; }
};
template <> struct AttnWords<bf16> {
  static __host__ __device__ constexpr int per_row(int dh) { return dh / 2; }
};
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}

// Key rows in shared memory are dense (VW words) with their 16-byte chunks rotated by the row
// index, so that 16-byte asynchronous copies land aligned and lanes that read the same logical
// word of consecutive rows spread over the banks.  Physical word of logical word w of row t:
template <int VW> __device__ __forceinline__ int attn_kword(int t, int w) {
  return t * VW + ((((w >> 2) + t) & (VW / 4 - 1)) << 2) + (w & 3);
}
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}

constexpr int ATTN_QT = 16;                             // queries per tile (at most)

// Scores, softmax and P.V of one query tile from shared memory.  All queries of the tile are
// processed together, so that every key and value row is read once for the whole tile:
// (1) scores, one key per thread, all queries; (2) softmax, one query per warp; (3) P.V with the
// keys dealt out over the four warps and each lane owning DH/32 output dims; (4) sum of the four
// partial outputs.  NQ = compile-time bound on the number of queries (loops are unrolled to it).
template <typename T, int DH, int NQ>
__device__ __forceinline__ void attn_tile(const uint32_t *Ks, const uint32_t *Vs, float *sc, const float *qs, float *po,
                                          float *row_max, float *row_sum, int nq, int nk, int nk_max, int k_lo,
                                          int p0, int j_lo) {
  constexpr bool BF = sizeof(T) == 2;
  constexpr int VW = AttnWords<T>::per_row(DH), DPL = DH / 32;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, tid = threadIdx.x;
  for (int t = tid; t < nk; t += blockDim.x) {
    float sacc[NQ];
#pragma unroll
    for (int i = 0; i < NQ; ++i) sacc[i] = 0.f;
    if (BF) {
#pragma unroll 4
      for (int c = 0; c < DH / 2; ++c) {
        const uint32_t kk = Ks[attn_kword<VW>(t, c)];
        const float k0 = __uint_as_float(kk << 16), k1 = __uint_as_float(kk & 0xffff0000u);
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
          const float2 qq = *reinterpret_cast<const float2 *>(qs + i * DH + 2 * c);
          sacc[i] = fmaf(qq.x, k0, fmaf(qq.y, k1, sacc[i]));
        }
      }
    } else {
#pragma unroll 4
      for (int c = 0; c < DH; ++c) {
        const float kf = __uint_as_float(Ks[attn_kword<VW>(t, c)]);
#pragma unroll
        for (int i = 0; i < NQ; ++i) sacc[i] = fmaf(qs[i * DH + c], kf, sacc[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < NQ; ++i)
      if (i < nq) sc[(size_t)i * nk_max + t] = (k_lo + t <= p0 + j_lo + i) ? sacc[i] : -INFINITY;   // causal mask
  }
  __syncthreads();
  for (int i = w; i < nq; i += 4) {
    float *row = sc + (size_t)i * nk_max;
    float mx = -INFINITY;
    for (int t = lane; t < nk; t += 32) mx = fmaxf(mx, row[t]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int t = lane; t < nk; t += 32) {
      const float pv = mx == -INFINITY ? 0.f : expf(row[t] - mx);   // no visible key in this CTA's range
      row[t] = pv;
      sum += pv;
    }
    sum = warp_sum(sum);
    if (lane == 0) { row_max[i] = mx; row_sum[i] = sum; }
  }
  __syncthreads();
  float acc[NQ][DPL];
#pragma unroll
  for (int i = 0; i < NQ; ++i)
#pragma unroll
    for (int c = 0; c < DPL; ++c) acc[i][c] = 0.f;
#pragma unroll 2
  for (int t = w; t < nk; t += 4) {
    float v[DPL];
    if (BF) {
      if (DPL == 1) {                                // DH = 32: half a word per lane
        const uint32_t vv = Vs[(size_t)t * VW + lane / 2];
        v[0] = __uint_as_float((lane & 1) ? (vv & 0xffff0000u) : (vv << 16));
      } else {
#pragma unroll
        for (int c = 0; c < DPL / 2; ++c) {
          const uint32_t vv = Vs[(size_t)t * VW + lane * (DPL / 2) + c];
          v[2 * c] = __uint_as_float(vv << 16);
          v[2 * c + (DPL > 1 ? 1 : 0)] = __uint_as_float(vv & 0xffff0000u);
        }
      }
    } else {
#pragma unroll
      for (int c = 0; c < DPL; ++c) v[c] = __uint_as_float(Vs[(size_t)t * VW + lane * DPL + c]);
    }
#pragma unroll
    for (int i = 0; i < NQ; ++i) {
      const float pv = sc[(size_t)i * nk_max + t];     // rows >= nq hold stale but finite-or-not values: never stored
#pragma unroll
      for (int c = 0; c < DPL; ++c) acc[i][c] = fmaf(pv, v[c], acc[i][c]);
    }
  }
#pragma unroll
  for (int i = 0; i < NQ; ++i)
    if (i < nq)
#pragma unroll
      for (int c = 0; c < DPL; ++c) po[((size_t)w * ATTN_QT + i) * DH + lane * DPL + c] = acc[i][c];
  __syncthreads();
}

// Warp-level tensor-core helpers (mma.sync m16n8k16, bf16 operands, fp32 accumulate) and the
// split of an fp32 pair into bf16 high and low parts, used by the bf16 attention kernel.
__device__ __forceinline__ void mma_bf16_16816(float *c, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split_bf16x2(float x, float y, uint32_t &hi, uint32_t &lo) {
  const float xh = __bfloat162float(__float2bfloat16_rn(x)), yh = __bfloat162float(__float2bfloat16_rn(y));
  hi = pack_bf16x2(xh, yh);
  lo = pack_bf16x2(x - xh, y - yh);
}

// Keys and values of a pass with several query tiles go to the cache once, before attention:
// rotated key and value of token j of series b, head h, to cache row pos0 + j.  Every tile of
// attn_kernel (launched with pre = 1) then finds all keys of the pass in the cache instead of
// rotating the earlier tiles' keys again.  grid = (heads, B, ceil(q_len / 16)), block = 128.
template <typename T, int DH>
__global__ void __launch_bounds__(128)
kv_append_kernel(const float *qkv, T *__restrict__ Kc, T *__restrict__ Vc,
                 const float2 *__restrict__ rope, PassGeom g, int n_heads) {
  constexpr int HALF = DH / 2;
  const int h = blockIdx.x, slot = blockIdx.y, d = n_heads * DH;
  const SlotPos sp = slot_lookup(g, slot);                      // before the dependency wait: see SlotPos
  pdl_sync();
  if (sp.dead) return;
  const int b = sp.b, p0 = sp.p0;
  const int j_lo = blockIdx.z * 16, j_hi = min(g.q_len, j_lo + 16);
  const size_t row0 = (size_t)slot * g.q_len;
  T *Kb = Kc + ((size_t)b * n_heads + h) * g.cap * DH;
  T *Vb = Vc + ((size_t)b * n_heads + h) * g.cap * DH;
  for (int i = threadIdx.x; i < (j_hi - j_lo) * (HALF / 2); i += blockDim.x) {
    const int j = j_lo + i / (HALF / 2), c = (i % (HALF / 2)) * 2;
    const float *src = qkv + (row0 + j) * 3 * d + h * DH;
    const int tg = p0 + j;
    const float4 cs = *reinterpret_cast<const float4 *>(rope + (size_t)tg * HALF + c);   // cos0 sin0 cos1 sin1
    const float2 ka = *reinterpret_cast<const float2 *>(src + d + c);
    const float2 kb = *reinterpret_cast<const float2 *>(src + d + c + HALF);
    const float2 va = *reinterpret_cast<const float2 *>(src + 2 * d + c);
    const float2 vb = *reinterpret_cast<const float2 *>(src + 2 * d + c + HALF);
    const float r1a = ka.x * cs.x - kb.x * cs.y, r1b = ka.y * cs.z - kb.y * cs.w;    // first half
    const float r2a = kb.x * cs.x + ka.x * cs.y, r2b = kb.y * cs.z + ka.y * cs.w;    // second half
    if (sizeof(T) == 2) {
      uint32_t *kg = reinterpret_cast<uint32_t *>(Kb + (size_t)tg * DH);
      uint32_t *vg = reinterpret_cast<uint32_t *>(Vb + (size_t)tg * DH);
      kg[c / 2] = pack_bf16x2(r1a, r1b); kg[(c + HALF) / 2] = pack_bf16x2(r2a, r2b);
      vg[c / 2] = pack_bf16x2(va.x, va.y); vg[(c + HALF) / 2] = pack_bf16x2(vb.x, vb.y);
    } else {
      float *kg = reinterpret_cast<float *>(Kb + (size_t)tg * DH);
      float *vg = reinterpret_cast<float *>(Vb + (size_t)tg * DH);
      kg[c] = r1a; kg[c + 1] = r1b; kg[c + HALF] = r2a; kg[c + HALF + 1] = r2b;
      vg[c] = va.x; vg[c + 1] = va.y; vg[c + HALF] = vb.x; vg[c + HALF + 1] = vb.y;
    }
  }
}

// Thread-block-cluster helpers of the key-split attention: every CTA of a cluster reaches
// attn_cluster_sync the same number of times; attn_peer_f32 reads one float of a peer CTA's
// shared memory at the same offset as `local`.
__device__ __forceinline__ void attn_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float attn_peer_f32(const float *local, uint32_t rank) {
  uint32_t remote;
  float v;
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(a), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

// skv = 1: one CTA holds every key of its (series, head).  skv > 1: the launch carries a cluster
// of skv CTAs along z (blockIdx.z = tile * skv + rank); rank r holds the keys
// [r * chunk, (r + 1) * chunk) of the row, chunk a multiple of 16, computes the softmax
// numerator, its row maxima and row sums over them, and the ranks combine the pieces through
// distributed shared memory: m = max_r m_r, l = sum_r l_r e^(m_r - m), o = sum_r o_r e^(m_r - m) / l.
// nk_max is the number of key rows one CTA can hold.  pre = 1: kv_append_kernel has already put
// the keys and values of this pass into the cache.
template <typename T, int DH>
__global__ void __launch_bounds__(128)
attn_kernel(const float *qkv, T *Kc, T *Vc,
            const float2 *__restrict__ rope, PassGeom g, int n_heads, int QT, int nk_max, int skv, int pre,
            T *__restrict__ out) {
  constexpr bool BF = sizeof(T) == 2;
  constexpr int VW = AttnWords<T>::per_row(DH);   // words per value row
  constexpr int KW = VW;                          // dense key row, chunks rotated (attn_kword)
  constexpr int HALF = DH / 2;
  constexpr int EPV = 16 / sizeof(T);             // elements per 16-byte vector
  extern __shared__ __align__(16) uint32_t smem_w[];
  uint32_t *Vs = smem_w;                          // [nk_max][VW], 16-byte aligned rows
  uint32_t *Ks = Vs + (size_t)nk_max * VW;        // [nk_max][KW]
  float *sc = reinterpret_cast<float *>(Ks + (size_t)nk_max * KW);
  float *qs = sc + (size_t)ATTN_QT * nk_max;        // [ATTN_QT][DH] rotated, scaled queries
  float *po = qs + ATTN_QT * DH;                    // [4][ATTN_QT][DH] partial outputs per warp
  float *row_max = po + 4 * ATTN_QT * DH;           // [ATTN_QT] maximum score over this CTA's keys
  float *row_sum = row_max + ATTN_QT;               // [ATTN_QT] sum of exp(score - row_max)

  const int h = blockIdx.x, slot = blockIdx.y;
  const int qt = skv > 1 ? blockIdx.z / skv : blockIdx.z;
  const int rank = skv > 1 ? blockIdx.z % skv : 0;   // == %cluster_ctarank: the cluster spans z only
  const int d = n_heads * DH;
  const SlotPos sp = slot_lookup(g, slot);           // before the dependency wait: see SlotPos
  pdl_sync();
  if (sp.dead) return;                               // the whole cluster (same y) leaves together
  const int b = sp.b, p0 = sp.p0;
  const int j_lo = qt * QT;
  const int j_hi = min(g.q_len, j_lo + QT);          // queries [j_lo, j_hi)
  const size_t row0 = (size_t)slot * g.q_len;
  const int nk_all = p0 + j_hi;                      // keys visible to the tile's last query
  const int chunk = skv > 1 ? (((nk_all + skv - 1) / skv + 15) & ~15) : nk_all;
  const int k_lo = min(rank * chunk, nk_all);        // this CTA holds keys [k_lo, k_hi) at rows t - k_lo
  const int k_hi = min(k_lo + chunk, nk_all);
  T *Kb = Kc + ((size_t)b * n_heads + h) * g.cap * DH;
  T *Vb = Vc + ((size_t)b * n_heads + h) * g.cap * DH;

  // cached keys/values: p0 rows of DH elements as 16-byte asynchronous copies, all issued up
  // front (the cache comes from HBM: the copy is bound by the bytes in flight)
  {
    constexpr int VPR = DH / EPV;                    // 16-byte chunks per row
    const int nvec = max(min(k_hi, pre ? nk_all : p0) - k_lo, 0) * VPR;
    const T *Kg = Kb + (size_t)k_lo * DH, *Vg = Vb + (size_t)k_lo * DH;
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
      const int t = i / VPR, c = i % VPR;
      cp_async16(Ks + (size_t)t * VW + (((c + t) & (VPR - 1)) << 2), Kg + (size_t)i * EPV);
      cp_async16(Vs + (size_t)i * 4, Vg + (size_t)i * EPV);
    }
  }
  // keys/values of this pass (rotate keys; the owning tile appends to the cache).
  // One thread handles the element pair (c, c + 1) of the first half and its rotation partners.
  for (int i = threadIdx.x; i < (pre ? 0 : j_hi * (HALF / 2)); i += blockDim.x) {
    const int j = i / (HALF / 2), c = (i % (HALF / 2)) * 2;
    const float *src = qkv + (row0 + j) * 3 * d + h * DH;
    const int tg = p0 + j, t = tg - k_lo;            // position in the row, row in this CTA
    if (tg < k_lo || tg >= k_hi) continue;
    const float4 cs = *reinterpret_cast<const float4 *>(rope + (size_t)tg * HALF + c);   // cos0 sin0 cos1 sin1
    const float2 ka = *reinterpret_cast<const float2 *>(src + d + c);
    const float2 kb = *reinterpret_cast<const float2 *>(src + d + c + HALF);
    const float2 va = *reinterpret_cast<const float2 *>(src + 2 * d + c);
    const float2 vb = *reinterpret_cast<const float2 *>(src + 2 * d + c + HALF);
    const float r1a = ka.x * cs.x - kb.x * cs.y, r1b = ka.y * cs.z - kb.y * cs.w;    // first half
    const float r2a = kb.x * cs.x + ka.x * cs.y, r2b = kb.y * cs.z + ka.y * cs.w;    // second half
    if (BF) {
      const uint32_t k1 = pack_bf16x2(r1a, r1b), k2 = pack_bf16x2(r2a, r2b);
      const uint32_t v1 = pack_bf16x2(va.x, va.y), v2 = pack_bf16x2(vb.x, vb.y);
      Ks[attn_kword<VW>(t, c / 2)] = k1;
      Ks[attn_kword<VW>(t, (c + HALF) / 2)] = k2;
      Vs[(size_t)t * VW + c / 2] = v1;
      Vs[(size_t)t * VW + (c + HALF) / 2] = v2;
      if (j >= j_lo) {
        uint32_t *kg = reinterpret_cast<uint32_t *>(Kb + (size_t)tg * DH);
        uint32_t *vg = reinterpret_cast<uint32_t *>(Vb + (size_t)tg * DH);
        kg[c / 2] = k1; kg[(c + HALF) / 2] = k2;
        vg[c / 2] = v1; vg[(c + HALF) / 2] = v2;
      }
    } else {
      float *kf = reinterpret_cast<float *>(Ks);
      float *vf = reinterpret_cast<float *>(Vs + (size_t)t * VW);
      kf[attn_kword<VW>(t, c)] = r1a; kf[attn_kword<VW>(t, c + 1)] = r1b;
      kf[attn_kword<VW>(t, c + HALF)] = r2a; kf[attn_kword<VW>(t, c + HALF + 1)] = r2b;
      vf[c] = va.x; vf[c + 1] = va.y; vf[c + HALF] = vb.x; vf[c + HALF + 1] = vb.y;
      if (j >= j_lo) {
        float *kg = reinterpret_cast<float *>(Kb + (size_t)tg * DH);
        float *vg = reinterpret_cast<float *>(Vb + (size_t)tg * DH);
        kg[c] = r1a; kg[c + 1] = r1b; kg[c + HALF] = r2a; kg[c + HALF + 1] = r2b;
        vg[c] = va.x; vg[c + 1] = va.y; vg[c + HALF] = vb.x; vg[c + HALF + 1] = vb.y;
      }
    }
  }

  const int tid = threadIdx.x;
  const float scale = rsqrtf((float)DH);
  const int nq = j_hi - j_lo;                        // <= ATTN_QT
  const int nk = k_hi - k_lo;                        // key rows held here
  // rows the tile routine will touch: its compile-time query bound
  const int nqb = nq <= 2 ? nq : nq <= 4 ? 4 : nq <= 6 ? 6 : nq <= 9 ? 9 : ATTN_QT;
  for (int idx = tid; idx < nqb * HALF; idx += blockDim.x) {       // rotated, scaled queries (zero past nq)
    const int i = idx / HALF, c = idx % HALF, j = j_lo + i;
    float r1 = 0.f, r2 = 0.f;
    if (i < nq) {
      const float *src = qkv + (row0 + j) * 3 * d + h * DH;
      const float2 cs = rope[(size_t)(p0 + j) * HALF + c];
      const float q1 = src[c], q2 = src[c + HALF];
      r1 = (q1 * cs.x - q2 * cs.y) * scale;
      r2 = (q2 * cs.x + q1 * cs.y) * scale;
    }
    qs[i * DH + c] = r1;
    qs[i * DH + c + HALF] = r2;
  }
  for (int idx = tid + nq * nk_max; idx < nqb * nk_max; idx += blockDim.x) sc[idx] = 0.f;       // unused score rows
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  if (nq == 1) attn_tile<T, DH, 1>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  else if (nq == 2) attn_tile<T, DH, 2>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  else if (nq <= 4) attn_tile<T, DH, 4>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  else if (nq <= 6) attn_tile<T, DH, 6>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  else if (nq <= 9) attn_tile<T, DH, 9>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  else attn_tile<T, DH, ATTN_QT>(Ks, Vs, sc, qs, po, row_max, row_sum, nq, nk, nk_max, k_lo, p0, j_lo);
  // the tile routines end on a block barrier: po holds each warp's unnormalised partial output

  if (skv <= 1) {
    for (int idx = tid; idx < nq * DH; idx += blockDim.x) {
      const int i = idx / DH, c = idx % DH;
      const float o = po[(size_t)(0 * ATTN_QT + i) * DH + c] + po[(size_t)(1 * ATTN_QT + i) * DH + c] +
                      po[(size_t)(2 * ATTN_QT + i) * DH + c] + po[(size_t)(3 * ATTN_QT + i) * DH + c];
      out[(row0 + j_lo + i) * d + h * DH + c] = from_f32<T>(o / row_sum[i]);
    }
    return;
  }
  // key-split: fold the four warps' partials into qs (the queries are no longer needed), then
  // rank (i mod skv) combines query i over the cluster
  for (int idx = tid; idx < nq * DH; idx += blockDim.x) {
    const int i = idx / DH, c = idx % DH;
    qs[idx] = po[(size_t)(0 * ATTN_QT + i) * DH + c] + po[(size_t)(1 * ATTN_QT + i) * DH + c] +
              po[(size_t)(2 * ATTN_QT + i) * DH + c] + po[(size_t)(3 * ATTN_QT + i) * DH + c];
  }
  attn_cluster_sync();
  for (int idx = tid; idx < nq * DH; idx += blockDim.x) {
    const int i = idx / DH, c = idx % DH;
    if (i % skv != rank) continue;
    float m = -INFINITY;
    for (int r = 0; r < skv; ++r) m = fmaxf(m, attn_peer_f32(row_max + i, r));
    float l = 0.f, o = 0.f;
    for (int r = 0; r < skv; ++r) {
      const float mr = attn_peer_f32(row_max + i, r);
      if (mr == -INFINITY) continue;               // that rank saw no visible key of this query
      const float w = expf(mr - m);
      l = fmaf(attn_peer_f32(row_sum + i, r), w, l);
      o = fmaf(attn_peer_f32(qs + idx, r), w, o);
    }
    out[(row0 + j_lo + i) * d + h * DH + c] = from_f32<T>(o / l);
  }
  attn_cluster_sync();                               // no CTA leaves while a peer still reads its shared memory
}

// ----------------------------------------------------------------------------------
// Final RMSNorm + mean head for selected tokens: o = W_head[P, d] . (g_f * x * rstd).
// Normalised activations stay fp32 here.  grid = (rows, ceil(P / 8)), block = 256: each warp
// produces one output element with 16-byte weight loads.
// only_last = 1: one row per series, the pass's last token, written behind the pass in the
//   series' history: the P values from token pos0 + q_len on (tok_len values per token)
//   (draft steps, target-only steps);
// only_last = 0: the boundary tokens head_step - 1, 2 head_step - 1, ... of the pass, boundary i
//   written to vout[b, i, :]  (verification; vout [B, q_len / head_step, P]); grid.x = B * that.
// ----------------------------------------------------------------------------------
__device__ float head_normal(const DevState *st, int series, int k_pos, int e);   // accept.cuh

template <typename T>
__global__ void __launch_bounds__(256)
head_kernel(const float *x, const float *__restrict__ gain, const T *__restrict__ Wh, int d,
            int P, float eps, PassGeom g, int only_last, float *__restrict__ hist,
            float *__restrict__ vout, const DevState *st, float *__restrict__ muq, int k_pos, int K,
            int tok_len) {
  extern __shared__ __align__(16) float xs[];
  __shared__ float red[32];
  constexpr int V = Vec16<T>::N, WPRE = 6, GPRE = 6;   // weight vectors per lane / gains per thread fetched early
  const int nb = g.q_len / g.head_step;                // boundaries per series
  int slot, j, ib = 0;
  if (only_last) { slot = blockIdx.x; j = g.q_len - 1; }
  else { slot = blockIdx.x / nb; ib = blockIdx.x % nb; j = (ib + 1) * g.head_step - 1; }
  const SlotPos sp = slot_lookup(g, slot);             // before the dependency wait: see SlotPos
  // also before the wait: the constants this thread needs -- the start of its warp's weight row and
  // its gains (two L2 round trips that would otherwise follow the normalisation one after the other)
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int p = blockIdx.y * 8 + w;
  const T *wr = Wh + (size_t)min(p, P - 1) * d;
  typename Vec16<T>::Raw wpre[WPRE];
  float gpre[GPRE];
#pragma unroll
  for (int k = 0; k < WPRE; ++k)
    if ((lane + 32 * k) * V < d) wpre[k] = Vec16<T>::raw(wr + (lane + 32 * k) * V);
#pragma unroll
  for (int k = 0; k < GPRE; ++k)
    if ((int)threadIdx.x + 256 * k < d) gpre[k] = gain[threadIdx.x + 256 * k];
  pdl_sync();
  if (sp.dead) return;
  const int b = sp.b;
  const float *xr = x + ((size_t)slot * g.q_len + j) * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = xr[i];
    xs[i] = v;
    ss = fmaf(v, v, ss);
  }
  const float rstd = rsqrtf(block_sum(ss, red) / d + eps);
#pragma unroll
  for (int k = 0; k < GPRE; ++k)
    if ((int)threadIdx.x + 256 * k < d) xs[threadIdx.x + 256 * k] = gpre[k] * xs[threadIdx.x + 256 * k] * rstd;
  for (int i = threadIdx.x + 256 * GPRE; i < d; i += blockDim.x) xs[i] = gain[i] * xs[i] * rstd;
  __syncthreads();
  float *dst = only_last ? hist + ((size_t)b * g.cap + sp.p0 + g.q_len) * tok_len
                         : vout + ((size_t)b * nb + ib) * P;
  if (p >= P) return;
  float acc = 0.f;
#pragma unroll
  for (int k = 0; k < WPRE; ++k) {
    const int i = (lane + 32 * k) * V;
    if (i < d) {
      float wv[V];
      Vec16<T>::unpack(wpre[k], wv);
#pragma unroll
      for (int c = 0; c < V; ++c) acc = fmaf(wv[c], xs[i + c], acc);
    }
  }
  for (int i = (lane + 32 * WPRE) * V; i < d; i += 32 * V) {
    float wv[V];
    Vec16<T>::load(wr + i, wv);
#pragma unroll
    for (int c = 0; c < V; ++c) acc = fmaf(wv[c], xs[i + c], acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) {
    if (only_last && st && (st->flags & VAR_SAMPLE_PROPOSALS)) {
      // sampled proposal x = mu_q + sigma_q eps (Sec. 3.3); the mean is kept for the statistic
      muq[((size_t)b * K + k_pos) * P + p] = acc;
      acc += st->sigma_q * head_normal(st, b, k_pos, p);
    }
    dst[p] = acc;
  }
}

// The head for the boundary tokens of a pass of many rows (verification: vout[b, i, :]): 8 rows
// per CTA (one warp normalises one row into shared memory), then each warp produces 4 of the CTA's
// 32 outputs for all 8 rows, so that a weight vector is loaded once per 8 rows.  M counts boundary
// rows (series x boundaries per series).
// grid = (ceil(M / 8), ceil(P / 32)), block = 256, dynamic shared memory 8 * d floats.
template <typename T>
__global__ void __launch_bounds__(256)
head_rows_kernel(const float *x, const float *__restrict__ gain, const T *__restrict__ Wh, int M,
                 int d, int P, float eps, float *__restrict__ vout, PassGeom g) {
  constexpr int R = 8;
  extern __shared__ __align__(16) float xs[];                  // [R][d] normalised rows
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int row0 = blockIdx.x * R;
  const int nb = g.q_len / g.head_step;                        // boundaries per series
  // live rows: read before the dependency wait (written when the previous round closed, a whole
  // pass of kernels back)
  if (g.n_live) M = min(M, *reinterpret_cast<const volatile int *>(g.n_live) * nb);
  if (row0 >= M) return;
  pdl_sync();
  {
    const int row = row0 + w;
    float *xw = xs + (size_t)w * d;
    float ss = 0.f;
    if (row < M) {
      const float *xr = x + ((size_t)(row / nb) * g.q_len + (row % nb + 1) * g.head_step - 1) * d;
      for (int i = lane; i < d; i += 32) {
        const float v = xr[i];
        xw[i] = v;
        ss = fmaf(v, v, ss);
      }
    } else {
      for (int i = lane; i < d; i += 32) xw[i] = 0.f;
    }
    const float rstd = rsqrtf(warp_sum(ss) / d + eps);
    for (int i = lane; i < d; i += 32) xw[i] = gain[i] * xw[i] * rstd;   // each lane rewrites what it wrote
  }
  __syncthreads();
  constexpr int V = Vec16<T>::N;
  for (int q = 0; q < 4; ++q) {
    const int p = blockIdx.y * 32 + q * 8 + w;
    if (p >= P) break;
    const T *wr = Wh + (size_t)p * d;
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;
    for (int i = lane * V; i < d; i += 32 * V) {
      float wv[V];
      Vec16<T>::load(wr + i, wv);
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < V; ++c) acc[r] = fmaf(wv[c], xs[(size_t)r * d + i + c], acc[r]);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float o = warp_sum(acc[r]);
      if (lane == 0 && row0 + r < M) {                         // vout is indexed by series, rows by slot
        const int row = row0 + r, b = series_of(g, row / nb);
        vout[((size_t)b * nb + row % nb) * P + p] = o;
      }
    }
  }
}

}  // namespace tsfm

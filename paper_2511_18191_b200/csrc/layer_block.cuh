// One launch for everything between two attention steps of a pass of a few tokens:
//
//     x += ao Wo^T ;  a = norm(x; g_mid) ;  x += W2 gelu(W1 a) ;  [ qkv_next = Wqkv_next norm(x; g_next) ]
//
// A pass of a few dozen tokens is a chain of dependent launches, and what each link costs is its
// latency, not its work (a draft step of C4 was 22 links of ~4.6 us for ~0.1 GFLOP).  This kernel
// replaces four of the five links of a layer (attention-output projection, MLP up, MLP down, the next
// layer's QKV projection) by one:
//   * the series of a pass are dealt out over clusters of R = n_heads CTAs (head size 64, so that
//     d / R = 64): a cluster owns up to 16 token rows -- series never interact -- and carries them
//     through all four contractions;
//   * inside a cluster CTA r owns a 1/R slice of every output (64 features of x, ff / R hidden units,
//     q / k / v of head r) and streams exactly the weight rows of its slices, as 64-column chunks
//     through a ring of asynchronous copies that keeps running across the four contractions (the
//     weights do not depend on the data, so the ring is primed BEFORE the dependency wait);
//   * what a contraction needs of its input -- all features of the cluster's rows -- is small (16 rows):
//     after each contraction the CTAs publish their slice (and the rows' partial sums of squares) in
//     their own shared memory, meet at a cluster barrier, and pull the other slices over distributed
//     shared memory with 16-byte loads;
//   * the arithmetic is mma.sync m16n8k16 (bf16 in, fp32 accumulate), each of the 8 warps owning
//     nf / 8 output features of the CTA's slice over the whole K: fixed summation order, no atomics.
// Every cluster reads every weight of the layer once from L2 (measured: all 148 SMs pull ~130 GB/s
// each, 19.7 TB/s together, from an L2-resident region), which is what bounds the launch: the
// weights of a layer / R per CTA at that rate.
//
// Shared memory: ring of 3 x 32 KB weight stages; ao rows [16][d], a rows [16][d], h rows [16][ff]
// (bf16, 16-byte chunks of a row XOR-ed with row & 7 for conflict-free ldmatrix); the CTA's published
// slices (a: [16][64], h: [16][ff / R] bf16; sums of squares [16]); the gathered sums [R][16]; rstd [16].
// grid = R x G CTAs, cluster (R, 1, 1), block = 256.
#pragma once
#include "common.cuh"
#include "kernels_simt.cuh"
#include "gemm_ws.cuh"

namespace tsfm {

constexpr int LB_ROWS = 16, LB_KC = 64, LB_STAGE = 32 * 1024, LB_NST = 3, LB_MAX_R = 8;

struct LbArgs {
  const bf16 *ao;            // [M][d] attention output of this layer
  float *x;                  // [M][d] residual stream, updated in place
  const bf16 *Wo, *W1, *W2;  // this layer: [d][d], [ff][d], [d][ff]
  const float *g_mid;        // gain of the norm between the two halves of the layer
  const float *g_next;       // gain of the next layer's first norm; NULL: last layer, no QKV stage
  const bf16 *Wqkv;          // next layer's [3d][d]
  float *qkv;                // [M][3d] fp32
  int d, ff, R;              // R = n_heads = cluster size; d = 64 R
  int q_len, Bg, B;          // tokens per series, series per cluster, series of the launch
  const int *n_live;         // live series (active-series compaction), or NULL
  float eps;
};

static inline int lb_smem_bytes(int d, int ff, int R) {
  return LB_NST * LB_STAGE + 2 * LB_ROWS * d * 2 + LB_ROWS * ff * 2 + LB_ROWS * 64 * 2 + LB_ROWS * (ff / R) * 2 +
         LB_ROWS * 4 + LB_MAX_R * LB_ROWS * 4 + LB_ROWS * 4 + 8 * LB_ROWS * 4 + 256;
}

__device__ __forceinline__ void lb_ldsm2(uint32_t addr, uint32_t &d0, uint32_t &d1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(d0), "=r"(d1) : "r"(addr));
}
__device__ __forceinline__ void lb_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void lb_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t lb_peer(uint32_t local, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
  return remote;
}
__device__ __forceinline__ uint4 lb_ld_peer16(uint32_t remote) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(remote) : "memory");
  return v;
}
__device__ __forceinline__ float lb_ld_peer_f32(uint32_t remote) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

// One 64-column chunk of a contraction: acc[t] (16 rows x 8 features, tile t of this warp's NT tiles) +=
// in[16][kc*64 .. +64] . Wchunk[feature][64]^T.  `in32` rows are row_bytes apart, `st32` rows 128 bytes.
template <int NT>
__device__ __forceinline__ void lb_chunk(float (&acc)[4][4], uint32_t in32, int row_bytes, int kc, uint32_t st32, int w,
                                         int lane) {
  const int a_row = lane & 15, a_chunk = lane >> 4;
  const int b_row = (lane & 7) + ((lane >> 4) & 1) * 8, b_chunk = (lane >> 3) & 1;
#pragma unroll
  for (int ks = 0; ks < LB_KC / 16; ++ks) {
    uint32_t a[4];
    ws_ldsm4(in32 + (uint32_t)(a_row * row_bytes + (((kc * 8 + ks * 2 + a_chunk) ^ (a_row & 7)) << 4)), a);
#pragma unroll
    for (int tp = 0; tp < NT / 2; ++tp) {
      const int fr = w * 8 * NT + tp * 16 + b_row;
      uint32_t b[4];
      ws_ldsm4(st32 + (uint32_t)(fr * 128 + (((ks * 2 + b_chunk) ^ (fr & 7)) << 4)), b);
      mma_bf16_16816(acc[2 * tp], a, b[0], b[1]);
      mma_bf16_16816(acc[2 * tp + 1], a, b[2], b[3]);
    }
    if (NT & 1) {
      const int fr = w * 8 * NT + (NT - 1) * 8 + (lane & 7);
      uint32_t b0, b1;
      lb_ldsm2(st32 + (uint32_t)(fr * 128 + (((ks * 2 + ((lane >> 3) & 1)) ^ (fr & 7)) << 4)), b0, b1);
      mma_bf16_16816(acc[NT - 1], a, b0, b1);
    }
  }
}

__global__ void __launch_bounds__(256, 1) layer_block_kernel(const LbArgs a) {
  extern __shared__ __align__(128) unsigned char lb_smem[];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int R = a.R, r = blockIdx.x % R, c = blockIdx.x / R;        // rank in the cluster (clusters span x), cluster index
  const int d = a.d, ff = a.ff, nfh = ff / R;                       // hidden units per CTA
  // rows of this cluster; the live count is read before the dependency wait (written by the kernel that
  // closed the previous round, at least two kernels back: see gemm_sk_kernel)
  const int n_series = a.n_live ? min(a.B, *reinterpret_cast<const volatile int *>(a.n_live)) : a.B;
  const int s0 = c * a.Bg;
  if (s0 >= n_series) return;                                       // the whole cluster leaves: no barrier is pending
  const int row0 = s0 * a.q_len, n_rows = min(a.Bg, n_series - s0) * a.q_len;

  unsigned char *ring = lb_smem;
  unsigned char *buf_ao = ring + LB_NST * LB_STAGE;                 // [16][d] bf16
  unsigned char *buf_a = buf_ao + LB_ROWS * d * 2;                  // [16][d] bf16
  unsigned char *buf_h = buf_a + LB_ROWS * d * 2;                   // [16][ff] bf16
  unsigned char *pub_a = buf_h + LB_ROWS * ff * 2;                  // [16][64] bf16   published slices
  unsigned char *pub_h = pub_a + LB_ROWS * 64 * 2;                  // [16][nfh] bf16
  float *pub_ssq = reinterpret_cast<float *>(pub_h + LB_ROWS * nfh * 2);   // [16]
  float *all_ssq = pub_ssq + LB_ROWS;                               // [R][16]
  float *rstd = all_ssq + LB_MAX_R * LB_ROWS;                       // [16]
  float *w_ssq = rstd + LB_ROWS;                                    // [8 warps][16]
  const uint32_t ring32 = (uint32_t)__cvta_generic_to_shared(ring);
  const uint32_t ao32 = (uint32_t)__cvta_generic_to_shared(buf_ao), a32 = (uint32_t)__cvta_generic_to_shared(buf_a);
  const uint32_t h32 = (uint32_t)__cvta_generic_to_shared(buf_h);

  // ---- the weight stream: chunk i of [Wo | W1 | W2 | Wqkv], each a [nf features][64 columns] block
  const int n1 = d / LB_KC, n2 = 2 * n1, n3 = n2 + ff / LB_KC, n4 = a.g_next ? n3 + n1 : n3;
  auto issue = [&](int i) {
    if (i < n4) {
      const bf16 *W;
      int K, nf, kc, kind;                                          // kind 0: contiguous rows from `base`; 1: q | k | v of head r
      int base;
      if (i < n1) { W = a.Wo; K = d; nf = 64; kc = i; kind = 0; base = r * 64; }
      else if (i < n2) { W = a.W1; K = d; nf = nfh; kc = i - n1; kind = 0; base = r * nfh; }
      else if (i < n3) { W = a.W2; K = ff; nf = 64; kc = i - n2; kind = 0; base = r * 64; }
      else { W = a.Wqkv; K = d; nf = 192; kc = i - n3; kind = 1; base = r * 64; }
      unsigned char *st = ring + (i % LB_NST) * LB_STAGE;
      for (int idx = tid; idx < nf * 8; idx += 256) {
        const int rr = idx >> 3, ch = idx & 7;
        const int grow = kind ? (rr >> 6) * d + base + (rr & 63) : base + rr;
        cp_async16(st + rr * 128 + ((ch ^ (rr & 7)) << 4), W + (size_t)grow * K + kc * LB_KC + ch * 8);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // chunk `ci` has landed and the stage that chunk ci + NST - 1 goes to is free
  auto turn = [&](int ci) {
    asm volatile("cp.async.wait_group %0;" ::"n"(LB_NST - 2) : "memory");
    __syncthreads();
    issue(ci + LB_NST - 1);
  };
#pragma unroll
  for (int i = 0; i < LB_NST - 1; ++i) issue(i);
  lb_cluster_arrive();                                              // (peers exist and run: their shared memory may be read later)
  pdl_sync();

  // ---- inputs of the cluster's rows: attention output (all features), this thread's 4 values of x
  const int cpr_d = d >> 3;                                         // 16-byte chunks per row of d
  for (int idx = tid; idx < LB_ROWS * cpr_d; idx += 256) {
    const int row = idx / cpr_d, ch = idx % cpr_d;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < n_rows) v = *reinterpret_cast<const uint4 *>(a.ao + (size_t)(row0 + row) * d + ch * 8);
    *reinterpret_cast<uint4 *>(buf_ao + row * d * 2 + ((ch ^ (row & 7)) << 4)) = v;
  }
  const int g = lane >> 2, q = (lane & 3) * 2;                      // accumulator rows g, g + 8; columns q, q + 1 of a tile
  const int xcol = r * 64 + w * 8 + q;                              // this thread's two features of x (contractions with NT = 1)
  float xv[4] = {0.f, 0.f, 0.f, 0.f};                               // x[row g][xcol..+1], x[row g + 8][xcol..+1]
  if (g < n_rows) { const float2 t = *reinterpret_cast<const float2 *>(a.x + (size_t)(row0 + g) * d + xcol); xv[0] = t.x; xv[1] = t.y; }
  if (g + 8 < n_rows) { const float2 t = *reinterpret_cast<const float2 *>(a.x + (size_t)(row0 + g + 8) * d + xcol); xv[2] = t.x; xv[3] = t.y; }
  lb_cluster_wait();

  float acc[4][4];
  auto zero = [&]() {
#pragma unroll
    for (int t = 0; t < 4; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
  };
  // x slice -> published operand slice bf16(gain * x) and the rows' sums of squares over this CTA's 64 features
  auto publish_x = [&](const float *gain) {
    const float2 gg = *reinterpret_cast<const float2 *>(gain + xcol);
    uint32_t *pa = reinterpret_cast<uint32_t *>(pub_a);
    pa[(g * 64 + w * 8 + q) >> 1] = pack_bf16x2(gg.x * xv[0], gg.y * xv[1]);
    pa[((g + 8) * 64 + w * 8 + q) >> 1] = pack_bf16x2(gg.x * xv[2], gg.y * xv[3]);
    float s_lo = xv[0] * xv[0] + xv[1] * xv[1], s_hi = xv[2] * xv[2] + xv[3] * xv[3];
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1);
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);
    if ((lane & 3) == 0) { w_ssq[w * LB_ROWS + g] = s_lo; w_ssq[w * LB_ROWS + g + 8] = s_hi; }
    __syncthreads();
    if (tid < LB_ROWS) {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) s += w_ssq[i * LB_ROWS + tid];
      pub_ssq[tid] = s;
    }
  };
  // after a cluster barrier: every CTA's operand slice into buf_a, every CTA's sums of squares -> rstd
  auto gather_a = [&]() {
    const uint32_t pa32 = (uint32_t)__cvta_generic_to_shared(pub_a), ps32 = (uint32_t)__cvta_generic_to_shared(pub_ssq);
    for (int p = tid >> 7; p < R; p += 2) {                         // 128 16-byte pieces per peer
      const int i = tid & 127, row = i >> 3, ch = i & 7;
      const uint4 v = lb_ld_peer16(lb_peer(pa32 + (uint32_t)(row * 128 + ch * 16), (uint32_t)p));
      *reinterpret_cast<uint4 *>(buf_a + row * d * 2 + (((p * 8 + ch) ^ (row & 7)) << 4)) = v;
    }
    if (tid < R * LB_ROWS) all_ssq[tid] = lb_ld_peer_f32(lb_peer(ps32 + (uint32_t)((tid & 15) * 4), (uint32_t)(tid >> 4)));
    __syncthreads();
    if (tid < LB_ROWS) {
      float s = 0.f;
      for (int p = 0; p < R; ++p) s += all_ssq[p * LB_ROWS + tid];
      rstd[tid] = rsqrtf(s / (float)d + a.eps);
    }
    __syncthreads();
  };

  int ci = 0;
  // ---- x += ao Wo^T (this CTA: 64 features, 8 per warp)
  zero();
  for (int kc = 0; kc < n1; ++kc, ++ci) { turn(ci); lb_chunk<1>(acc, ao32, d * 2, kc, ring32 + (uint32_t)((ci % LB_NST) * LB_STAGE), w, lane); }
#pragma unroll
  for (int e = 0; e < 4; ++e) xv[e] += acc[0][e];
  publish_x(a.g_mid);
  lb_cluster_arrive();
  lb_cluster_wait();
  gather_a();

  // ---- h = gelu(rstd * (a W1^T))  (this CTA: ff / R hidden units, NT tiles of 8 per warp)
  zero();
  const int nt_h = nfh / 64;
  for (int kc = 0; kc < n1; ++kc, ++ci) {
    turn(ci);
    const uint32_t st32 = ring32 + (uint32_t)((ci % LB_NST) * LB_STAGE);
    if (nt_h == 4) lb_chunk<4>(acc, a32, d * 2, kc, st32, w, lane);
    else if (nt_h == 3) lb_chunk<3>(acc, a32, d * 2, kc, st32, w, lane);
    else if (nt_h == 2) lb_chunk<2>(acc, a32, d * 2, kc, st32, w, lane);
    else lb_chunk<1>(acc, a32, d * 2, kc, st32, w, lane);
  }
  {
    const float k_lo = rstd[g], k_hi = rstd[g + 8];
    uint32_t *ph = reinterpret_cast<uint32_t *>(pub_h);
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      if (t >= nt_h) break;
      const int col = w * 8 * nt_h + t * 8 + q;
      ph[(g * nfh + col) >> 1] = pack_bf16x2(gelu_erf_fast(acc[t][0] * k_lo), gelu_erf_fast(acc[t][1] * k_lo));
      ph[((g + 8) * nfh + col) >> 1] = pack_bf16x2(gelu_erf_fast(acc[t][2] * k_hi), gelu_erf_fast(acc[t][3] * k_hi));
    }
  }
  lb_cluster_arrive();
  lb_cluster_wait();
  {
    const uint32_t ph32 = (uint32_t)__cvta_generic_to_shared(pub_h);
    const int cpp = nfh >> 3;                                       // 16-byte pieces per row of a peer's slice
    for (int idx = tid; idx < R * LB_ROWS * cpp; idx += 256) {
      const int p = idx / (LB_ROWS * cpp), i = idx % (LB_ROWS * cpp), row = i / cpp, ch = i % cpp;
      const uint4 v = lb_ld_peer16(lb_peer(ph32 + (uint32_t)(row * nfh * 2 + ch * 16), (uint32_t)p));
      *reinterpret_cast<uint4 *>(buf_h + row * ff * 2 + (((p * cpp + ch) ^ (row & 7)) << 4)) = v;
    }
  }
  __syncthreads();

  // ---- x += h W2^T
  zero();
  for (int kc = 0; kc < ff / LB_KC; ++kc, ++ci) { turn(ci); lb_chunk<1>(acc, h32, ff * 2, kc, ring32 + (uint32_t)((ci % LB_NST) * LB_STAGE), w, lane); }
#pragma unroll
  for (int e = 0; e < 4; ++e) xv[e] += acc[0][e];
  if (g < n_rows) *reinterpret_cast<float2 *>(a.x + (size_t)(row0 + g) * d + xcol) = make_float2(xv[0], xv[1]);
  if (g + 8 < n_rows) *reinterpret_cast<float2 *>(a.x + (size_t)(row0 + g + 8) * d + xcol) = make_float2(xv[2], xv[3]);
  if (!a.g_next) {                                                  // last layer: the head kernel takes it from here
    lb_cluster_arrive();                                            // (no peer may leave while its slices are still being read)
    lb_cluster_wait();
    return;
  }
  __syncthreads();                                                  // (w_ssq of the first publication has been read by all)
  publish_x(a.g_next);
  lb_cluster_arrive();
  lb_cluster_wait();
  gather_a();
  lb_cluster_arrive();                                              // last remote read done: waited for at the end

  // ---- next layer's q | k | v of head r = rstd * (a Wqkv^T)   (192 features: 3 tiles of 8 per warp)
  zero();
  for (int kc = 0; kc < n1; ++kc, ++ci) { turn(ci); lb_chunk<3>(acc, a32, d * 2, kc, ring32 + (uint32_t)((ci % LB_NST) * LB_STAGE), w, lane); }
  {
    const float k_lo = rstd[g], k_hi = rstd[g + 8];
#pragma unroll
    for (int t = 0; t < 3; ++t) {
      const int tile = w * 3 + t;                                   // 24 tiles: 8 of q, 8 of k, 8 of v
      const int col = (tile >> 3) * d + r * 64 + (tile & 7) * 8 + q;
      if (g < n_rows)
        *reinterpret_cast<float2 *>(a.qkv + (size_t)(row0 + g) * 3 * d + col) = make_float2(acc[t][0] * k_lo, acc[t][1] * k_lo);
      if (g + 8 < n_rows)
        *reinterpret_cast<float2 *>(a.qkv + (size_t)(row0 + g + 8) * 3 * d + col) = make_float2(acc[t][2] * k_hi, acc[t][3] * k_hi);
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  lb_cluster_wait();
}

// ------------------------------------------------------------------ host side
// Series per cluster and clusters for B series of q_len tokens, or false when the shape is outside the
// kernel's domain: head size 64, at most 8 heads, ff / heads a multiple of 64 up to 256, at most 16 rows
// per cluster with the series spread over all SMs, everything within shared memory.
static bool lb_geometry(int d, int n_heads, int ff, int B, int q_len, int *Bg, int *G) {
  if (n_heads < 1 || n_heads > LB_MAX_R || d != 64 * n_heads || ff % (64 * n_heads) || ff / n_heads > 256) return false;
  if (q_len < 1 || q_len > LB_ROWS) return false;
  if (lb_smem_bytes(d, ff, n_heads) > 227 * 1024) return false;
  const int max_clusters = 148 / n_heads;
  int bg = (B + max_clusters - 1) / max_clusters;
  if (bg * q_len > LB_ROWS) return false;
  *Bg = bg;
  *G = (B + bg - 1) / bg;
  return true;
}

static int lb_init() {
  static std::mutex mu;
  static bool dev_done[TC_MAX_DEVICES] = {false};
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TC_MAX_DEVICES) return -4;
  if (dev_done[dev]) return 0;
  if (cudaFuncSetAttribute(layer_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) return -4;
  dev_done[dev] = true;
  return 0;
}

static bool lb_launch(cudaStream_t st, bool pdl, const LbArgs &args, int G) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(args.R * G);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = lb_smem_bytes(args.d, args.ff, args.R);
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = args.R; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, layer_block_kernel, args) == cudaSuccess;
}

}  // namespace tsfm

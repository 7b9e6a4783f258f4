// Small-batch contraction with the whole weight tile resident in shared memory.
//
//   C[t, f] (op)= sum_k A[t, k] * W[f, k]        A: [M, K] tokens (bf16), W: [N, K] weights (bf16)
//
// For the passes of a few dozen tokens (draft steps, one-token decode steps, short verification
// passes) a contraction is a dependent link in a chain of launches, and what it costs is the
// latency between "my input is ready" and "my output is written".  This kernel keeps that path
// short:
//   * a CTA owns 16 output features x 32 tokens over the WHOLE K range, so nothing is exchanged
//     between CTAs and every epilogue (GELU, residual, folded norm) sees complete sums;
//   * its weight tile (16 x K) does not depend on the preceding kernel: it is requested with
//     asynchronous copies BEFORE the dependency wait (programmatic dependent launch) and is in
//     shared memory by the time the activations are;
//   * the eight warps split K among them (warp w takes the 16-wide k steps w, w + 8, ...), each
//     accumulating a 32 x 16 partial tile in registers with mma.sync m16n8k16 (bf16 in, fp32
//     accumulate); the partial tiles are summed through shared memory in a fixed order.
// The tensor-memory kernel (gemm_sk.cuh) stays the tool wherever K is long, tokens are many or the
// grid would not fit in one wave: an MMA issued there costs ~72 ns whatever its width, and its
// chain (TMA -> MMA -> commit -> tcgen05.ld -> cluster exchange) is about 2 us longer than this one.
//
// Shared memory: W tile [16][K], A tile [32][K] (bf16, 16-byte chunks of a row XOR-ed with row & 7
// so that ldmatrix reads are conflict-free), partial tiles [8][32][16] fp32, rstd [32].
// grid = (ceil(N / 16), ceil(M / 32)), block = 256.  K a multiple of 64, at most WS_MAX_K.
#pragma once
#include "common.cuh"
#include "kernels_simt.cuh"
#include "gemm_sk.cuh"

namespace tsfm {

constexpr int WS_FN = 16, WS_MT = 32, WS_WARPS = 8, WS_MAX_K = 2048;

static inline int ws_smem_bytes(int K) { return (WS_FN + WS_MT) * K * 2 + WS_WARPS * WS_MT * WS_FN * 4 + WS_MT * 4; }

__device__ __forceinline__ void ws_ldsm4(uint32_t addr, uint32_t (&d)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(addr));
}

// NORM: compile the folded-RMSNorm epilogues (SkNorm; slices of 16 features).
template <bool NORM>
__global__ void __launch_bounds__(256)
gemm_ws_kernel(const bf16 *A, const bf16 *__restrict__ W, void *C, int M, int N, int K,
               int epi, const SkNorm nm, const LiveRows lr) {
  extern __shared__ __align__(128) unsigned char ws_smem[];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int f0 = blockIdx.x * WS_FN, t0 = blockIdx.y * WS_MT;
  // rows in use (active-series compaction): read before the dependency wait, see gemm_sk_kernel
  if (lr.n_live) {
    M = min(M, *reinterpret_cast<const volatile int *>(lr.n_live) * lr.q_len);
    if (t0 >= M) return;
  }
  const int row_bytes = K * 2, cpr = K >> 3;                   // bytes and 16-byte chunks per tile row
  unsigned char *Ws = ws_smem, *As = ws_smem + WS_FN * row_bytes;
  float *red = reinterpret_cast<float *>(As + WS_MT * row_bytes);        // [8][32][16]
  float *rs = red + WS_WARPS * WS_MT * WS_FN;                            // [32]
  const uint32_t Ws32 = (uint32_t)__cvta_generic_to_shared(Ws), As32 = (uint32_t)__cvta_generic_to_shared(As);

  // ---- weight tile: independent of the preceding kernel
  for (int i = tid; i < WS_FN * cpr; i += 256) {
    const int r = i / cpr, c = i % cpr;
    const uint32_t dst = Ws32 + (uint32_t)(r * row_bytes + ((c ^ (r & 7)) << 4));
    if (f0 + r < N) cp_async16(Ws + (dst - Ws32), W + (size_t)(f0 + r) * K + c * 8);
    else *reinterpret_cast<uint4 *>(Ws + (dst - Ws32)) = make_uint4(0u, 0u, 0u, 0u);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // the gains of this thread's two output features (folded norm): constants, fetched before the wait
  float2 gg = make_float2(0.f, 0.f);
  if (NORM && nm.a_out && f0 + (tid & 7) * 2 < N) gg = *reinterpret_cast<const float2 *>(nm.gain + f0 + (tid & 7) * 2);
  pdl_sync();
  // ---- activation tile (rows past M are zero)
  for (int i = tid; i < WS_MT * cpr; i += 256) {
    const int r = i / cpr, c = i % cpr;
    unsigned char *dst = As + r * row_bytes + ((c ^ (r & 7)) << 4);
    if (t0 + r < M) cp_async16(dst, A + (size_t)(t0 + r) * K + c * 8);
    else *reinterpret_cast<uint4 *>(dst) = make_uint4(0u, 0u, 0u, 0u);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // ---- while the copies fly: this thread's two outputs, their old values, the rows' rstd
  const int orow = tid >> 3, ocol = (tid & 7) * 2;             // output (orow, ocol), (orow, ocol + 1) of the tile
  const int t = t0 + orow, f = f0 + ocol;
  const bool live = t < M && f < N;                            // (N is even: both columns or none)
  float2 old = make_float2(0.f, 0.f);
  if (epi == EPI_RESID && live) old = *reinterpret_cast<const float2 *>((const float *)C + (size_t)t * N + f);
  if (NORM && nm.ssq_in) {
    float acc = 0.f;
    if (t < M)
      for (int j = tid & 7; j < nm.n_part; j += 8) acc += nm.ssq_in[(size_t)t * nm.n_part + j];
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    if ((tid & 7) == 0) rs[orow] = rsqrtf(acc * nm.inv_d + nm.eps);
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();

  // ---- main loop: warp w takes k steps w, w + 8, ...; acc[row tile][feature tile][4]
  float acc[2][2][4];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = acc[a][b][2] = acc[a][b][3] = 0.f;
  const int a_row = lane & 15, a_chunk = lane >> 4;                           // A fragment addressing
  const int b_row = (lane & 7) + ((lane >> 4) & 1) * 8, b_chunk = (lane >> 3) & 1;   // B: two feature tiles at once
  for (int ks = w; ks < (K >> 4); ks += WS_WARPS) {
    uint32_t bw[4], a0[4], a1[4];
    ws_ldsm4(Ws32 + (uint32_t)(b_row * row_bytes + (((ks * 2 + b_chunk) ^ (b_row & 7)) << 4)), bw);
    ws_ldsm4(As32 + (uint32_t)(a_row * row_bytes + (((ks * 2 + a_chunk) ^ (a_row & 7)) << 4)), a0);
    ws_ldsm4(As32 + (uint32_t)((16 + a_row) * row_bytes + (((ks * 2 + a_chunk) ^ (a_row & 7)) << 4)), a1);
    mma_bf16_16816(acc[0][0], a0, bw[0], bw[1]);
    mma_bf16_16816(acc[0][1], a0, bw[2], bw[3]);
    mma_bf16_16816(acc[1][0], a1, bw[0], bw[1]);
    mma_bf16_16816(acc[1][1], a1, bw[2], bw[3]);
  }
  // ---- partial tiles to shared memory, summed in warp order
  {
    float *mine = red + w * (WS_MT * WS_FN);
    const int g = lane >> 2, q = (lane & 3) * 2;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        *reinterpret_cast<float2 *>(mine + (a * 16 + g) * WS_FN + b * 8 + q) = make_float2(acc[a][b][0], acc[a][b][1]);
        *reinterpret_cast<float2 *>(mine + (a * 16 + g + 8) * WS_FN + b * 8 + q) = make_float2(acc[a][b][2], acc[a][b][3]);
      }
  }
  __syncthreads();
  float2 v = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < WS_WARPS; ++i) {
    const float2 p = *reinterpret_cast<const float2 *>(red + i * (WS_MT * WS_FN) + orow * WS_FN + ocol);
    v.x += p.x;
    v.y += p.y;
  }
  // ---- epilogue
  if (NORM && nm.ssq_in) { const float k = rs[orow]; v.x *= k; v.y *= k; }
  const size_t o = (size_t)t * N + f;
  if (epi == EPI_RESID) {
    v.x += old.x;
    v.y += old.y;
    if (live) *reinterpret_cast<float2 *>((float *)C + o) = v;
    if (NORM && nm.a_out) {
      // the next contraction's operand bf16(gain * x) and the row's sum of squares over these 16 features
      if (live) *reinterpret_cast<uint32_t *>(nm.a_out + o) = pack_bf16x2(gg.x * v.x, gg.y * v.y);
      float sq = live ? v.x * v.x + v.y * v.y : 0.f;
      sq += __shfl_xor_sync(0xffffffffu, sq, 1);
      sq += __shfl_xor_sync(0xffffffffu, sq, 2);
      sq += __shfl_xor_sync(0xffffffffu, sq, 4);
      if ((tid & 7) == 0 && t < M && f0 < N) nm.ssq_out[(size_t)t * (N >> 4) + (f0 >> 4)] = sq;
    }
  } else if (live) {
    if (epi == EPI_F32) *reinterpret_cast<float2 *>((float *)C + o) = v;
    else if (epi == EPI_T) *reinterpret_cast<uint32_t *>((bf16 *)C + o) = pack_bf16x2(v.x, v.y);
    else *reinterpret_cast<uint32_t *>((bf16 *)C + o) = pack_bf16x2(gelu_erf_fast(v.x), gelu_erf_fast(v.y));
  }
}

// ------------------------------------------------------------------ host side
static int gemm_ws_init() {
  static std::mutex mu;
  static bool dev_done[TC_MAX_DEVICES] = {false};
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TC_MAX_DEVICES) return -4;
  if (dev_done[dev]) return 0;
  if (cudaFuncSetAttribute(gemm_ws_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_ws_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
    return -4;
  dev_done[dev] = true;
  return 0;
}

// Whether this kernel is the better tool for the shape: few tokens, the two tiles fit in shared
// memory, N even and the operands 16-byte aligned, and the whole grid is resident at once.
static bool gemm_ws_eligible(const void *A, const void *W, int M, int N, int K) {
  if (M < 1 || M > 256 || K < 64 || K % 64 || K > WS_MAX_K || N % 2) return false;
  if (((uintptr_t)A & 15) || ((uintptr_t)W & 15)) return false;
  const int smem = ws_smem_bytes(K);
  if (smem > 227 * 1024) return false;
  const int per_sm = std::min(8, (228 * 1024) / (smem + 1024));
  const long ctas = (long)((N + WS_FN - 1) / WS_FN) * ((M + WS_MT - 1) / WS_MT);
  return ctas <= (long)per_sm * 148;
}

static bool gemm_ws_launch(cudaStream_t st, bool pdl, const void *A, const void *W, void *C, int M, int N, int K, int epi,
                           const SkNorm *norm, LiveRows lr) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((N + WS_FN - 1) / WS_FN, (M + WS_MT - 1) / WS_MT);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = ws_smem_bytes(K);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  const SkNorm nm = norm ? *norm : SkNorm{};
  if (norm)
    return cudaLaunchKernelEx(&cfg, gemm_ws_kernel<true>, (const bf16 *)A, (const bf16 *)W, C, M, N, K, epi, nm, lr) == cudaSuccess;
  return cudaLaunchKernelEx(&cfg, gemm_ws_kernel<false>, (const bf16 *)A, (const bf16 *)W, C, M, N, K, epi, nm, lr) == cudaSuccess;
}

}  // namespace tsfm

// bf16 x bf16 -> fp32 contraction on the sm_100a tensor cores, split along K across a
// thread-block cluster.
//
//   C[t, f] (op)= sum_k A[t, k] * W[f, k]        A: [M, K] tokens, W: [N, K] weights
//
// Same swap-AB tiling as gemm_tc.cuh (128 weight rows = MMA M, BN tokens = MMA N, 64-wide K
// stages fed by TMA into a 128-byte-swizzled ring, accumulator in tensor memory), with two
// differences that matter when the token count is small and the call is latency-bound:
//   * BN is a run-time value (any multiple of 16 up to 256), so M = 160 verification tokens
//     are one tile, not a padded 256;
//   * the K loop is split over the S CTAs of a cluster (grid.z = cluster.z = S <= 8).  Each CTA
//     parks its partial tile in its own shared memory; after a cluster barrier CTA r sums rows
//     r, r + S, ... of all S partial tiles through distributed shared memory and applies the
//     epilogue once.  No atomics, no pre-zeroed accumulator, a fixed summation order, and every
//     epilogue (GELU included) can be split.
//   * a residual epilogue (x += A W^T) on a feature count that is a multiple of 128 leaves the
//     read-modify-write to the TMA unit: the tile (summed over the cluster first) is staged in
//     shared memory as [token][128 features] fp32 and added to x by one
//     cp.reduce.async.bulk.tensor per CTA, so no thread waits for the old values of x.
// Warp roles and bounded waits as in gemm_tc.cuh.
#pragma once
#include "gemm_tc.cuh"
#include <vector>

namespace tsfm {

constexpr int SK_MAX_SPLIT = 8;

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}
__host__ __device__ constexpr uint32_t umma_idesc_rt(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

// RMSNorm folded into the contractions around it.  The norm of a row is a scalar factor, so it
// commutes with the contraction that consumes the row: the kernel that PRODUCES the residual
// stream (residual epilogue) also writes a' = bf16(gain * x) -- the next contraction's operand,
// not yet normalised -- and the sum of squares of every 16-feature slice of the row; the kernel
// that CONSUMES a' multiplies its result rows by rstd = rsqrt(sum of the slices / d + eps).
struct SkNorm {
  const float *ssq_in;      // [M][n_part] slice sums of squares of this contraction's input rows, or NULL
  float *ssq_out;           // [M][N / 16] written by a residual epilogue, or NULL
  const float *gain;        // [N] gain of the norm that follows the residual epilogue
  bf16 *a_out;              // [M][N] bf16(gain * x_new), or NULL
  int n_part;               // partial sums per input row (d / 16)
  float inv_d, eps;
};

struct SkShape {
  int BN, stages, tmem_cols, smem_bytes;
};
// Ring of `stages` x (W tile 16 KB + A tile BN x 128 B); the partial-sum tile (BN x 128 fp32)
// reuses the ring once the accumulator is complete.
// (stages_hint > 0: the ring depth the tile rule asks for instead of the default.)
static inline SkShape sk_shape(int BN, int kb_per_cta, bool split, int wt = 1, int stages_hint = 0) {
  SkShape s;
  s.BN = BN;
  const int stage = TC_W_BYTES * wt + BN * TC_BK * 2;
  int stages = stages_hint > 0 ? stages_hint : wt == 2 ? 3 : BN > 160 ? 4 : BN > 64 ? 3 : 4;
  if (stages > kb_per_cta) stages = kb_per_cta < 1 ? 1 : kb_per_cta;
  int bytes = stages * stage;
  if (split && bytes < BN * TC_BM * 4) bytes = BN * TC_BM * 4;
  s.stages = stages;
  const int cols = BN * wt;
  s.tmem_cols = cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
  s.smem_bytes = bytes + 1024 + 256 + 1024;        // + alignment slack, barriers, rstd of the tile's rows
  return s;
}

__device__ __forceinline__ void sk_store_rt(void *C, size_t o, float v, int epi) {
  if (epi == EPI_F32) ((float *)C)[o] = v;
  else if (epi == EPI_T) ((bf16 *)C)[o] = __float2bfloat16_rn(v);
  else if (epi == EPI_GELU_T) ((bf16 *)C)[o] = __float2bfloat16_rn(gelu_erf_fast(v));
  else ((float *)C)[o] += v;
}

// grid = (ceil(N / 128), ceil(M / BN), S), cluster = (1, 1, S), block = 192.
// ring_bytes = size of the tile region (a multiple of 1024); barriers sit behind it.
// WT = weight tiles per CTA.
// NORM = compile the folded-RMSNorm epilogues (SkNorm); the plain instantiations carry none of it.
// tma_c = SK_TMA_ADD: residual epilogue through mapC (fp32 [M][N], box = BN / S tokens x 128 features);
// tma_c = SK_TMA_BF16 (S = 1 only): bf16 output (with or without GELU) staged as [token][128
// features] bf16 and written by one TMA store per weight tile through mapC (bf16 [M][N]) -- whole
// 128-byte lines at once, where per-thread 2-byte stores leave each line to be completed by a
// second warp later.
// tma_c = SK_TMA_F32: fp32 output, staged (and summed over the cluster) like SK_TMA_ADD, stored.
enum { SK_TMA_NONE = 0, SK_TMA_ADD = 1, SK_TMA_BF16 = 2, SK_TMA_F32 = 3 };
// (Both wait only until the copy has READ its shared-memory source: the staging tile may then be reused
// or the CTA may leave.  The writes themselves complete before the grid does, which is what the next
// kernel's dependency wait waits for.)
__device__ __forceinline__ void sk_tma_store(const CUtensorMap *map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void sk_tma_reduce_add(const CUtensorMap *map, uint32_t src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

template <int WT, bool NORM>
__global__ void __launch_bounds__(192, 1)
gemm_sk_kernel(const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapA,
               const __grid_constant__ CUtensorMap mapC, void *C, int M, int N, int K, int BN,
               int stages, int tmem_cols, int ring_bytes, int epi, int tma_c, const SkNorm nm,
               int *__restrict__ status, const LiveRows lr) {
  constexpr int wt = WT;
  // Active-series compaction: only the first n_live * q_len rows are in use.  CTAs (whole clusters:
  // the split shares the token tile) of token tiles past them leave before touching anything.  The
  // count is read before the dependency wait on purpose, so that such CTAs cost nothing: it was
  // written by the kernel that closed the previous round, and every contraction has at least two
  // kernels of its own pass between itself and that one, so it is complete and visible by the time
  // this grid may start (a grid starts only after every CTA of its predecessor has passed its own
  // wait, i.e. after the predecessor's predecessor has finished).
  if (lr.n_live) {
    M = min(M, *reinterpret_cast<const volatile int *>(lr.n_live) * lr.q_len);
    if ((int)blockIdx.y * BN >= M) return;
  }
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = tiles + (uint32_t)ring_bytes;
  const uint32_t full0 = bars, empty0 = bars + 64, accum = bars + 128, slot = bars + 136;
  uint32_t *slot_ptr = reinterpret_cast<uint32_t *>(smem_raw + (slot - smem_u32(smem_raw)));
  float *rs = reinterpret_cast<float *>(smem_raw + (bars + 256 - smem_u32(smem_raw)));   // [BN] rstd of the tile's rows
  float *stage_f = reinterpret_cast<float *>(smem_raw + (tiles - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // wt = weight tiles (of 128 output features) per CTA, 1 or 2.  Two tiles share each token tile
  // in shared memory: per K block a 256 x 256 output tile loads 64 KB instead of 2 x 48 KB, which
  // is what lets one CTA's TMA stream (~120 GB/s) keep up with its tensor core.
  const int f0 = blockIdx.x * TC_BM * wt, t0 = blockIdx.y * BN;
  const int S = gridDim.z, rank = blockIdx.z;
  const int KB_all = (K + TC_BK - 1) / TC_BK;
  const int kb_lo = (int)(((long long)KB_all * rank) / S);
  const int kb_hi = (int)(((long long)KB_all * (rank + 1)) / S);
  const int KB = kb_hi - kb_lo;
  const int a_bytes = BN * TC_BK * 2, w_bytes = TC_W_BYTES * wt, stage_bytes = w_bytes + a_bytes;
  // (Measured: spreading the K steps of a stage over several accumulators does not help a narrow
  // tile -- one MMA of 128 x BN x 16 takes ~90 ns whatever BN is -- so one accumulator per tile.)

  if (warp == 4 && lane == 0) {
    // descriptor fetches off the critical path of the first loads (and of the output copy)
    asm volatile("prefetch.tensormap [%0];" ::"l"(&mapW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&mapA) : "memory");
    if (tma_c) asm volatile("prefetch.tensormap [%0];" ::"l"(&mapC) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(accum, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"((uint32_t)tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *slot_ptr;

  float g_direct = 0.f;
  float4 g_vec = make_float4(0.f, 0.f, 0.f, 0.f);
  if (warp == 4 && lane == 0) {
    // ---------------- TMA producer.  The weights do not depend on the preceding kernel: the
    // first ring-full of weight tiles is requested before waiting for it, the activation tiles
    // after.
    const int pre = KB < stages ? KB : stages;
    for (int kb = 0; kb < pre; ++kb) {
      mbar_expect_tx(full0 + 8 * kb, (uint32_t)stage_bytes);
      for (int q = 0; q < wt; ++q)
        tma_load_2d(tiles + kb * stage_bytes + q * TC_W_BYTES, &mapW, (kb_lo + kb) * TC_BK, f0 + q * TC_BM, full0 + 8 * kb);
    }
    pdl_sync();
    for (int kb = 0; kb < pre; ++kb)
      tma_load_2d(tiles + kb * stage_bytes + w_bytes, &mapA, (kb_lo + kb) * TC_BK, t0, full0 + 8 * kb);
    for (int kb = pre; kb < KB; ++kb) {
      const int s = kb % stages;
      const uint32_t ph = (uint32_t)(kb / stages) & 1u;
      if (!mbar_wait(empty0 + 8 * s, ph ^ 1u)) { atomicExch(status, DEV_TIMEOUT_TMA); break; }
      const uint32_t dst = tiles + s * stage_bytes;
      mbar_expect_tx(full0 + 8 * s, (uint32_t)stage_bytes);
      for (int q = 0; q < wt; ++q)
        tma_load_2d(dst + q * TC_W_BYTES, &mapW, (kb_lo + kb) * TC_BK, f0 + q * TC_BM, full0 + 8 * s);
      tma_load_2d(dst + w_bytes, &mapA, (kb_lo + kb) * TC_BK, t0, full0 + 8 * s);
    }
  } else {
    if (NORM && nm.a_out && warp < 4) {
      // gains of the features this thread finishes in either epilogue: constants, fetched before the wait
      const int fd = f0 + threadIdx.x, fv = f0 + (threadIdx.x & 31) * 4;
      if (fd < N) g_direct = nm.gain[fd];
      if (N % 4 == 0 && fv + 3 < N) g_vec = *reinterpret_cast<const float4 *>(nm.gain + fv);
    }
    pdl_sync();
    if (warp < 4) {
      if (NORM && nm.ssq_in) {                                // overlaps the main loop
        for (int i = threadIdx.x; i < BN; i += 128) {
          float acc = 0.f;
          if (t0 + i < M)
            for (int j = 0; j < nm.n_part; ++j) acc += nm.ssq_in[(size_t)(t0 + i) * nm.n_part + j];
          rs[i] = rsqrtf(acc * nm.inv_d + nm.eps);
        }
      }
      if (NORM) asm volatile("bar.sync 1, 128;" ::: "memory");
    }
  }
  if (warp == 4 && lane == 0) {
  } else if (warp == 5 && lane == 0) {
    // ---------------- MMA issuer
    const uint32_t idesc = umma_idesc_rt(BN);
    bool ok = true;
    for (int kb = 0; kb < KB && ok; ++kb) {
      const int s = kb % stages;
      const uint32_t ph = (uint32_t)(kb / stages) & 1u;
      if (!mbar_wait(full0 + 8 * s, ph)) { atomicExch(status, DEV_TIMEOUT_MMA); ok = false; break; }
      tc_fence_after();
      const uint32_t sw = tiles + s * stage_bytes;
      const uint64_t dw = umma_smem_desc(sw), dw2 = umma_smem_desc(sw + TC_W_BYTES), da = umma_smem_desc(sw + w_bytes);
#pragma unroll
      for (int k = 0; k < TC_BK / 16; ++k) {
        umma_bf16(tmem, dw + 2 * k, da + 2 * k, idesc, (kb | k) ? 1u : 0u);
        if (wt == 2) umma_bf16(tmem + BN, dw2 + 2 * k, da + 2 * k, idesc, (kb | k) ? 1u : 0u);
      }
      umma_commit(empty0 + 8 * s);
    }
    if (ok) umma_commit(accum);
  }
  // ---------------- epilogue, part 1: drain the accumulator(s), one weight tile at a time
  const bool staged = S > 1 || tma_c;                  // through shared memory ([token][128 features] fp32)
  bool acc_ok = false;
  if (warp < 4) {
    acc_ok = KB > 0 && mbar_wait(accum, 0);
    if (!acc_ok && KB > 0 && lane == 0) atomicExch(status, DEV_TIMEOUT_EPILOGUE);
    tc_fence_after();
  }
#pragma unroll 1
  for (int q = 0; q < wt; ++q) {
    if (warp < 4 && acc_ok) {
      const int fl = warp * 32 + lane, f = f0 + q * TC_BM + fl;
      const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(q * BN);
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 16) {
        if (t0 + cc >= M) break;
        float v[16];
        tmem_ld16(tbase + cc, v);
        if (tma_c == SK_TMA_BF16) {
          bf16 *stage_h = reinterpret_cast<bf16 *>(stage_f);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            stage_h[(cc + j) * TC_BM + fl] = __float2bfloat16_rn(epi == EPI_GELU_T ? gelu_erf_fast(v[j]) : v[j]);
          continue;
        }
        if (staged) {
#pragma unroll
          for (int j = 0; j < 16; ++j) stage_f[(cc + j) * TC_BM + fl] = v[j];
          continue;
        }
        if (f < N) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (t0 + cc + j < M) {
              const size_t o = (size_t)(t0 + cc + j) * N + f;
              if (NORM && nm.ssq_in) v[j] *= rs[cc + j];
              if (NORM && epi == EPI_RESID && nm.a_out) {
                const float xn = ((float *)C)[o] + v[j];
                ((float *)C)[o] = xn;
                nm.a_out[o] = __float2bfloat16_rn(g_direct * xn);
                v[j] = xn * xn;
              } else {
                sk_store_rt(C, o, v[j], epi);
              }
            }
        }
        if (NORM && epi == EPI_RESID && nm.a_out) {          // sums of squares over slices of 16 features (N % 32 == 0)
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            float sq = v[j];
            sq += __shfl_xor_sync(0xffffffffu, sq, 1);
            sq += __shfl_xor_sync(0xffffffffu, sq, 2);
            sq += __shfl_xor_sync(0xffffffffu, sq, 4);
            sq += __shfl_xor_sync(0xffffffffu, sq, 8);
            if ((lane & 15) == 0 && f < N && t0 + cc + j < M) nm.ssq_out[(size_t)(t0 + cc + j) * (N >> 4) + (f >> 4)] = sq;
          }
        }
      }
    }
    if (tma_c && S == 1 && warp < 4) {
      // the staged tile goes to x as one TMA reduction (rows past M are clipped by the map)
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (threadIdx.x == 0 && acc_ok) {
        if (tma_c == SK_TMA_ADD) sk_tma_reduce_add(&mapC, tiles, f0 + q * TC_BM, t0);
        else sk_tma_store(&mapC, tiles, f0 + q * TC_BM, t0);
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");       // the stage is free again
    }
  }
  __syncwarp();
  if (S > 1) {
    // ---------------- epilogue, part 2: reduce the S partial tiles through distributed shared memory
    tc_fence_before();
    cluster_sync_all();
    if (warp < 4 && (tma_c == SK_TMA_ADD || tma_c == SK_TMA_F32)) {
      // CTA r sums its block of BN / S rows over the S partial tiles, in place in its own tile,
      // and hands the block to the TMA unit
      const int RB = BN / S, rg = threadIdx.x >> 5, c4 = (threadIdx.x & 31) * 4;
      uint32_t remote[SK_MAX_SPLIT];
#pragma unroll
      for (int r = 0; r < SK_MAX_SPLIT; ++r) {
        const uint32_t a = tiles + (uint32_t)c4 * 4;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote[r]) : "r"(a), "r"((uint32_t)(r < S ? r : 0)));
      }
      for (int tl = rank * RB + rg; tl < (rank + 1) * RB; tl += 4) {
        if (t0 + tl >= M) break;
        float4 v[SK_MAX_SPLIT];
#pragma unroll
        for (int r = 0; r < SK_MAX_SPLIT; ++r)
          if (r < S)
            asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(v[r].x), "=f"(v[r].y), "=f"(v[r].z), "=f"(v[r].w)
                         : "r"(remote[r] + (uint32_t)tl * (TC_BM * 4)) : "memory");
        float4 sum = v[0];
#pragma unroll
        for (int r = 1; r < SK_MAX_SPLIT; ++r)
          if (r < S) { sum.x += v[r].x; sum.y += v[r].y; sum.z += v[r].z; sum.w += v[r].w; }
        *reinterpret_cast<float4 *>(stage_f + (size_t)tl * TC_BM + c4) = sum;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (threadIdx.x == 0 && t0 + rank * RB < M) {
        if (tma_c == SK_TMA_ADD) sk_tma_reduce_add(&mapC, tiles + (uint32_t)(rank * RB) * (TC_BM * 4), f0, t0 + rank * RB);
        else sk_tma_store(&mapC, tiles + (uint32_t)(rank * RB) * (TC_BM * 4), f0, t0 + rank * RB);
      }
    } else if (warp < 4) {
      // thread -> (row group, 4 consecutive features): one 16-byte load per partial tile, all S
      // loads of a row in flight together, one 16-byte (fp32) or 8-byte (bf16) store per row
      const int rg = threadIdx.x >> 5, c4 = (threadIdx.x & 31) * 4, f = f0 + c4;
      uint32_t remote[SK_MAX_SPLIT];
#pragma unroll
      for (int r = 0; r < SK_MAX_SPLIT; ++r) {
        const uint32_t a = tiles + (uint32_t)c4 * 4;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote[r]) : "r"(a), "r"((uint32_t)(r < S ? r : 0)));
      }
      const bool vec = (N % 4 == 0) && (f + 3 < N);
      for (int tl = rank + S * rg; tl < BN; tl += 4 * S) {
        const int t = t0 + tl;
        if (t >= M) break;
        float4 v[SK_MAX_SPLIT];
#pragma unroll
        for (int r = 0; r < SK_MAX_SPLIT; ++r)
          if (r < S)
            asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(v[r].x), "=f"(v[r].y), "=f"(v[r].z), "=f"(v[r].w)
                         : "r"(remote[r] + (uint32_t)tl * (TC_BM * 4)) : "memory");
        float4 sum = v[0];
#pragma unroll
        for (int r = 1; r < SK_MAX_SPLIT; ++r)
          if (r < S) { sum.x += v[r].x; sum.y += v[r].y; sum.z += v[r].z; sum.w += v[r].w; }
        const size_t o = (size_t)t * N + f;
        if (NORM && nm.ssq_in) { const float k = rs[tl]; sum.x *= k; sum.y *= k; sum.z *= k; sum.w *= k; }
        if (vec) {
          if (epi == EPI_F32) {
            *reinterpret_cast<float4 *>((float *)C + o) = sum;
          } else if (epi == EPI_RESID) {
            float4 old = *reinterpret_cast<float4 *>((float *)C + o);
            old.x += sum.x; old.y += sum.y; old.z += sum.z; old.w += sum.w;
            *reinterpret_cast<float4 *>((float *)C + o) = old;
            if (NORM && nm.a_out) {
              const float4 gg = g_vec;
              const __nv_bfloat162 lo = __floats2bfloat162_rn(gg.x * old.x, gg.y * old.y), hi = __floats2bfloat162_rn(gg.z * old.z, gg.w * old.w);
              uint2 pk;
              pk.x = *reinterpret_cast<const uint32_t *>(&lo);
              pk.y = *reinterpret_cast<const uint32_t *>(&hi);
              *reinterpret_cast<uint2 *>(nm.a_out + o) = pk;
              // 4 lanes = one 16-feature slice.  N is a multiple of 32 here, so a slice is inside N
              // or outside it as a whole: only its own 4 lanes are named in the shuffles (the lanes
              // of a feature tile's slices beyond N never get here).
              const unsigned grp = 0xfu << (threadIdx.x & 28);
              float sq = old.x * old.x + old.y * old.y + old.z * old.z + old.w * old.w;
              sq += __shfl_xor_sync(grp, sq, 1);
              sq += __shfl_xor_sync(grp, sq, 2);
              if ((threadIdx.x & 3) == 0) nm.ssq_out[(size_t)t * (N >> 4) + (f >> 4)] = sq;
            }
          } else {
            if (epi == EPI_GELU_T) { sum.x = gelu_erf_fast(sum.x); sum.y = gelu_erf_fast(sum.y); sum.z = gelu_erf_fast(sum.z); sum.w = gelu_erf_fast(sum.w); }
            const __nv_bfloat162 lo = __floats2bfloat162_rn(sum.x, sum.y), hi = __floats2bfloat162_rn(sum.z, sum.w);
            uint2 pk;
            pk.x = *reinterpret_cast<const uint32_t *>(&lo);
            pk.y = *reinterpret_cast<const uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>((bf16 *)C + o) = pk;
          }
        } else {
          const float e[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (f + i < N) sk_store_rt(C, o + i, e[i], epi);
        }
      }
    }
    cluster_sync_all();          // no CTA leaves while a peer may still read its tile
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------ host side
struct GemmSkPlan {
  bool valid = false;
  int N = 0, K = 0, M_max = 0;
  const void *A = nullptr;
  CUtensorMap mapW;
  CUtensorMap mapA[16];            // box (BN = 16 * (i + 1)) x 64, encoded on first use
  bool haveA[16] = {false};
  // outputs written by the TMA unit (fp32 residual stream, bf16 activations): one map per
  // (buffer, M, rows per box, element type)
  struct CMap { const void *C; int M, rows; bool is_bf16; CUtensorMap map; };
  std::vector<CMap> mapC;
};

// fp32 [rows][N] row-major, box = box_rows x 128 features, no swizzle.
static int sk_encode_c(CUtensorMap *map, const void *base, int rows, int N, int box_rows, bool is_bf16) {
  cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)N * (is_bf16 ? 2 : 4)};
  cuuint32_t box[2] = {(cuuint32_t)TC_BM, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -4;
}

static int gemm_sk_init() {
  if (int rc = gemm_tc_init()) return rc;
  static bool dev_done[TC_MAX_DEVICES] = {false};       // per device, like gemm_tc_init
  std::lock_guard<std::mutex> lock(g_tc_init_mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TC_MAX_DEVICES) return -4;
  if (dev_done[dev]) return 0;
  if (cudaFuncSetAttribute(gemm_sk_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_sk_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(gemm_sk_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
    return -4;
  dev_done[dev] = true;
  return 0;
}

static int gemm_sk_plan(GemmSkPlan *plan, const void *W, int N, int K, const void *A, int M_max) {
  plan->valid = false;
  plan->N = N; plan->K = K; plan->M_max = M_max; plan->A = A;
  for (bool &b : plan->haveA) b = false;
  plan->mapC.clear();
  if (K % 8 || K < 16 || N < 1 || M_max < 1) return 0;
  if (((uintptr_t)W & 15) || ((uintptr_t)A & 15)) return 0;
  if (!g_encode) return -4;
  if (tc_encode(&plan->mapW, W, N, K, TC_BM)) return -4;
  plan->valid = true;
  return 0;
}

// Tile and split choice for M tokens: one token tile up to 256 rows (rounded up to 16), and
// as many K splits (a power of two, at most 8, at most the number of K blocks) as it takes to
// put the grid on most of the 148 SMs.
// epi: the epilogue (EPI_*); *STG: ring depth, 0 = the default for the tile.
static void gemm_sk_geometry(int N, int K, int M, int epi, int *BN, int *S, int *WT, int *STG) {
  *WT = 1;
  *STG = 0;
  // Measured on B200 (graph replay, dependent launches): up to a few hundred tokens a 32-token
  // tile with K split until the grid has ~150-250 CTAs is fastest (the partial-tile exchange
  // grows with the tile, the latency chain does not shrink); large M takes 128/256-token tiles.
  const int FT = (N + TC_BM - 1) / TC_BM, KB = (K + TC_BK - 1) / TC_BK;
  if (M >= 4096) {
    // Very large M (prefill, wide verification), no split.  Measured on B200 (graph replay):
    // 128 x 128 tiles with two CTAs per SM (one's epilogue under the other's main loop) win
    // unless the K loop is long (>= 32 blocks) and the 256 x 256 grid (two weight tiles per CTA,
    // token tiles shared in shared memory) still covers most SMs.
    const int ctas_b = ((FT + 1) / 2) * ((M + 255) / 256);
    *S = 1;
    if (KB >= 32 && ctas_b >= 100) {
      // one 256-feature CTA per SM: of 256- and 192-token tiles the one with fewer waves x tile
      // (C4's prefill W2, M = 16320, N = 1280: 320 CTAs of 256 tokens are 2.2 waves, 183 us;
      // 425 of 192 are 2.9, 162 us)
      const int w256 = (ctas_b + 147) / 148, w192 = (((FT + 1) / 2) * ((M + 191) / 192) + 147) / 148;
      *BN = w192 * 192 < w256 * 256 ? 192 : 256;
      *WT = 2;
    } else if (KB >= 32) {
      *BN = 128;
    } else if (epi == EPI_T || epi == EPI_GELU_T) {
      // bf16 outputs (the GELU epilogue is the longest): a two-stage ring lets a third CTA onto the
      // SM, so that two main loops run under every epilogue (M = 16320, N = 5120, K = 1280: 295 ->
      // 247 us; M = 7424, N = 4096, K = 1024: 106 -> 93 us)
      *BN = 128;
      *STG = 2;
    } else if (epi == EPI_F32 || FT * ((M + 159) / 160) >= 3 * 296) {
      // fp32 outputs, and residual updates of at least three waves: 160-token tiles (less shared-
      // memory fill per flop; M = 16320, N = 3840: 165 -> 152 us, M = 5120, N = 2304: 25.2 -> 20.6 us)
      *BN = 160;
    } else {
      *BN = 128;
    }
    return;
  }
  if (M > 512 && KB < 32) {
    // A few hundred to a few thousand tokens with a short K loop: no split (its exchange costs more
    // than the loop).  The time of these shapes is set by wave quantisation -- two CTAs fit on an SM,
    // 296 on the device, and a grid of 297 takes twice as long as one of 296 -- so the token tile is
    // the multiple of 16 up to 160 that minimises waves x (tile + fixed part); within one wave that
    // is the smallest tile, i.e. the most CTAs.  Measured (graph replay) on the layer shapes of
    // C2-C4: M = 1280, N = 4096 takes 16.3 us with 144-token tiles (288 CTAs) against 24.9 us with 96
    // (448 CTAs, two waves); M = 3072, N = 3072 27.5 us with 128 against 34.6 us with 96.
    int best = 96, best_cost = 1 << 30;
    for (int bnc = 64; bnc <= 160; bnc += 16) {
      const int ctas = FT * ((M + bnc - 1) / bnc);
      const int cost = ((ctas + 295) / 296) * (bnc + 48) * 10;
      if (cost < best_cost) { best = bnc; best_cost = cost; }
    }
    // With a two-stage ring a third CTA fits on the SM (444 on the device); such a CTA is about
    // 30 % slower, which pays where it saves a whole wave (M = 2048, N = 3072 GELU: 384 CTAs of 128
    // tokens, 23.7 -> 17.2 us; M = 3072, N = 2304: 432 CTAs, 16.9 -> 13.4 us).
    for (int bnc = 80; bnc <= 128; bnc += 16) {
      const int ctas = FT * ((M + bnc - 1) / bnc);
      const int cost = ((ctas + 443) / 444) * (bnc + 48) * 13;
      if (cost < best_cost) { best = bnc; best_cost = cost; *STG = 2; }
    }
    *BN = best;
    *S = 1;
    return;
  }
  if (M > 512) {
    // The same token counts with a long K loop: K split 2 or 4 ways; of the measured combinations
    // the one with the most CTAs within one wave.
    const int cand[5][2] = {{96, 2}, {128, 2}, {96, 4}, {128, 4}, {160, 4}};
    int bb = 128, bs = 2, best_ctas = 0;
    for (const auto &c : cand) {
      const int ctas = FT * ((M + c[0] - 1) / c[0]) * c[1];
      if (ctas <= 296 && ctas > best_ctas) { bb = c[0]; bs = c[1]; best_ctas = ctas; }
    }
    *BN = bb;
    *S = bs;
    return;
  }
  int bn = M <= 16 ? 16 : M <= 512 ? 32 : 128;
  const int tiles = FT * ((M + bn - 1) / bn);
  int s = 1;
  while (s * 2 <= SK_MAX_SPLIT && s * 2 <= KB && tiles * s * 2 <= 256) s *= 2;
  *BN = bn;
  *S = s;
}

static bool gemm_sk_launch(cudaStream_t st, bool pdl, GemmSkPlan &p, void *C, int M, int epi, int *status,
                           const SkNorm *norm = nullptr, LiveRows lr = LiveRows{nullptr, 0}) {
  if (!p.valid || M < 1 || M > p.M_max) return false;
  int BN, S, wt, stg;
  gemm_sk_geometry(p.N, p.K, M, epi, &BN, &S, &wt, &stg);
  const int idx = BN / 16 - 1;
  if (!p.haveA[idx]) {
    if (tc_encode(&p.mapA[idx], p.A, p.M_max, p.K, BN)) return false;
    p.haveA[idx] = true;
  }
  const int KB = (p.K + TC_BK - 1) / TC_BK;
  const int FT = (p.N + TC_BM - 1) / TC_BM, TT = (M + BN - 1) / BN;
  // residual epilogue through the TMA unit: x and its row pitch 16-byte aligned, whole feature tiles
  int tma_c = SK_TMA_NONE;
  if (!norm && p.N % TC_BM == 0 && BN % S == 0 && !((uintptr_t)C & 15)) {
    if (epi == EPI_RESID) tma_c = SK_TMA_ADD;
    else if (epi == EPI_F32) tma_c = SK_TMA_F32;
    else if ((epi == EPI_T || epi == EPI_GELU_T) && S == 1) tma_c = SK_TMA_BF16;
  }
  const CUtensorMap *mapC = &p.mapW;                         // placeholder when unused
  if (tma_c) {
    const int rows = BN / S;
    const bool hb = tma_c == SK_TMA_BF16;
    const GemmSkPlan::CMap *hit = nullptr;
    for (const auto &c : p.mapC)
      if (c.C == C && c.M == M && c.rows == rows && c.is_bf16 == hb) { hit = &c; break; }
    if (!hit) {
      GemmSkPlan::CMap c{C, M, rows, hb, {}};
      if (sk_encode_c(&c.map, C, M, p.N, rows, hb)) return false;
      p.mapC.push_back(c);
      hit = &p.mapC.back();
    }
    mapC = &hit->map;
  }
  const SkShape sh = sk_shape(BN, (KB + S - 1) / S, S > 1 || tma_c, wt, stg);
  if (sh.smem_bytes > 227 * 1024) return false;
  const int ring_bytes = sh.smem_bytes - 1024 - 256 - 1024;
  const SkNorm nm = norm ? *norm : SkNorm{};
  const int tc = tma_c;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((FT + wt - 1) / wt, TT, S);
  cfg.blockDim = dim3(192);
  cfg.dynamicSmemBytes = sh.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = S;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  int N = p.N, K = p.K, stages = sh.stages, cols = sh.tmem_cols, rb = ring_bytes;
  auto go = [&](auto kernel) {
    return cudaLaunchKernelEx(&cfg, kernel, p.mapW, p.mapA[idx], *mapC, C, M, N, K, BN, stages, cols, rb, epi, tc, nm, status,
                              lr) == cudaSuccess;
  };
  if (wt == 2) return go(gemm_sk_kernel<2, false>);
  return norm ? go(gemm_sk_kernel<1, true>) : go(gemm_sk_kernel<1, false>);
}

}  // namespace tsfm

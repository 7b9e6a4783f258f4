// bf16 x bf16 -> fp32 contraction on the sm_100a tensor cores.
//
//   C[t, f] (op)= sum_k A[t, k] * W[f, k]        A: [M, K] tokens, W: [N, K] weights
//
// "Swap-AB" form: the weight tile (128 output features) is the MMA's M operand and the
// token tile (BN = 16..256 tokens) its N operand, so that small token counts (draft steps,
// one-token decode, K+1-token verification) still fill the 128-row datapath and the
// weight stream is read exactly once.  Both operands are K-major; TMA brings 64-wide K
// slices into a 128-byte-swizzled shared-memory ring, one elected thread issues
// tcgen05.mma with the accumulator in tensor memory, and four warps drain it with
// tcgen05.ld, writing C transposed back to [token, feature] with coalesced rows.
//
// Warp roles (192 threads): warps 0-3 epilogue (TMEM lanes 32w..32w+31), warp 4 lane 0 TMA
// producer, warp 5 TMEM allocation + lane 0 MMA issuer.  Every mbarrier wait is bounded by
// wall-clock time; on expiry the kernel records a status code, skips the remaining work,
// still frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <mutex>
#include "common.cuh"
#include "kernels_simt.cuh"   // EPI_* codes

namespace tsfm {

constexpr int TC_BM = 128;         // output features per CTA (MMA M)
constexpr int TC_BK = 64;          // K elements per pipeline stage (one 128-byte swizzle row)
constexpr int TC_W_BYTES = TC_BM * TC_BK * 2;
// Bound of every mbarrier wait.  The longest legitimate wait is an epilogue warp waiting for its
// own CTA's main loop (tens of microseconds); 100 ms is far beyond that and short enough that a
// wedged pipeline gives the device back at once.
constexpr unsigned long long TC_WAIT_NS = 100000000ull;

struct GemmTcPlan {
  bool valid = false;
  int N = 0, K = 0;
  CUtensorMap mapW;                // weights [N, K], box 128 x 64
  CUtensorMap mapA[5];             // activations [M_max, K], box BN x 64, BN = 16 << i
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within TC_WAIT_NS.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it == 256) t0 = globaltimer_ns();
    if (it > 256 && (it & 255) == 0 && globaltimer_ns() - t0 > TC_WAIT_NS) return false;
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 bytes apart,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
  d |= (uint64_t)1 << 46;                          // version
  d |= (uint64_t)2 << 61;                          // layout: SWIZZLE_128B
  return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

template <int BN> struct TcShape {
  static constexpr int A_BYTES = BN * TC_BK * 2;
  static constexpr int STAGE_BYTES = TC_W_BYTES + A_BYTES;
  static constexpr int STAGES = (BN >= 256) ? 4 : (BN >= 128) ? 6 : 8;
  static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
};

// grid = (ceil(N / 128), ceil(M / BN), splits), block = 192, dynamic smem = TcShape<BN>::SMEM_BYTES.
// With splits > 1 CTA z reduces K blocks [z * KB / splits, (z + 1) * KB / splits) and the epilogue
// must be additive (EPI_RESID / EPI_ATOMIC): partial sums are added with fp32 atomics.
template <int BN>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapW, const __grid_constant__ CUtensorMap mapA,
               void *__restrict__ C, int M, int N, int K, int epi, int *__restrict__ status) {
  using S = TcShape<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = tiles + S::STAGES * S::STAGE_BYTES;      // 8-byte aligned
  const uint32_t full0 = bars, empty0 = bars + 8 * S::STAGES, accum = bars + 16 * S::STAGES;
  const uint32_t slot = accum + 8;
  uint32_t *slot_ptr = reinterpret_cast<uint32_t *>(smem_raw + (slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f0 = blockIdx.x * TC_BM, t0 = blockIdx.y * BN;
  const int KB_all = (K + TC_BK - 1) / TC_BK;
  const int kb_lo = (int)(((long long)KB_all * blockIdx.z) / gridDim.z);
  const int kb_hi = (int)(((long long)KB_all * (blockIdx.z + 1)) / gridDim.z);
  const int KB = kb_hi - kb_lo;
  const bool atomic = epi == EPI_ATOMIC || (epi == EPI_RESID && gridDim.z > 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(accum, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"((uint32_t)S::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *slot_ptr;

  if (warp == 4 && lane == 0) {
    // ---------------- TMA producer
    for (int kb = 0; kb < KB; ++kb) {
      const int s = kb % S::STAGES;
      const uint32_t ph = (uint32_t)(kb / S::STAGES) & 1u;
      if (!mbar_wait(empty0 + 8 * s, ph ^ 1u)) { atomicExch(status, DEV_TIMEOUT_TMA); break; }
      const uint32_t dst = tiles + s * S::STAGE_BYTES;
      mbar_expect_tx(full0 + 8 * s, S::STAGE_BYTES);
      tma_load_2d(dst, &mapW, (kb_lo + kb) * TC_BK, f0, full0 + 8 * s);
      tma_load_2d(dst + TC_W_BYTES, &mapA, (kb_lo + kb) * TC_BK, t0, full0 + 8 * s);
    }
  } else if (warp == 5 && lane == 0) {
    // ---------------- MMA issuer
    constexpr uint32_t idesc = umma_idesc(BN);
    bool ok = true;
    for (int kb = 0; kb < KB && ok; ++kb) {
      const int s = kb % S::STAGES;
      const uint32_t ph = (uint32_t)(kb / S::STAGES) & 1u;
      if (!mbar_wait(full0 + 8 * s, ph)) { atomicExch(status, DEV_TIMEOUT_MMA); ok = false; break; }
      tc_fence_after();
      const uint32_t sw = tiles + s * S::STAGE_BYTES;
      const uint64_t dw = umma_smem_desc(sw), da = umma_smem_desc(sw + TC_W_BYTES);
#pragma unroll
      for (int k = 0; k < TC_BK / 16; ++k)       // 16 K elements = 32 bytes = 2 descriptor units
        umma_bf16(tmem, dw + 2 * k, da + 2 * k, idesc, (kb | k) ? 1u : 0u);
      umma_commit(empty0 + 8 * s);               // frees the stage when these MMAs have read it
    }
    if (ok) umma_commit(accum);                  // accumulator complete
  } else if (warp < 4) {
    // ---------------- epilogue: lane = output feature, registers = tokens
    if (mbar_wait(accum, 0)) {
      tc_fence_after();
      const int f = f0 + warp * 32 + lane;
      const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 16) {
        if (t0 + c0 >= M) break;
        float v[16];
        tmem_ld16(tbase + c0, v);
        if (f < N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = t0 + c0 + j;
            if (t < M) {
              const size_t o = (size_t)t * N + f;
              if (atomic) atomicAdd((float *)C + o, v[j]);
              else if (epi == EPI_F32) ((float *)C)[o] = v[j];
              else if (epi == EPI_T) ((bf16 *)C)[o] = __float2bfloat16_rn(v[j]);
              else if (epi == EPI_GELU_T) ((bf16 *)C)[o] = __float2bfloat16_rn(gelu_erf(v[j]));
              else ((float *)C)[o] += v[j];
            }
          }
        }
      }
    } else if (lane == 0) {
      atomicExch(status, DEV_TIMEOUT_EPILOGUE);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)S::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*PFN_encodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);
static PFN_encodeTiled g_encode = nullptr;

template <int BN> static int gemm_tc_set_attr() {
  return cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TcShape<BN>::SMEM_BYTES) == cudaSuccess ? 0 : -4;
}

// Resolve the driver's tensor-map encoder (once per process) and opt the kernels into large
// shared memory (once per device: function attributes belong to the current device).  Calls from
// several threads are serialised.
constexpr int TC_MAX_DEVICES = 64;
static std::mutex g_tc_init_mu;
static int gemm_tc_init() {
  static bool dev_done[TC_MAX_DEVICES] = {false};
  std::lock_guard<std::mutex> lock(g_tc_init_mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TC_MAX_DEVICES) return -4;
  if (!g_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
      return -4;
    g_encode = (PFN_encodeTiled)fn;
  }
  if (dev_done[dev]) return 0;
  if (gemm_tc_set_attr<16>() || gemm_tc_set_attr<32>() || gemm_tc_set_attr<64>() || gemm_tc_set_attr<128>() ||
      gemm_tc_set_attr<256>())
    return -4;
  dev_done[dev] = true;
  return 0;
}

static int tc_encode(CUtensorMap *map, const void *base, int rows, int K, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -4;
}

// Describe W [N, K] and the activation buffer A [M_max, K] (both bf16, 16-byte aligned).
// Leaves plan->valid false (not an error) when the shape is outside the kernel's domain.
static int gemm_tc_plan(GemmTcPlan *plan, const void *W, int N, int K, const void *A, int M_max) {
  plan->valid = false;
  plan->N = N;
  plan->K = K;
  if (K % 8 || K < 16 || N < 1 || M_max < 1) return 0;   // row pitch must be a multiple of 16 bytes
  if (((uintptr_t)W & 15) || ((uintptr_t)A & 15)) return 0;
  if (!g_encode) return -4;
  if (tc_encode(&plan->mapW, W, N, K, TC_BM)) return -4;
  for (int i = 0; i < 5; ++i)
    if (tc_encode(&plan->mapA[i], A, M_max, K, 16 << i)) return -4;
  plan->valid = true;
  return 0;
}

// Token-tile width for M tokens.
static int gemm_tc_bn(int N, int M) {
  (void)N;
  if (M <= 16) return 16;
  if (M <= 32) return 32;
  if (M <= 64) return 64;
  if (M <= 128) return 128;
  return 256;
}

// Number of K splits: fill the SMs when the (feature tile x token tile) grid is small.  Only
// additive epilogues can be split.
static int gemm_tc_splits(int N, int K, int M, bool additive) {
  if (!additive) return 1;
  const int bn = gemm_tc_bn(N, M);
  const int tiles = ((N + TC_BM - 1) / TC_BM) * ((M + bn - 1) / bn);
  const int KB = (K + TC_BK - 1) / TC_BK;
  if (tiles >= 96 || KB < 2) return 1;
  int s = 148 / tiles;
  if (s > KB) s = KB;
  return s < 1 ? 1 : s;
}

template <int BN>
static void gemm_tc_launch_bn(cudaStream_t s, const GemmTcPlan &p, int idx, void *C, int M, int epi, int *status) {
  const bool additive = epi == EPI_RESID || epi == EPI_ATOMIC;
  dim3 grid((p.N + TC_BM - 1) / TC_BM, (M + BN - 1) / BN, gemm_tc_splits(p.N, p.K, M, additive));
  gemm_tc_kernel<BN><<<grid, 192, TcShape<BN>::SMEM_BYTES, s>>>(p.mapW, p.mapA[idx], C, M, p.N, p.K, epi, status);
}

// Launch on the plan's buffers (A must be the buffer the plan was made for).
static bool gemm_tc_launch(cudaStream_t s, const GemmTcPlan &p, const void *A, void *C, int M, int epi,
                           int *status) {
  (void)A;
  if (!p.valid) return false;
  switch (gemm_tc_bn(p.N, M)) {
    case 16: gemm_tc_launch_bn<16>(s, p, 0, C, M, epi, status); break;
    case 32: gemm_tc_launch_bn<32>(s, p, 1, C, M, epi, status); break;
    case 64: gemm_tc_launch_bn<64>(s, p, 2, C, M, epi, status); break;
    case 128: gemm_tc_launch_bn<128>(s, p, 3, C, M, epi, status); break;
    default: gemm_tc_launch_bn<256>(s, p, 4, C, M, epi, status); break;
  }
  return true;
}

}  // namespace tsfm

// Shared device/host helpers of the decoder library (types, conversions, reductions).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace tsfm {

typedef __nv_bfloat16 bf16;

// Device status codes written by kernels whose bounded waits expire (0 = fine).
// From DEV_GUARD_BASE on: guard region (code - DEV_GUARD_BASE) behind a buffer was overwritten.
enum : int { DEV_OK = 0, DEV_TIMEOUT_TMA = 1, DEV_TIMEOUT_MMA = 2, DEV_TIMEOUT_EPILOGUE = 3, DEV_GUARD_BASE = 16 };

// Guard regions of the bounds-checking mode: n_blocks runs of `len` bytes, `stride` bytes apart, that
// were filled with GUARD_BYTE when the handle was made and that no kernel may ever write (the bytes
// behind an allocation; the spare last row of every (layer, series, head) block of a KV cache; the
// spare last token of every series' history).
constexpr unsigned char GUARD_BYTE = 0xA5;
struct GuardRegion {
  const unsigned char *base;
  unsigned long long stride;
  unsigned int n_blocks, len;
};

// Per-forecast state in device memory.  The first block holds the call's parameters (written
// by the host before the work is enqueued, so that a captured graph can be replayed with new
// ones); the rest is loop state and phase clocks kept by the kernels themselves.
struct DevState {
  const float *series;            // [B, ctx_len] raw context values
  float *out;                     // [B, H] forecast
  float tau;                      // acceptance temperature (the paper's sigma; sigma_p of Eq. 5)
  float sigma_q;                  // draft surrogate scale (= tau in the deployed scheme)
  float fallback_r;               // r of t = mu_p + r eps (0 in the deployed scheme)
  int flags;                      // VAR_* bits
  uint32_t key0, key1;            // Philox key = forecast seed
  int round;                      // index of the round in flight
  unsigned long long t_call;      // %globaltimer stamps: call start, ...
  unsigned long long t_phase[3];  // ... start of this round's draft / verify / accept phase
  unsigned long long t_end;
  unsigned long long ns_prefill, ns_draft, ns_verify, ns_accept;   // accumulated phase times
};

enum : int { VAR_SAMPLE_PROPOSALS = 1, VAR_NO_TEMPERING = 2 };

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization
// attribute may start while its predecessor in the stream is still running; pdl_wait() blocks
// until that predecessor has completed and its writes are visible, pdl_release() lets the
// successor start its own preamble.  Both are no-ops for an ordinary launch.  Every kernel here
// calls pdl_wait() in every thread before its first access to memory another kernel writes.
// Pointers to such memory are never `const T *__restrict__` kernel parameters: loads through
// those compile to the read-only path (ld.global.nc), which promises data that no one writes while
// the kernel runs, and such a load whose address is known before the wait was seen to be
// scheduled ahead of it (attention read the previous pass's queries).  Only the constants of a
// handle (weights, gains, RoPE tables) carry the qualifier pair.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_sync() { pdl_wait(); pdl_release(); }

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over a whole block (all threads get the result); `scratch` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float *scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  float t = (lane < nw) ? scratch[lane] : 0.f;
  return warp_sum(t);
}
__device__ __forceinline__ double block_sum_d(double v, double *scratch) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum_d(v);
  __syncthreads();
  if (lane == 0) scratch[w] = v;
  __syncthreads();
  double t = (lane < nw) ? scratch[lane] : 0.0;
  return warp_sum_d(t);
}

// Exact (erf) GELU.
__device__ __forceinline__ float gelu_erf(float v) {
  return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
}

// The same function for epilogues that round their result to bf16: v * Phi(v) with
// erfc(z) = t (a1 + t (a2 + t (a3 + t (a4 + t a5)))) exp(-z^2), t = 1 / (1 + p z), z = |v| / sqrt(2)
// (Abramowitz & Stegun 7.1.26, absolute error of erf below 1.5e-7, far inside half a bf16 ulp),
// two special-function instructions and no branch instead of erff's two divergent paths.
// Phi(-|v|) = erfc(z) / 2 is taken directly, so the negative side has no cancellation.
__device__ __forceinline__ float gelu_erf_fast(float v) {
  const float z = fabsf(v) * 0.70710678118654752440f;
  const float t = __fdividef(1.0f, fmaf(0.3275911f, z, 1.0f));
  float poly = fmaf(t, 1.061405429f, -1.453152027f);
  poly = fmaf(t, poly, 1.421413741f);
  poly = fmaf(t, poly, -0.284496736f);
  poly = fmaf(t, poly, 0.254829592f);
  const float half_erfc = 0.5f * t * poly * __expf(-z * z);
  return v * (v >= 0.f ? 1.0f - half_erfc : half_erfc);
}

}  // namespace tsfm

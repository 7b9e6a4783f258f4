// Fused acceptance step of one speculative round (Sec. 3.2 Eq. 5, Sec. 3.3, Algorithm 1):
// per series, the K tempered Gaussian log-ratios, the K Philox uniforms, the first rejection
// by warp ballot, the correction / bonus patch, the new committed count (= the ragged KV
// rollback length) and the round's counters -- one warp per series, one launch per round.
#pragma once
#include "common.cuh"

namespace tsfm {

// Philox4x32-10 (Salmon et al., SC'11): 128-bit counter, 64-bit key, ten rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// u in (0, 1) on a 23-bit grid, exact in fp32: ((w >> 9) + 0.5) * 2^-23.
__device__ __forceinline__ float uniform_from_word(uint32_t w) {
  return ((float)(w >> 9) + 0.5f) * 1.1920928955078125e-07f;
}

// Standard normal draw for element e of a patch, for the sampled variants of Sec. 3.3: Box-Muller
// on the Philox words of counter (series, round, position, stream | e / 2); the even element takes
// the cosine branch, the odd one the sine branch.
constexpr uint32_t NOISE_PROPOSAL = 0x10000000u, NOISE_FALLBACK = 0x20000000u;
__device__ __forceinline__ float standard_normal(uint2 key, uint32_t series, uint32_t round, uint32_t pos,
                                                 uint32_t stream, int e) {
  const uint4 w = philox4x32_10(make_uint4(series, round, pos, stream | (uint32_t)(e >> 1)), key);
  const float rad = sqrtf(-2.f * logf(uniform_from_word(w.x)));
  float sn, cs;
  sincospif(2.f * uniform_from_word(w.y), &sn, &cs);
  return rad * ((e & 1) ? sn : cs);
}

__device__ float head_normal(const DevState *st, int series, int k_pos, int e) {
  return standard_normal(make_uint2(st->key0, st->key1), (uint32_t)series, (uint32_t)st->round, (uint32_t)k_pos, NOISE_PROPOSAL, e);
}

struct AcceptCounters {            // device mirror of the integer part of tsfm_stats
  unsigned long long drafted, tested, accepted, committed, near_margin;
  unsigned long long tested_by_pos[32], accepted_by_pos[32], L_hist[34];
};

struct AcceptArgs {
  // proposals x_i (= draft means in the deployed scheme) and draft means mu_q^(i):
  // element (b, i, :) at x + b * x_stride_b + i * P   (i = 0..K-1)
  const float *x, *mu_q;
  long long x_stride_b;
  // where the draft means live when they are not the proposals themselves (sampled proposals):
  // element (b, i, :) at mu_q_alt + (b * K + i) * P; NULL = use mu_q as above
  const float *mu_q_alt;
  const float *mu_p;               // [B, K+1, P] boundary predictions
  // where committed patches go: patch c of this round (c = 0..n) at
  // commit + b * commit_stride_b + c * P.  When commit_accepted == 0 the accepted
  // proposals already sit there and only the correction / bonus patch is written.
  float *commit;
  long long commit_stride_b;
  int commit_accepted;
  // commit_follows_done: the base above additionally advances by done[b] * P (history buffer)
  int commit_follows_done;
  int *done;                       // [B] in/out
  int B, K, P, T;
  float sigma_p, sigma_q, margin;
  uint2 key;
  int round_idx, series0;
  const float *forced_u;           // [B, K] or NULL
  int *n_accept;                   // [B] (or NULL)
  float *ell, *log_u;              // [B, K] (or NULL)
  AcceptCounters *ctr;             // or NULL
  int *unfinished;                 // or NULL: += 1 per series still short of T after this round
  // When st is non-NULL the scales (tau), the Philox key and the round index come from it, and
  // n_accept / ell / log_u / unfinished are per-round arrays indexed by that round.
  DevState *st;
};

// Closes a round: accumulates the phase clocks, advances the round counter, adds the round's
// kernel launches to the device-side launch counter, lists the series that still have patches
// to commit (ascending, for the next round's compacted passes) and, inside a captured graph, tells
// the WHILE node whether another round is needed.  One CTA of 256 threads.
__global__ void __launch_bounds__(256)
round_end_kernel(DevState *st, const int *unfinished, int T, cudaGraphConditionalHandle handle, int use_handle,
                 const int *body_launches, unsigned long long *launch_ctr, const int *done, int B,
                 int *live, int *n_live) {
  __shared__ int warp_count[8];
  __shared__ int base;
  pdl_sync();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int b0 = 0; b0 < B; b0 += 256) {             // ordered compaction, 256 series at a time
    const int b = b0 + threadIdx.x;
    const bool alive = b < B && done[b] < T;
    const unsigned m = __ballot_sync(0xffffffffu, alive);
    if (lane == 0) warp_count[w] = __popc(m);
    __syncthreads();
    int off = base;
    for (int i = 0; i < w; ++i) off += warp_count[i];
    if (alive) live[off + __popc(m & ((1u << lane) - 1u))] = b;
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
      for (int i = 0; i < 8; ++i) t += warp_count[i];
      base += t;
    }
    __syncthreads();
  }
  if (threadIdx.x != 0) return;
  *n_live = base;
  const int r = st->round;
  const unsigned long long now = globaltimer_ns();
  if (r == 0) st->ns_prefill = st->t_phase[0] - st->t_call;
  st->ns_draft += st->t_phase[1] - st->t_phase[0];
  st->ns_verify += st->t_phase[2] - st->t_phase[1];
  st->ns_accept += now - st->t_phase[2];
  st->round = r + 1;
  if (body_launches && launch_ctr) *launch_ctr += (unsigned long long)*body_launches;
  // every round commits at least one patch per unfinished series, so T rounds always suffice:
  // the second condition bounds the loop whatever the counters say
  if (use_handle) cudaGraphSetConditional(handle, (unfinished[r] > 0 && r + 1 < T) ? 1u : 0u);
}

// block = 128 (4 series per CTA), grid = ceil(B / 4).
__global__ void __launch_bounds__(128) accept_kernel(AcceptArgs a) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
  pdl_sync();
  if (a.st) {
    if (blockIdx.x == 0 && threadIdx.x == 0) a.st->t_phase[2] = globaltimer_ns();
    const int r = a.st->round;
    a.sigma_p = a.st->tau;
    a.sigma_q = a.st->sigma_q;
    a.key = make_uint2(a.st->key0, a.st->key1);
    a.round_idx = r;
    if (a.n_accept) a.n_accept += (size_t)r * a.B;
    if (a.ell) a.ell += (size_t)r * a.B * a.K;
    if (a.log_u) a.log_u += (size_t)r * a.B * a.K;
    if (a.unfinished) a.unfinished += r;
  }
  if (b >= a.B) return;
  const int m = a.done[b];
  if (m >= a.T) {                                   // finished earlier: nothing to decide
    if (lane == 0 && a.n_accept) a.n_accept[b] = -1;
    return;
  }
  const int K = a.K, P = a.P;
  const long long hist_adv = a.commit_follows_done ? (long long)m * P : 0;
  const float *xb = a.x + b * a.x_stride_b + hist_adv;
  const int flags = a.st ? a.st->flags : 0;
  const float fallback_r = a.st ? a.st->fallback_r : 0.f;
  const float *qb = (a.mu_q_alt && (flags & VAR_SAMPLE_PROPOSALS)) ? a.mu_q_alt + (size_t)b * a.K * a.P
                                                                     : a.mu_q + b * a.x_stride_b + hist_adv;
  const float *pb = a.mu_p + (size_t)b * (K + 1) * P;

  // energies ||x - mu_p||_d^2 and ||x - mu_q||_d^2 of every position; lane i keeps position i
  float my_ep = 0.f, my_eq = 0.f;
  for (int i = 0; i < K; ++i) {
    float ep = 0.f, eq = 0.f;
    for (int c = lane; c < P; c += 32) {
      const float xv = xb[(size_t)i * P + c];
      const float dp = xv - pb[(size_t)i * P + c];
      const float dq = xv - qb[(size_t)i * P + c];
      ep = fmaf(dp, dp, ep);
      eq = fmaf(dq, dq, eq);
    }
    ep = warp_sum(ep) / (float)P;
    eq = warp_sum(eq) / (float)P;
    if (lane == i) { my_ep = ep; my_eq = eq; }
  }
  // Eq. 5 and the log-domain test  log u <= min(l, 0)
  bool ok = true;
  float l = 0.f, lu = 0.f;
  if (lane < K) {
    l = -my_ep / (2.f * a.sigma_p * a.sigma_p) + my_eq / (2.f * a.sigma_q * a.sigma_q)
        + 0.5f * logf((a.sigma_q * a.sigma_q) / (a.sigma_p * a.sigma_p));
    if (flags & VAR_NO_TEMPERING) l *= (float)P;     // l is (1/d) log p/q: undo the 1/d (component ablation)
    float u;
    if (a.forced_u) u = a.forced_u[(size_t)b * K + lane];
    else u = uniform_from_word(philox4x32_10(
                 make_uint4((uint32_t)(a.series0 + b), (uint32_t)a.round_idx, (uint32_t)lane, 0u), a.key).x);
    lu = logf(u);
    ok = (lu <= l) && (lu <= 0.f);                   // log u <= min(l, 0); a NaN statistic compares false: rejected
    if (a.ell) a.ell[(size_t)b * K + lane] = l;
    if (a.log_u) a.log_u[(size_t)b * K + lane] = lu;
  }
  const unsigned rejected = __ballot_sync(0xffffffffu, !ok);     // lanes >= K vote "accepted"
  const int n = rejected ? min(__ffs(rejected) - 1, K) : K;      // leading accepts
  const int L = n + 1;
  const int keep = min(L, a.T - m);

  // commit: accepted proposals (if they are not in place already) then mu_p^(n+1)
  float *cb = a.commit + b * a.commit_stride_b + hist_adv;
  if (a.commit_accepted)
    for (int c = lane; c < n * P; c += 32) cb[c] = xb[c];
  for (int c = lane; c < P; c += 32) {
    float t = pb[(size_t)n * P + c];
    if (fallback_r != 0.f)                          // t = mu_p + r eps (Algorithm 1, correction and bonus)
      t += fallback_r * standard_normal(a.key, (uint32_t)(a.series0 + b), (uint32_t)a.round_idx, (uint32_t)n, NOISE_FALLBACK, c);
    cb[(size_t)n * P + c] = t;
  }

  const bool tested = lane < min(n + 1, K);
  const bool near = tested && fabsf(l - lu) < a.margin;
  const unsigned near_mask = __ballot_sync(0xffffffffu, near);
  if (a.ctr) {
    if (tested) {
      atomicAdd(&a.ctr->tested_by_pos[lane], 1ull);
      if (lane < n) atomicAdd(&a.ctr->accepted_by_pos[lane], 1ull);
    }
    if (lane == 0) {
      atomicAdd(&a.ctr->drafted, (unsigned long long)K);
      atomicAdd(&a.ctr->tested, (unsigned long long)min(n + 1, K));
      atomicAdd(&a.ctr->accepted, (unsigned long long)n);
      atomicAdd(&a.ctr->committed, (unsigned long long)keep);
      atomicAdd(&a.ctr->near_margin, (unsigned long long)__popc(near_mask));
      atomicAdd(&a.ctr->L_hist[L], 1ull);
    }
  }
  if (lane == 0) {
    if (a.unfinished && m + keep < a.T) atomicAdd(a.unfinished, 1);
    a.done[b] = m + keep;
    if (a.n_accept) a.n_accept[b] = n;
  }
}

}  // namespace tsfm

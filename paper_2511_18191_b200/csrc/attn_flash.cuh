// Causal attention over a bf16 KV cache with a running softmax (one pass over the keys).
//
// Work unit = one warp: 16 queries (the M side of mma.sync m16n8k16) against a range of keys of
// one (series, head).  The warp streams its keys in chunks of 32 through a private ring of
// shared-memory stages filled by 16-byte asynchronous copies, and keeps, per query row, the
// running maximum m, the running sum l of exp(s - m) and the unnormalised output o in registers:
//     m' = max(m, max_t s_t),  l' = l e^(m - m') + sum_t e^(s_t - m'),  o' = o e^(m - m') + sum_t e^(s_t - m') v_t.
// No block-wide barrier is needed while the keys stream.
//   mode FLASH_TILES: passes of more than 16 tokens.  kv_append_kernel has put the keys and values
//              of the pass into the cache; the four warps of a CTA take four consecutive query
//              tiles (64 queries), each over all keys its queries may see.
//              grid = (heads, B, ceil(q_len / 64)).
//   mode FLASH_SPLIT: passes of at most 16 tokens (one query tile), long rows.  The cached keys
//              [0, pos0) are dealt out over the four warps; the last warp also takes the keys of
//              the pass itself, which it rotates, rounds, puts into a stage of its ring and
//              appends to the cache; the four (m, l, o) are merged through shared memory.
//              grid = (heads, B, 1).
//   mode FLASH_WARP: the same passes on short rows with many (series, head) pairs: each warp
//              takes one pair on its own (cached keys, then the keys of the pass).
//              grid = (ceil(B * heads / 4), 1, 1).
//   NB = 1, 2 (the last two modes, caches of at most 32 NB rows): a warp's cached keys and the
//              keys of the pass share one stage of 32 NB rows and are processed as NB chunks; the
//              CTA then asks for 8 NB KB per warp (head size 64) instead of a ring of 24 KB, so
//              that more of these latency-bound warps fit on an SM.  NB = 0: the ring.
// S = Q K^T uses the rotated, scaled fp32 queries split into a bf16 high and low part (two MMAs),
// so the scores keep fp32-like accuracy; P is rounded to bf16 for P V.  Scores are kept in
// base-2 units (the queries carry log2(e) / sqrt(DH)).
#pragma once
#include "common.cuh"
#include "kernels_simt.cuh"

namespace tsfm {

enum { FLASH_WARP = 0, FLASH_TILES = 1, FLASH_SPLIT = 4 };

template <int DH, int ST = 3> struct FlashGeom {
  static constexpr int CHUNK = 32;                              // keys per stage
  static constexpr int STAGES = ST;                             // ring depth (3: prefill tiles; 2: one-tile passes)
  static constexpr int ROW_BYTES = DH * 2;
  static constexpr int TILE_BYTES = CHUNK * ROW_BYTES;          // keys (or values) of one stage
  static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  static constexpr int WARP_BYTES = STAGES * STAGE_BYTES;       // also holds (o, m, l) for the merge
  static constexpr int SMEM_BYTES = 4 * WARP_BYTES;
  static_assert(STAGE_BYTES >= 16 * DH * 4 + 2 * 16 * 4, "merge buffers must fit in one stage");
  static constexpr int single_bytes(int nb) { return 4 * nb * STAGE_BYTES; }   // CTA, single stage of 32 nb rows
};

// 16-byte chunk c of row r sits at chunk (c ^ f(r)) of that row: the eight rows that one
// ldmatrix phase reads then fall into eight different 16-byte bank groups.
template <int DH> __device__ __forceinline__ int flash_swz(int r, int c) {
  return DH == 32 ? (c ^ ((r >> 1) & 3)) : (c ^ (r & 7));
}

__device__ __forceinline__ void flash_ldsm4(uint32_t addr, uint32_t (&d)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(addr));
}
__device__ __forceinline__ void flash_ldsm4_trans(uint32_t addr, uint32_t (&d)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]) : "r"(addr));
}
__device__ __forceinline__ void flash_cp16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void flash_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void flash_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int DH, int NB, int ST>
__device__ __forceinline__ void
attn_flash_body(const float *qkv, bf16 *__restrict__ Kc, bf16 *__restrict__ Vc,
                const float2 *__restrict__ rope, const PassGeom &g, int n_heads, int n_pairs, int mode,
                bf16 *__restrict__ out) {
  constexpr bool single = NB > 0;
  using G = FlashGeom<DH, ST>;
  constexpr int S_TILE = (NB > 0 ? NB : 1) * G::TILE_BYTES;     // key (or value) rows of the single stage
  constexpr int HALF = DH / 2, KS = DH / 16, CPR = DH / 8;     // k-steps of Q K^T, 16-byte chunks per row
  extern __shared__ __align__(128) unsigned char flash_smem[];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int gr = lane >> 2, q4 = lane & 3;                     // fragment row group, column pair
  const int d = n_heads * DH;
  int h = blockIdx.x, slot = blockIdx.y;
  if (mode == FLASH_WARP) {
    const int pair = blockIdx.x * 4 + w;
    if (pair >= n_pairs) return;                               // no block-wide barrier in this mode
    slot = pair / n_heads;
    h = pair % n_heads;
  }
  const int warp_bytes = single ? 2 * S_TILE : G::WARP_BYTES;   // shared memory of one warp
  unsigned char *ring = flash_smem + (size_t)w * warp_bytes;
  const uint32_t ring32 = (uint32_t)__cvta_generic_to_shared(ring);
  const SlotPos sp = slot_lookup(g, slot);                     // before the dependency wait: see SlotPos
  // Passes of one query tile also start streaming their cached keys before the dependency wait: rows
  // below pos0 of this layer's cache were written by this layer's attention in an earlier pass, a
  // whole layer of kernels ago at least.  Passes of several tiles read the rows that the directly
  // preceding kernel (kv_append_kernel) has just appended: they wait first.
  if (mode == FLASH_TILES) pdl_sync();
  if (sp.dead) return;                                         // per warp (FLASH_WARP) or per CTA: no barrier is pending
  const int b = sp.b, p0 = sp.p0;
  const size_t row0 = (size_t)slot * g.q_len;
  bf16 *Kb = Kc + ((size_t)b * n_heads + h) * g.cap * DH;
  bf16 *Vb = Vc + ((size_t)b * n_heads + h) * g.cap * DH;

  // this warp's queries [jq, jq + 16), cached keys [t_beg, t_end), and whether it takes the
  // keys of the pass itself as one more chunk
  int jq = 0, t_beg = 0, t_end = p0;
  bool own_pass_keys = true;
  if (mode == FLASH_TILES) {
    jq = (blockIdx.z * 4 + w) * 16;
    if (jq >= g.q_len) return;                                 // no block-wide barrier in this mode
    t_end = p0 + min(jq + 16, g.q_len);
    own_pass_keys = false;
  } else if (mode == FLASH_SPLIT) {
    // whole chunks, the keys of the pass counted as one more chunk at the end
    const int R = (((p0 + G::CHUNK - 1) / G::CHUNK + 1 + 3) / 4) * G::CHUNK;
    t_beg = min(w * R, p0);
    t_end = min(t_beg + R, p0);
    own_pass_keys = w == 3;
  }
  const int nq = min(16, g.q_len - jq);
  const int n_c = t_end - t_beg;                               // cached keys of this warp
  const int nch = single ? 0 : (n_c + G::CHUNK - 1) / G::CHUNK;   // chunks that go through the ring

  auto issue = [&](int c) {
    if (c < nch) {
      const int t0 = t_beg + c * G::CHUNK;
      const uint32_t kst = ring32 + (uint32_t)((c % G::STAGES) * G::STAGE_BYTES), vst = kst + G::TILE_BYTES;
#pragma unroll
      for (int i = 0; i < CPR; ++i) {
        const int idx = i * 32 + lane, r = idx / CPR, ch = idx % CPR;
        const int t = min(t0 + r, t_end - 1);                  // rows past the range repeat its last key (masked below)
        const uint32_t off = (uint32_t)(r * G::ROW_BYTES + flash_swz<DH>(r, ch) * 16);
        flash_cp16(kst + off, Kb + (size_t)t * DH + ch * 8);
        flash_cp16(vst + off, Vb + (size_t)t * DH + ch * 8);
      }
    }
    flash_commit();
  };
  if (single) {
    for (int idx = lane; idx < n_c * CPR; idx += 32) {
      const int r = idx / CPR, ch = idx % CPR;
      const uint32_t off = (uint32_t)(r * G::ROW_BYTES + flash_swz<DH>(r, ch) * 16);
      flash_cp16(ring32 + off, Kb + (size_t)(t_beg + r) * DH + ch * 8);
      flash_cp16(ring32 + S_TILE + off, Vb + (size_t)(t_beg + r) * DH + ch * 8);
    }
    flash_commit();
  } else {
#pragma unroll
    for (int c = 0; c < G::STAGES - 1; ++c) issue(c);
  }
  // q, k, v of the pass come from the preceding kernel.  They are read with ld.global.cg: their
  // addresses are known before the wait, and a load on the read-only path (what a plain load through
  // a const __restrict__ pointer compiles to) may be scheduled ahead of it.
  if (mode != FLASH_TILES) pdl_sync();

  // rotated, scaled queries as A fragments (rows gr and gr + 8), high and low bf16 parts
  uint32_t qhi[KS][4], qlo[KS][4];
  {
    const float sc = rsqrtf((float)DH) * 1.4426950408889634f;
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int i = gr + rr * 8, j = jq + i;
      const bool live = i < nq;
      const float *src = qkv + (row0 + (live ? j : jq)) * 3 * d + h * DH;
      const float2 *rp = rope + (size_t)(p0 + (live ? j : jq)) * HALF;
#pragma unroll
      for (int ks = 0; ks < KS / 2; ++ks)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int c = ks * 16 + hh * 8 + q4 * 2;             // first-half dims c, c + 1; partners c + HALF
          const float2 q1 = __ldcg(reinterpret_cast<const float2 *>(src + c));   // (not a read-only-path load: see below)
          const float2 q2 = __ldcg(reinterpret_cast<const float2 *>(src + c + HALF));
          const float4 cs = *reinterpret_cast<const float4 *>(rp + c);      // cos0 sin0 cos1 sin1
          float a0 = (q1.x * cs.x - q2.x * cs.y) * sc, a1 = (q1.y * cs.z - q2.y * cs.w) * sc;
          float b0 = (q2.x * cs.x + q1.x * cs.y) * sc, b1 = (q2.y * cs.z + q1.y * cs.w) * sc;
          if (!live) a0 = a1 = b0 = b1 = 0.f;
          split_bf16x2(a0, a1, qhi[ks][hh * 2 + rr], qlo[ks][hh * 2 + rr]);
          split_bf16x2(b0, b1, qhi[ks + KS / 2][hh * 2 + rr], qlo[ks + KS / 2][hh * 2 + rr]);
        }
    }
  }

  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const int qpos0 = p0 + jq + gr;                              // position of row gr; row gr + 8 is 8 further

  // one chunk: 32 keys at positions t0.. from the stage at kst (values at vst); keys at or past
  // t_lim, and keys after a query's own position, are masked
  auto chunk = [&](uint32_t kst, uint32_t vst, int t0, int t_lim) {
    // ---- scores of 16 queries x 32 keys
    float s[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
    for (int n2 = 0; n2 < 2; ++n2) {
      const int r = n2 * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;        // key row this lane addresses
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t bk[4];
        flash_ldsm4(kst + (uint32_t)(r * G::ROW_BYTES + flash_swz<DH>(r, ks * 2 + ((lane >> 3) & 1)) * 16), bk);
        mma_bf16_16816(s[n2 * 2], qhi[ks], bk[0], bk[1]);
        mma_bf16_16816(s[n2 * 2], qlo[ks], bk[0], bk[1]);
        mma_bf16_16816(s[n2 * 2 + 1], qhi[ks], bk[2], bk[3]);
        mma_bf16_16816(s[n2 * 2 + 1], qlo[ks], bk[2], bk[3]);
      }
    }
    // ---- causal mask and range end (only chunks that reach either)
    if (t0 + G::CHUNK > t_lim || t0 + G::CHUNK - 1 > p0 + jq) {
#pragma unroll
      for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int t = t0 + n * 8 + q4 * 2 + (e & 1);
          if (t >= t_lim || t > qpos0 + (e >> 1) * 8) s[n][e] = -INFINITY;
        }
    }
    // ---- running softmax
    uint32_t pa[2][4];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      float mx = -INFINITY;
#pragma unroll
      for (int n = 0; n < 4; ++n) mx = fmaxf(mx, fmaxf(s[n][rr * 2], s[n][rr * 2 + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run[rr], mx);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;    // nothing visible yet: every p below is 0
      const float alpha = exp2f(m_run[rr] - m_use);
      m_run[rr] = m_new;
      float sum = 0.f;
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const float p0v = exp2f(s[n][rr * 2] - m_use), p1v = exp2f(s[n][rr * 2 + 1] - m_use);
        sum += p0v + p1v;
        pa[n >> 1][(n & 1) * 2 + rr] = pack_bf16x2(p0v, p1v);
      }
      l_run[rr] = fmaf(l_run[rr], alpha, sum);
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) { o[n][rr * 2] *= alpha; o[n][rr * 2 + 1] *= alpha; }
    }
    // ---- o += P V
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
      const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int n0 = 0; n0 < DH / 8; n0 += 2) {
        uint32_t bv[4];
        flash_ldsm4_trans(vst + (uint32_t)(r * G::ROW_BYTES + flash_swz<DH>(r, n0 + (lane >> 4)) * 16), bv);
        mma_bf16_16816(o[n0], pa[kk], bv[0], bv[1]);
        mma_bf16_16816(o[n0 + 1], pa[kk], bv[2], bv[3]);
      }
    }
  };

  // Keys and values of this pass (at most 16 tokens) first, while the copies of the first cached
  // chunks are in flight: rotate the keys, round both to bf16, append them to the cache and put
  // them into the ring's last stage, which is not used before its first refill -- or, with a
  // single stage, behind the cached rows.  Value rows past the last key of a stage are zeroed:
  // their probabilities are 0, but 0 x NaN would not be.  One lane handles the element pairs
  // (c, c + 1) and (c + HALF, c + HALF + 1) of a token.
  {
    unsigned char *st = ring + (single ? 0 : (G::STAGES - 1) * G::STAGE_BYTES);
    uint32_t *ks = reinterpret_cast<uint32_t *>(st), *vs = reinterpret_cast<uint32_t *>(st + S_TILE);
    const int in_base = single ? n_c : 0;                      // stage row of the pass's first key
    int filled = single ? n_c : G::CHUNK;                      // stage rows that hold (or will hold) keys
    if (own_pass_keys) {
#pragma unroll 2
      for (int i = lane; i < g.q_len * (HALF / 2); i += 32) {
        const int j = i / (HALF / 2), c = (i % (HALF / 2)) * 2, jr = in_base + j;
        const float *src = qkv + (row0 + j) * 3 * d + h * DH;
        const int tg = p0 + j;
        const float4 cs = *reinterpret_cast<const float4 *>(rope + (size_t)tg * HALF + c);   // cos0 sin0 cos1 sin1
        const float2 ka = __ldcg(reinterpret_cast<const float2 *>(src + d + c));
        const float2 kb = __ldcg(reinterpret_cast<const float2 *>(src + d + c + HALF));
        const float2 va = __ldcg(reinterpret_cast<const float2 *>(src + 2 * d + c));
        const float2 vb = __ldcg(reinterpret_cast<const float2 *>(src + 2 * d + c + HALF));
        const uint32_t k1 = pack_bf16x2(ka.x * cs.x - kb.x * cs.y, ka.y * cs.z - kb.y * cs.w);
        const uint32_t k2 = pack_bf16x2(kb.x * cs.x + ka.x * cs.y, kb.y * cs.z + ka.y * cs.w);
        const uint32_t v1 = pack_bf16x2(va.x, va.y), v2 = pack_bf16x2(vb.x, vb.y);
        const int w1 = c / 2, w2 = (c + HALF) / 2;               // 32-bit words of the row
        const int a1 = jr * (DH / 2) + flash_swz<DH>(jr, w1 >> 2) * 4 + (w1 & 3);
        const int a2 = jr * (DH / 2) + flash_swz<DH>(jr, w2 >> 2) * 4 + (w2 & 3);
        ks[a1] = k1; ks[a2] = k2;
        vs[a1] = v1; vs[a2] = v2;
        uint32_t *kg = reinterpret_cast<uint32_t *>(Kb + (size_t)tg * DH);
        uint32_t *vg = reinterpret_cast<uint32_t *>(Vb + (size_t)tg * DH);
        kg[w1] = k1; kg[w2] = k2;
        vg[w1] = v1; vg[w2] = v2;
      }
      filled = in_base + g.q_len;
    }
    // (zero up to the end of the last 32-row block that holds a key)
    for (int i = filled * (DH / 2) + lane; i < ((filled + G::CHUNK - 1) & ~(G::CHUNK - 1)) * (DH / 2); i += 32) vs[i] = 0u;
    if (single) {
      flash_wait<0>();
      __syncwarp();
      const int t_lim = own_pass_keys ? p0 + g.q_len : t_end;
#pragma unroll
      for (int blk = 0; blk < NB; ++blk)
        if (filled > blk * G::CHUNK)
          chunk(ring32 + (uint32_t)(blk * G::TILE_BYTES), ring32 + (uint32_t)(S_TILE + blk * G::TILE_BYTES),
                t_beg + blk * G::CHUNK, t_lim);
    } else if (own_pass_keys) {
      __syncwarp();
      const uint32_t st32 = ring32 + (uint32_t)((G::STAGES - 1) * G::STAGE_BYTES);
      chunk(st32, st32 + G::TILE_BYTES, p0, p0 + g.q_len);
      // the first refill of this stage follows the warp barrier at the top of the loop below
    }
  }

  for (int c = 0; c < nch; ++c) {
    flash_wait<G::STAGES - 2>();
    __syncwarp();
    issue(c + G::STAGES - 1);                                  // refills the stage consumed in the previous turn
    const uint32_t kst = ring32 + (uint32_t)((c % G::STAGES) * G::STAGE_BYTES);
    chunk(kst, kst + G::TILE_BYTES, t_beg + c * G::CHUNK, t_end);
  }
  flash_wait<0>();
  __syncwarp();

#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    l_run[rr] += __shfl_xor_sync(0xffffffffu, l_run[rr], 1);
    l_run[rr] += __shfl_xor_sync(0xffffffffu, l_run[rr], 2);
  }
  if (mode != FLASH_SPLIT) {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int i = gr + rr * 8;
      if (i >= nq) continue;
      const float inv = 1.f / l_run[rr];
      uint32_t *dst = reinterpret_cast<uint32_t *>(out + (row0 + jq + i) * d + h * DH);
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) dst[n * 4 + q4] = pack_bf16x2(o[n][rr * 2] * inv, o[n][rr * 2 + 1] * inv);
    }
    return;
  }
  // ---- merge the four key ranges: this warp's (o, m, l) into its ring, then every thread combines
  float *ob = reinterpret_cast<float *>(ring);                 // [16][DH]
  float *mb = ob + 16 * DH, *lb = mb + 16;                     // [16], [16]
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int i = gr + rr * 8;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n)
      *reinterpret_cast<float2 *>(ob + i * DH + n * 8 + q4 * 2) = make_float2(o[n][rr * 2], o[n][rr * 2 + 1]);
    if (q4 == 0) { mb[i] = m_run[rr]; lb[i] = l_run[rr]; }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nq * (DH / 2); idx += blockDim.x) {
    const int i = idx / (DH / 2), c = (idx % (DH / 2)) * 2;
    float m = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < 4; ++ww)
      m = fmaxf(m, reinterpret_cast<const float *>(flash_smem + (size_t)ww * warp_bytes)[16 * DH + i]);
    float l = 0.f, ox = 0.f, oy = 0.f;
#pragma unroll
    for (int ww = 0; ww < 4; ++ww) {
      const float *wb = reinterpret_cast<const float *>(flash_smem + (size_t)ww * warp_bytes);
      const float mw = wb[16 * DH + i];
      if (mw == -INFINITY) continue;                           // that range held no visible key
      const float sc = exp2f(mw - m);
      const float2 ov = *reinterpret_cast<const float2 *>(wb + i * DH + c);
      l = fmaf(wb[16 * DH + 16 + i], sc, l);
      ox = fmaf(ov.x, sc, ox);
      oy = fmaf(ov.y, sc, oy);
    }
    const float inv = 1.f / l;
    *reinterpret_cast<uint32_t *>(out + (row0 + jq + i) * d + h * DH + c) = pack_bf16x2(ox * inv, oy * inv);
  }
}

// The ring variant (ST stages per warp) and the single-stage variant; the latter is compiled
// for four CTAs per SM where the head size allows it.
template <int DH, int ST>
__global__ void __launch_bounds__(128)
attn_flash_kernel(const float *qkv, bf16 *__restrict__ Kc, bf16 *__restrict__ Vc,
                  const float2 *__restrict__ rope, PassGeom g, int n_heads, int n_pairs, int mode,
                  bf16 *__restrict__ out) {
  attn_flash_body<DH, 0, ST>(qkv, Kc, Vc, rope, g, n_heads, n_pairs, mode, out);
}
template <int DH, int NB>
__global__ void __launch_bounds__(128, DH <= 64 ? (NB == 1 ? 4 : 3) : 1)
attn_flash_single_kernel(const float *qkv, bf16 *__restrict__ Kc, bf16 *__restrict__ Vc,
                         const float2 *__restrict__ rope, PassGeom g, int n_heads, int n_pairs, int mode,
                         bf16 *__restrict__ out) {
  attn_flash_body<DH, NB, 3>(qkv, Kc, Vc, rope, g, n_heads, n_pairs, mode, out);
}

}  // namespace tsfm

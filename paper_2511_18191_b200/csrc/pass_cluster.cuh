// One whole causal pass of a patch transformer over a few new tokens per series, as ONE kernel:
// the weight-streaming path for small batches (draft steps, one-token decode, K+1-token
// verification).
//
// Series never interact, so the batch is cut into groups of series and each group is given to
// one thread-block cluster of R = n_heads CTAs that runs the complete pass for its tokens --
// embedding, every layer, final norm and mean head -- with nothing but cluster-local
// synchronisation: no kernel boundary and no grid-wide barrier between the ~5 dependent stages
// of a layer.  Every cluster streams all the weights once (they sit in the L2 cache for the
// model sizes this path accepts), split over its CTAs:
//   CTA r owns attention head r: it computes q_r, k_r, v_r for all the cluster's tokens
//   (tcgen05.mma, weight tiles by TMA through one mbarrier ring that runs ahead across stage and
//   layer boundaries), appends k_r, v_r to the KV cache, runs causal attention for its head, and
//   multiplies by its 64-column slice of W_o: a K-split partial of the attention output
//   projection.  The partials meet in distributed shared memory: the CTA that owns a token row
//   (row t belongs to CTA t mod R) adds them to its fp32 residual row, applies the next
//   RMSNorm to the complete row and scatters the bf16 result into every CTA's operand buffer.
//   The MLP is cut the same way: CTA r owns d_ff / R hidden units (W_1 rows, then the matching
//   W_2 columns as a K-split partial), and the mean head is K-split over the CTAs as well.
// Activations never leave shared memory between the embedding and the head.
//
// Shapes: head size 64, 1 <= n_heads <= 8, d_model = 64 * n_heads a multiple of 128,
// (d_ff / n_heads) a multiple of 128, patch length <= 128, at most 32 tokens per cluster.
// Warp roles: warps 0-3 compute (128 threads = 128 TMEM lanes), warp 4 lane 0 TMA producer,
// warp 5 TMEM allocation + lane 0 MMA issuer.  Every wait is bounded; a wait that expires sets
// the status word and a CTA-wide abort flag, and every role falls through to the common exit.
#pragma once
#include "gemm_tc.cuh"

namespace tsfm {

constexpr int CL_MAX_R = 8;
constexpr int CL_MAX_BN = 32;
constexpr int CL_TILE_BYTES = TC_BM * TC_BK * 2;          // 16 KB weight tile
constexpr unsigned long long CL_WAIT_NS = 300000000ull;   // 0.3 s

struct alignas(64) ClLayer {
  CUtensorMap qkv;          // Wq|Wk|Wv [3d, d], box 64 rows x 64
  CUtensorMap wo;           // [d, d],  box 128 x 64
  CUtensorMap w1;           // [ff, d], box 128 x 64
  CUtensorMap w2;           // [d, ff], box 128 x 64
  const float *g1, *g2;
  bf16 *Kc, *Vc;            // this layer's cache [B][heads][cap][64]
};
struct alignas(64) ClModel {
  CUtensorMap head;         // W_head [P, d], box 128 x 64 (rows past P read as zero)
  const bf16 *W_emb;        // [d, P]
  const float *g_f;
  const float2 *rope;       // [cap][32]
  int n_layers, d, heads, ff, P;
};

struct ClArgs {
  const ClModel *model;
  const ClLayer *layers;
  const float *hist_in;     // [B][cap][P] history (tokens of this pass are read from it)
  float *hist_out;          // same buffer: the last token's prediction goes to its next slot
  float *vout;              // [B][q_len][P] (head_all)
  PassGeom g;
  int B, Bg, BN, stages, head_all;
  float eps;
  int *status;
  unsigned long long *stamp;
};

// ------------------------------------------------------------------ small PTX helpers
__device__ __forceinline__ uint32_t cl_mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cl_st_remote_v2(uint32_t raddr, uint32_t a, uint32_t b) {
  asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(raddr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ float4 cl_ld_remote_f4(uint32_t raddr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(raddr) : "memory");
  return v;
}
__device__ __forceinline__ float cl_ld_remote_f1(uint32_t raddr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(raddr) : "memory");
  return v;
}
__device__ __forceinline__ void cl_arrive_remote(uint32_t raddr) {   // ordering comes from a preceding cluster fence
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(raddr) : "memory");
}
__device__ __forceinline__ void cl_arrive_local(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool cl_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void cl_fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void cl_fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
__device__ __forceinline__ void cl_bar_compute() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Bounded wait that also gives up as soon as another role of this CTA has aborted.
__device__ __forceinline__ bool cl_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, bool cluster_scope) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (cluster_scope ? cl_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if ((it & 63) == 63) {
      if (*abort_flag) return false;
      if (t0 == 0) t0 = globaltimer_ns();
      else if (globaltimer_ns() - t0 > CL_WAIT_NS) return false;
    }
  }
}

// Byte offset of element (row t, column k) of a K-major bf16 operand [rows][K] in the 128-byte
// swizzled layout tcgen05.mma reads: 64-column blocks of rows x 128 B, 16-byte chunks XOR-ed with
// the row index modulo 8.
__device__ __forceinline__ uint32_t cl_opnd_off(int t, int k, int rows) {
  const int kb = k >> 6, c = k & 63;
  return (uint32_t)(kb * rows * 128 + t * 128 + ((((c >> 3) ^ (t & 7))) << 4) + ((c & 7) << 1));
}

struct ClSmem {           // byte offsets from the 1024-aligned base
  int ring, a_buf, ao_buf, h_buf, part, qkv, xrow, sc, zs, red, bars, total;
};
__host__ __device__ inline ClSmem cl_smem_layout(int d, int ffr, int BN, int R, int stages, int cap, int P) {
  ClSmem s;
  int o = 0;
  s.ring = o; o += stages * CL_TILE_BYTES;
  s.a_buf = o; o += (d / 64) * BN * 128;
  s.ao_buf = o; o += BN * 128;
  s.h_buf = o; o += (ffr / 64) * BN * 128;
  s.part = o; o += BN * d * 4;
  s.qkv = o; o += BN * 192 * 4;
  s.xrow = o; o += ((BN + R - 1) / R) * d * 4;
  s.sc = o; o += 4 * ((cap + 3) & ~3) * 4;
  s.zs = o; o += ((P + 3) & ~3) * 4;
  s.red = o; o += 64;
  s.bars = o; o += 512;
  s.total = o + 1024;
  return s;
}

// Work of the four compute warps (threads 0..127) of one CTA; see the file header.
__device__ __noinline__ void cl_compute(const ClArgs &a, uint8_t *sm, const ClSmem &so, uint32_t base32, uint32_t tmem,
                                        uint32_t acc_bar, uint32_t opnd_bar, uint32_t cbar, volatile int *abort_flag) {
  const ClModel &md = *a.model;
  const int R = md.heads, d = md.d, ffr = md.ff / md.heads, L = md.n_layers, P = md.P;
  const int TD = d / 128, TF = ffr / 128, BN = a.BN;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = blockIdx.x, grp = blockIdx.y;
  const int q_len = a.g.q_len, cap = a.g.cap, capr = (cap + 3) & ~3;
  const int b0 = grp * a.Bg, nb = min(a.Bg, a.B - b0), Mc = nb * q_len;
  float *part = reinterpret_cast<float *>(sm + so.part);
  float *qkv = reinterpret_cast<float *>(sm + so.qkv);
  float *xrow = reinterpret_cast<float *>(sm + so.xrow);
  float *sc = reinterpret_cast<float *>(sm + so.sc);
  float *zs = reinterpret_cast<float *>(sm + so.zs);
  float *red = reinterpret_cast<float *>(sm + so.red);
  uint8_t *ao_buf = sm + so.ao_buf, *h_buf = sm + so.h_buf;
  uint32_t rem_abuf[CL_MAX_R], rem_part[CL_MAX_R], rem_cbar[CL_MAX_R];
#pragma unroll
  for (int rr = 0; rr < CL_MAX_R; ++rr) {
    const uint32_t rank = rr < R ? rr : 0;
    rem_abuf[rr] = cl_mapa(base32 + so.a_buf, rank);
    rem_part[rr] = cl_mapa(base32 + so.part, rank);
    rem_cbar[rr] = cl_mapa(cbar, rank);
  }
  const uint32_t tbase = tmem + ((uint32_t)(warp * 32) << 16);
  int gi = 0, ci = 0;

  pdl_sync();
  if (a.stamp && r == 0 && grp == 0 && tid == 0) *a.stamp = globaltimer_ns();

  auto fail = [&]() {
    if (lane == 0) atomicExch(a.status, DEV_TIMEOUT_EPILOGUE);
    *abort_flag = 1;
  };
  // all compute threads of all CTAs of the cluster meet here; earlier (distributed) shared-memory
  // writes of every participant are visible afterwards
  auto csync = [&]() -> bool {
    cl_bar_compute();
    if (tid == 0) {
      cl_fence_cluster();
      for (int rr = 0; rr < R; ++rr) cl_arrive_remote(rem_cbar[rr]);
    }
    const bool w = cl_wait(cbar, (uint32_t)ci & 1u, abort_flag, true);
    ++ci;
    return w;
  };
  auto wait_acc = [&]() -> bool {
    const bool w = cl_wait(acc_bar, (uint32_t)gi & 1u, abort_flag, false);
    ++gi;
    tc_fence_after();
    return w;
  };
  auto operand_ready = [&]() {
    tc_fence_before();
    cl_fence_proxy_async();
    cl_arrive_local(opnd_bar);
  };
  auto block_sum128 = [&](float v) -> float {
    v = warp_sum(v);
    if (lane == 0) red[warp] = v;
    cl_bar_compute();
    v = red[0] + red[1] + red[2] + red[3];
    cl_bar_compute();
    return v;
  };
  // RMSNorm of an owned residual row, rounded to bf16 and written into every CTA's operand buffer
  auto norm_allgather = [&](int own, int tl, const float *gain) {
    const float *xr = xrow + (size_t)own * d;
    float ss = 0.f;
    for (int f = tid * 4; f < d; f += 512) {
      const float4 v = *reinterpret_cast<const float4 *>(xr + f);
      ss = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, fmaf(v.w, v.w, ss))));
    }
    const float rstd = rsqrtf(block_sum128(ss) / d + a.eps);
    for (int f = tid * 4; f < d; f += 512) {
      const float4 v = *reinterpret_cast<const float4 *>(xr + f);
      const float4 gg = *reinterpret_cast<const float4 *>(gain + f);
      const uint32_t u0 = pack_bf16x2(gg.x * v.x * rstd, gg.y * v.y * rstd);
      const uint32_t u1 = pack_bf16x2(gg.z * v.z * rstd, gg.w * v.w * rstd);
      const uint32_t off = cl_opnd_off(tl, f, BN);
#pragma unroll
      for (int rr = 0; rr < CL_MAX_R; ++rr)
        if (rr < R) cl_st_remote_v2(rem_abuf[rr] + off, u0, u1);
    }
  };
  // residual rows owned by this CTA += sum of the R partial tiles; then norm + all-gather
  auto reduce_rows = [&](const float *gain) {
    int own = 0;
    for (int tl = r; tl < Mc; tl += R, ++own) {
      float *xr = xrow + (size_t)own * d;
      for (int f = tid * 4; f < d; f += 512) {
        float4 v[CL_MAX_R];
#pragma unroll
        for (int rr = 0; rr < CL_MAX_R; ++rr)
          if (rr < R) v[rr] = cl_ld_remote_f4(rem_part[rr] + (uint32_t)(tl * d + f) * 4);
        float4 x = *reinterpret_cast<float4 *>(xr + f);
#pragma unroll
        for (int rr = 0; rr < CL_MAX_R; ++rr)
          if (rr < R) { x.x += v[rr].x; x.y += v[rr].y; x.z += v[rr].z; x.w += v[rr].w; }
        *reinterpret_cast<float4 *>(xr + f) = x;
      }
      norm_allgather(own, tl, gain);
    }
  };
  // accumulator tiles (features x tokens) of a K-split contraction -> part[token][feature]
  auto dump_partial = [&](int n_tiles, int row_stride) {
    for (int j = 0; j < n_tiles; ++j)
      for (int c0 = 0; c0 < BN && c0 < Mc; c0 += 16) {
        float v[16];
        tmem_ld16(tbase + j * BN + c0, v);
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) part[(size_t)(c0 + jj) * row_stride + 128 * j + tid] = v[jj];
      }
    tc_fence_before();
  };

  // ---------------- embedding of the owned tokens, first norm
  {
    int own = 0;
    for (int tl = r; tl < Mc; tl += R, ++own) {
      const int b = b0 + tl / q_len, j = tl % q_len;
      const float *z = a.hist_in + ((size_t)b * cap + pos0_of(a.g, b) + j) * P;
      for (int i = tid; i < P; i += 128) zs[i] = z[i];
      cl_bar_compute();
      for (int f = tid * 4; f < d; f += 512) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const bf16 *wr = md.W_emb + (size_t)(f + i) * P;
          float acc = 0.f;
          for (int c = 0; c < P; c += 8) {
            float w[8];
            Vec16<bf16>::load(wr + c, w);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(w[e], zs[c + e], acc);
          }
          xrow[(size_t)own * d + f + i] = acc;
        }
      }
      cl_bar_compute();
      norm_allgather(own, tl, a.layers[0].g1);
    }
  }
  if (!csync()) { fail(); return; }
  operand_ready();

  for (int l = 0; l < L; ++l) {
    const ClLayer &ly = a.layers[l];
    // ---------------- q, k, v of head r: TMEM (features x tokens) -> qkv[token][q | k | v]
    if (!wait_acc()) { fail(); return; }
    for (int c0 = 0; c0 < BN && c0 < Mc; c0 += 16) {
      float v[16];
      tmem_ld16(tbase + c0, v);
#pragma unroll
      for (int jj = 0; jj < 16; ++jj) qkv[(c0 + jj) * 192 + tid] = v[jj];
      if (warp < 2) {
        tmem_ld16(tbase + BN + c0, v);
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) qkv[(c0 + jj) * 192 + 128 + tid] = v[jj];
      }
    }
    tc_fence_before();
    cl_bar_compute();
    // ---------------- RoPE on q and k; k and v rounded to the cache type and appended to the cache
    for (int tl = warp; tl < Mc; tl += 4) {
      const int b = b0 + tl / q_len, pos = pos0_of(a.g, b) + tl % q_len;
      float *row = qkv + tl * 192;
      const float2 cs = md.rope[(size_t)pos * 32 + lane];
      const float q1 = row[lane], q2 = row[32 + lane], k1 = row[64 + lane], k2 = row[96 + lane];
      row[lane] = (q1 * cs.x - q2 * cs.y) * 0.125f;
      row[32 + lane] = (q2 * cs.x + q1 * cs.y) * 0.125f;
      const bf16 kr1 = __float2bfloat16_rn(k1 * cs.x - k2 * cs.y), kr2 = __float2bfloat16_rn(k2 * cs.x + k1 * cs.y);
      const bf16 v1 = __float2bfloat16_rn(row[128 + lane]), v2 = __float2bfloat16_rn(row[160 + lane]);
      row[64 + lane] = __bfloat162float(kr1);
      row[96 + lane] = __bfloat162float(kr2);
      row[128 + lane] = __bfloat162float(v1);
      row[160 + lane] = __bfloat162float(v2);
      bf16 *kg = ly.Kc + (((size_t)b * R + r) * cap + pos) * 64, *vg = ly.Vc + (((size_t)b * R + r) * cap + pos) * 64;
      kg[lane] = kr1; kg[32 + lane] = kr2;
      vg[lane] = v1; vg[32 + lane] = v2;
    }
    cl_bar_compute();
    // ---------------- causal attention of head r, one warp per token
    for (int tl = warp; tl < Mc; tl += 4) {
      const int bl = tl / q_len, j = tl % q_len, b = b0 + bl;
      const int p0 = pos0_of(a.g, b), nv = p0 + j + 1;
      const float *q = qkv + tl * 192;
      const bf16 *Kb = ly.Kc + ((size_t)b * R + r) * cap * 64, *Vb = ly.Vc + ((size_t)b * R + r) * cap * 64;
      float *my_sc = sc + warp * capr;
      for (int t = lane; t < p0; t += 32)          // the value rows are walked one by one below: fetch them now
        asm volatile("prefetch.global.L1 [%0];" ::"l"(Vb + (size_t)t * 64));
      float mx = -INFINITY;
      for (int t = lane; t < nv; t += 32) {
        float s = 0.f;
        if (t < p0) {
          const uint4 *kr = reinterpret_cast<const uint4 *>(Kb + (size_t)t * 64);
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 kk = kr[c];
            const uint32_t w[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              s = fmaf(q[c * 8 + 2 * e], __uint_as_float(w[e] << 16), s);
              s = fmaf(q[c * 8 + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), s);
            }
          }
        } else {
          const float *kr = qkv + (bl * q_len + (t - p0)) * 192 + 64;
#pragma unroll 8
          for (int c = 0; c < 64; ++c) s = fmaf(q[c], kr[c], s);
        }
        my_sc[t] = s;
        mx = fmaxf(mx, s);
      }
      mx = warp_max(mx);
      float sum = 0.f;
      for (int t = lane; t < nv; t += 32) {
        const float p = expf(my_sc[t] - mx);
        my_sc[t] = p;
        sum += p;
      }
      sum = warp_sum(sum);
      __syncwarp();
      float o0 = 0.f, o1 = 0.f;
      const uint32_t *Vw = reinterpret_cast<const uint32_t *>(Vb);
#pragma unroll 4
      for (int t = 0; t < p0; ++t) {
        const float p = my_sc[t];
        const uint32_t vv = Vw[(size_t)t * 32 + lane];
        o0 = fmaf(p, __uint_as_float(vv << 16), o0);
        o1 = fmaf(p, __uint_as_float(vv & 0xffff0000u), o1);
      }
      for (int t = p0; t < nv; ++t) {
        const float p = my_sc[t];
        const float *vr = qkv + (bl * q_len + (t - p0)) * 192 + 128;
        o0 = fmaf(p, vr[2 * lane], o0);
        o1 = fmaf(p, vr[2 * lane + 1], o1);
      }
      const float inv = 1.f / sum;
      *reinterpret_cast<uint32_t *>(ao_buf + cl_opnd_off(tl, 2 * lane, BN)) = pack_bf16x2(o0 * inv, o1 * inv);
      __syncwarp();
    }
    operand_ready();
    // ---------------- attention output projection: K-split partials, residual, norm
    if (!wait_acc()) { fail(); return; }
    dump_partial(TD, d);
    if (!csync()) { fail(); return; }
    reduce_rows(ly.g2);
    if (!csync()) { fail(); return; }
    operand_ready();
    // ---------------- MLP up-projection of this CTA's hidden units + GELU -> operand of W_2
    if (!wait_acc()) { fail(); return; }
    for (int j = 0; j < TF; ++j)
      for (int c0 = 0; c0 < BN && c0 < Mc; c0 += 16) {
        float v[16];
        tmem_ld16(tbase + j * BN + c0, v);
#pragma unroll
        for (int jj = 0; jj < 16; ++jj)
          *reinterpret_cast<bf16 *>(h_buf + cl_opnd_off(c0 + jj, 128 * j + tid, BN)) = __float2bfloat16_rn(gelu_erf(v[jj]));
      }
    operand_ready();
    // ---------------- MLP down-projection: K-split partials, residual, next norm
    if (!wait_acc()) { fail(); return; }
    dump_partial(TD, d);
    if (!csync()) { fail(); return; }
    reduce_rows(l + 1 < L ? a.layers[l + 1].g1 : md.g_f);
    if (!csync()) { fail(); return; }
    operand_ready();
  }
  // ---------------- mean head (K-split over the CTAs), written by the token's owner
  if (!wait_acc()) { fail(); return; }
  dump_partial(1, 128);
  if (!csync()) { fail(); return; }
  for (int tl = r; tl < Mc; tl += R) {
    const int b = b0 + tl / q_len, j = tl % q_len;
    if (!a.head_all && j != q_len - 1) continue;
    if (tid < P) {
      float s = 0.f;
#pragma unroll
      for (int rr = 0; rr < CL_MAX_R; ++rr)
        if (rr < R) s += cl_ld_remote_f1(rem_part[rr] + (uint32_t)(tl * 128 + tid) * 4);
      if (a.head_all) a.vout[((size_t)b * q_len + j) * P + tid] = s;
      else a.hist_out[((size_t)b * cap + pos0_of(a.g, b) + q_len) * P + tid] = s;
    }
  }
}

// grid = (R, n_groups), cluster = (R, 1, 1), block = 192.
__global__ void __launch_bounds__(192, 1) pass_cluster_kernel(const ClArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const ClModel &md = *a.model;
  const int R = md.heads, d = md.d, ffr = md.ff / md.heads, L = md.n_layers, P = md.P;
  const int KBd = d / 64, KBf = ffr / 64, TD = d / 128, TF = ffr / 128;
  const int BN = a.BN, stages = a.stages;
  const int r = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;

  const uint32_t raw32 = smem_u32(smem_raw);
  const uint32_t base32 = (raw32 + 1023u) & ~1023u;
  uint8_t *sm = smem_raw + (base32 - raw32);
  const ClSmem so = cl_smem_layout(d, ffr, BN, R, stages, a.g.cap, P);
  const uint32_t ring32 = base32 + so.ring, abuf32 = base32 + so.a_buf, aobuf32 = base32 + so.ao_buf,
                 hbuf32 = base32 + so.h_buf;
  const uint32_t bars = base32 + so.bars;
  const uint32_t full0 = bars, empty0 = bars + 128, acc_bar = bars + 256, opnd_bar = bars + 264, cbar = bars + 272;
  uint32_t *slot_ptr = reinterpret_cast<uint32_t *>(sm + so.bars + 288);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + so.bars + 292);

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(acc_bar, 1);
    mbar_init(opnd_bar, 128);
    mbar_init(cbar, (uint32_t)R);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + 288), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  // peers must not signal this CTA's cluster barrier before it is initialised
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  tc_fence_after();
  const uint32_t tmem = *slot_ptr;

  if (warp == 4) {
    // =============================================================== TMA producer
    // Streams this CTA's weight tiles of the whole pass in a fixed order, as far ahead as the
    // ring allows.  Weights do not depend on the preceding kernel: no dependency wait here.
    if (lane == 0) {
      pdl_release();
      int it = 0;
      bool ok = true;
      auto acquire = [&](uint32_t bytes) -> uint32_t {
        const int s = it % stages;
        if (it >= stages && !cl_wait(empty0 + 8 * s, (uint32_t)((it / stages) - 1) & 1u, abort_flag, false)) {
          ok = false;
          return 0;
        }
        mbar_expect_tx(full0 + 8 * s, bytes);
        ++it;
        return (uint32_t)s;
      };
      for (int l = 0; l < L && ok; ++l) {
        const ClLayer &ly = a.layers[l];
        for (int kb = 0; kb < KBd && ok; ++kb) {       // [q_r; k_r] then [v_r; -]
          uint32_t s = acquire(CL_TILE_BYTES);
          if (!ok) break;
          tma_load_2d(ring32 + s * CL_TILE_BYTES, &ly.qkv, kb * 64, r * 64, full0 + 8 * s);
          tma_load_2d(ring32 + s * CL_TILE_BYTES + 8192, &ly.qkv, kb * 64, d + r * 64, full0 + 8 * s);
          s = acquire(8192);
          if (!ok) break;
          tma_load_2d(ring32 + s * CL_TILE_BYTES, &ly.qkv, kb * 64, 2 * d + r * 64, full0 + 8 * s);
        }
        for (int j = 0; j < TD && ok; ++j) {           // W_o[:, head r]
          const uint32_t s = acquire(CL_TILE_BYTES);
          if (!ok) break;
          tma_load_2d(ring32 + s * CL_TILE_BYTES, &ly.wo, r * 64, j * 128, full0 + 8 * s);
        }
        for (int j = 0; j < TF && ok; ++j)             // W_1 rows of this CTA's hidden units
          for (int kb = 0; kb < KBd && ok; ++kb) {
            const uint32_t s = acquire(CL_TILE_BYTES);
            if (!ok) break;
            tma_load_2d(ring32 + s * CL_TILE_BYTES, &ly.w1, kb * 64, r * ffr + j * 128, full0 + 8 * s);
          }
        for (int j = 0; j < TD && ok; ++j)             // W_2 columns of the same hidden units
          for (int kb = 0; kb < KBf && ok; ++kb) {
            const uint32_t s = acquire(CL_TILE_BYTES);
            if (!ok) break;
            tma_load_2d(ring32 + s * CL_TILE_BYTES, &ly.w2, r * ffr + kb * 64, j * 128, full0 + 8 * s);
          }
      }
      if (ok) {                                        // mean head, K slice r
        const uint32_t s = acquire(CL_TILE_BYTES);
        if (ok) tma_load_2d(ring32 + s * CL_TILE_BYTES, &md.head, r * 64, 0, full0 + 8 * s);
      }
      if (!ok) { atomicExch(a.status, DEV_TIMEOUT_TMA); *abort_flag = 1; }
    }
  } else if (warp == 5) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      pdl_release();
      const uint32_t idesc = umma_idesc_rt(BN);
      int it = 0, gi = 0;
      bool ok = true;
      // one weight tile (128 rows x 64 k) times one 64-wide block of an operand buffer
      auto mma_tile = [&](uint32_t opnd32, int col, bool first) {
        const int s = it % stages;
        if (!cl_wait(full0 + 8 * s, (uint32_t)(it / stages) & 1u, abort_flag, false)) { ok = false; return; }
        tc_fence_after();
        const uint64_t dw = umma_smem_desc(ring32 + s * CL_TILE_BYTES), db = umma_smem_desc(opnd32);
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16(tmem + col, dw + 2 * k, db + 2 * k, idesc, (first && k == 0) ? 0u : 1u);
        umma_commit(empty0 + 8 * s);
        ++it;
      };
      auto begin_gemm = [&]() {
        if (!cl_wait(opnd_bar, (uint32_t)gi & 1u, abort_flag, false)) { ok = false; return; }
        tc_fence_after();
      };
      auto end_gemm = [&]() { umma_commit(acc_bar); ++gi; };
      for (int l = 0; l < L && ok; ++l) {
        begin_gemm();
        for (int kb = 0; kb < KBd && ok; ++kb) {
          mma_tile(abuf32 + kb * BN * 128, 0, kb == 0);
          if (ok) mma_tile(abuf32 + kb * BN * 128, BN, kb == 0);
        }
        if (!ok) break;
        end_gemm();
        begin_gemm();
        for (int j = 0; j < TD && ok; ++j) mma_tile(aobuf32, j * BN, true);
        if (!ok) break;
        end_gemm();
        begin_gemm();
        for (int j = 0; j < TF && ok; ++j)
          for (int kb = 0; kb < KBd && ok; ++kb) mma_tile(abuf32 + kb * BN * 128, j * BN, kb == 0);
        if (!ok) break;
        end_gemm();
        begin_gemm();
        for (int j = 0; j < TD && ok; ++j)
          for (int kb = 0; kb < KBf && ok; ++kb) mma_tile(hbuf32 + kb * BN * 128, j * BN, kb == 0);
        if (!ok) break;
        end_gemm();
      }
      if (ok) {
        begin_gemm();
        if (ok) mma_tile(abuf32 + r * BN * 128, 0, true);
        if (ok) end_gemm();
      }
      if (!ok) { atomicExch(a.status, DEV_TIMEOUT_MMA); *abort_flag = 1; }
    }
  } else {
    // =============================================================== compute warps
    cl_compute(a, sm, so, base32, tmem, acc_bar, opnd_bar, cbar, abort_flag);
  }
  // common exit: nobody leaves while a peer may still touch this CTA's shared memory
  __syncwarp();
  tc_fence_before();
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
  }
}

// ------------------------------------------------------------------ host side
struct ClPlan {
  bool valid = false;
  int R = 0, d = 0, ff = 0, P = 0, L = 0;
  ClModel *model = nullptr;       // device
  ClLayer *layers = nullptr;      // device
};

static bool cl_model_ok(int n_heads, int d, int ff, int P) {
  return n_heads >= 1 && n_heads <= CL_MAX_R && d == 64 * n_heads && d % 128 == 0 && ff % n_heads == 0 &&
         (ff / n_heads) % 128 == 0 && P <= 128 && P % 16 == 0;
}

// Series per cluster, padded token count and ring depth for a pass of q_len tokens per series
// over B series; false if the pass does not fit this kernel.
static bool cl_geometry(const ClPlan &p, int B, int q_len, int cap, int *Bg, int *BN, int *G, int *stages, int *smem) {
  if (!p.valid || B < 1 || q_len < 1) return false;
  const int gmax = 148 / p.R;
  const int bg = (B + gmax - 1) / gmax;
  const int tokens = bg * q_len;
  if (tokens > CL_MAX_BN) return false;
  const int bn = tokens <= 16 ? 16 : 32;
  int st = 12;
  for (; st >= 3; --st)
    if (cl_smem_layout(p.d, p.ff / p.R, bn, p.R, st, cap, p.P).total <= 227 * 1024) break;
  if (st < 3) return false;
  *Bg = bg; *BN = bn; *G = (B + bg - 1) / bg; *stages = st;
  *smem = cl_smem_layout(p.d, p.ff / p.R, bn, p.R, st, cap, p.P).total;
  return true;
}

static int cl_init() {
  if (int rc = gemm_tc_init()) return rc;
  static bool done = false;
  if (done) return 0;
  if (cudaFuncSetAttribute(pass_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
    return -4;
  cudaFuncSetAttribute(pass_cluster_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  done = true;
  return 0;
}

static bool cl_launch(cudaStream_t st, bool pdl, const ClPlan &p, const ClArgs &args, int G, int smem) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.R, G, 1);
  cfg.blockDim = dim3(192);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = p.R; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, pass_cluster_kernel, args) == cudaSuccess;
}

}  // namespace tsfm

// Fused dequantize + GQA decode attention over the packed mixed-precision cache (Eq. 9 + softmax
// attention), split over the sequence (flash-decoding) with a separate combine kernel.
//
// Per (batch, kv_head) slice the grid has one "aux" CTA for the INT16 tokens (sink + window ring)
// and `body_splits` CTAs that share the body tiles.  A warp owns whole 16-token tiles and keeps its
// own running (max, sum, accumulator); warps are merged in shared memory.  Body tiles are staged
// through a per-warp cp.async ring in shared memory (a tile is one contiguous run of bytes), so a
// warp has several tiles in flight while it works on one.  The CTA that finishes last for a slice
// (atomic ticket, no waiting) merges the slice's split partials and writes the output.
//
// The contraction runs on the tensor cores with mma.sync.m16n8k16 (f16 inputs, f32 accumulate) and
// register operands: packed codes go from 128-bit global loads to MMA fragments with one AND (and
// a shared shift) per pair of codes - a code field left in place inside an fp16 bit pattern below
// bit 11 is the exact value code * 2^(pos-24) (fp16 subnormals and the first binade are linear).
//   scores:  S[h, t]  = sum_i Q''[h, i] * c_K[t, i]      A = Q'' (rows 0-7: fp16 "hi" part of the 8 heads,
//                                                        rows 8-15: the "lo" remainder), B = K codes
//   output:  O^T[i,h] = sum_t c_V[t, i] * w[t, h]        A = V codes, B = w = p * S_V (one fp16)
// The per-token scale and zero-point never touch the codes: q.k = S_K (q.c) + Z_K sum(q) and
// sum_t p_t v_t = sum_t (p_t S_V,t) c_t + sum_t p_t Z_V,t.  The probability actually used for a token is
// the fp16-rounded w divided by its scale, in numerator and denominator alike, so the fp16 rounding
// of w is a consistent (softmax-invariant to first order) perturbation.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "kernels_cache.cuh"
#include "layout.cuh"

namespace pmkvq {

constexpr int kMaxGroup = 8;        // query heads per KV head handled by one MMA row block
constexpr int kPartialStride = 132; // floats per (cta, head): m, l, 2 pad, o[128]
constexpr float kNegBig = -1.0e30f;

struct AttnParams {
  LayerGeom geom;
  const uint16_t *Q;          // bf16 [batch][q_heads][128]
  const float *lambda;        // [kv_heads][128] of this block
  const unsigned *vmax_bits;  // [n_slices] running max of the INT16 V scales (fp32 bit patterns)
  float *partials;            // [n_slices][1 + body_splits][8][kPartialStride]
  float *out;                 // fp32 [batch][q_heads][128]
  unsigned *tickets;          // [n_slices], zero between launches: CTAs of a slice that have finished
  int kv_heads, group, q_heads;
  int n_tokens, n_sink_eff, win_start, cur_bits;
  int n_body, body_tiles, body_splits, tiles_per_split;
  float qk_scale;  // sm_scale * log2(e)
};

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void *gptr) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ uint32_t mul_half2(uint32_t a, float f) {
  const __half2 r = __hmul2(*reinterpret_cast<const __half2 *>(&a), __float2half2_rn(f));
  return *reinterpret_cast<const uint32_t *>(&r);
}

// Bit position of code j of a half-word after extraction, per width (see extract<>), and the fp16
// exponent budget: A/B operands built from Q or w are scaled by 2^(E - pos) so that they stay
// below 2^15 while products keep at least 20 significant bits inside the MMA's alignment window.
template <int BITS> struct Fmt;
template <> struct Fmt<2> {
  static constexpr int N = 8, E = 14, SIGMA_LOG2 = 15, STAGES = 4;
  __device__ static constexpr int pos(int j) { return j < 3 ? 5 + 2 * j : (j < 5 ? 2 * j : 2 * j - 5); }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[8]) {
    const uint32_t xl = x << 5, xr = x >> 5;
    e[0] = xl & 0x00600060u; e[1] = xl & 0x01800180u; e[2] = xl & 0x06000600u;
    e[3] = x & 0x00C000C0u;  e[4] = x & 0x03000300u;
    e[5] = xr & 0x00600060u; e[6] = xr & 0x01800180u; e[7] = xr & 0x06000600u;
  }
};
template <> struct Fmt<4> {
  static constexpr int N = 4, E = 14, SIGMA_LOG2 = 13, STAGES = 4;
  __device__ static constexpr int pos(int j) { return (j & 1) ? 7 : 3; }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[4]) {
    const uint32_t xl = x << 3, xr = x >> 5;
    e[0] = xl & 0x00780078u; e[1] = xl & 0x07800780u;
    e[2] = xr & 0x00780078u; e[3] = xr & 0x07800780u;
  }
};
template <> struct Fmt<8> {
  static constexpr int N = 2, E = 14, SIGMA_LOG2 = 9, STAGES = 3;
  __device__ static constexpr int pos(int) { return 0; }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[2]) {
    e[0] = x & 0x00FF00FFu;
    e[1] = (x >> 8) & 0x00FF00FFu;
  }
};
// 16 bit: a code is split into its low byte (pos 0, weight 1) and its high byte moved to pos 3
// (weight 256); the operand that multiplies the high bytes is the low one times 2^5.
template <> struct Fmt<16> {
  static constexpr int N = 1, E = 9, SIGMA_LOG2 = 0, STAGES = 0;  // 16-bit tiles are read straight from global memory
  __device__ static constexpr int pos(int) { return 0; }
};

struct WarpState {
  float m, l, zs;      // running max (log2 units), sum of probabilities, sum of p * Z_V, for head g (this lane's quad)
  float acc[8][4];     // O^T accumulators: [m-tile][channel row g / g+8 x head col 2tig / 2tig+1]
};

// One 16-token tile.  `mask` has bit r set when token row r of the tile is a live token.
template <int BITS, bool MASKED>
__device__ __forceinline__ void process_tile(const uint8_t *tile, uint32_t mask, WarpState &st,
                                             const uint32_t (&qa)[8][4], float mu, float sumq, float sigma_u,
                                             float inv_sigma_e, int lane) {
  using F = Fmt<BITS>;
  constexpr int CHUNKS = BITS / 2;
  const int tig = lane & 3;
  uint32_t kw[2 * BITS], vw[2 * BITS];
  {
    const uint8_t *kp = tile + lane * 16;
    const uint8_t *vp = tile + v_part_offset(BITS) + lane * 16;
#pragma unroll
    for (int q = 0; q < CHUNKS; ++q) {
      const uint4 a = *reinterpret_cast<const uint4 *>(kp + q * 512);
      kw[4 * q] = a.x; kw[4 * q + 1] = a.y; kw[4 * q + 2] = a.z; kw[4 * q + 3] = a.w;
    }
#pragma unroll
    for (int q = 0; q < CHUNKS; ++q) {
      const uint4 a = *reinterpret_cast<const uint4 *>(vp + q * 512);
      vw[4 * q] = a.x; vw[4 * q + 1] = a.y; vw[4 * q + 2] = a.z; vw[4 * q + 3] = a.w;
    }
  }
  const float4 *mp = reinterpret_cast<const float4 *>(tile + meta_offset(BITS) + tig * 64);
  const float4 sk4 = mp[0], zk4 = mp[1], sv4 = mp[2], zv4 = mp[3];
  float sk[4] = {sk4.x, sk4.y, sk4.z, sk4.w}, zk[4] = {zk4.x, zk4.y, zk4.z, zk4.w};
  float sv[4] = {sv4.x, sv4.y, sv4.z, sv4.w}, zv[4] = {zv4.x, zv4.y, zv4.z, zv4.w};

  // ---- scores: S = Q'' K^T, heads on M (hi rows 0-7, lo rows 8-15), tokens on N ----
  float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  if constexpr (BITS == 16) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const uint32_t x0 = kw[r * 16 + 2 * s], x1 = kw[r * 16 + 2 * s + 1];
        mma_f16(sacc[r], qa[s], x0 & 0x00FF00FFu, x1 & 0x00FF00FFu);
        mma_f16(sacc[r], mul_half2(qa[s][0], 32.f), mul_half2(qa[s][1], 32.f), mul_half2(qa[s][2], 32.f),
                mul_half2(qa[s][3], 32.f), (x0 >> 5) & 0x07F807F8u, (x1 >> 5) & 0x07F807F8u);
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
#pragma unroll
      for (int w = 0; w < BITS; ++w) {
        uint32_t e[F::N];
        F::extract(kw[r * BITS + w], e);
#pragma unroll
        for (int jj = 0; jj < F::N / 2; ++jj) mma_f16(sacc[r], qa[(w * F::N) / 2 + jj], e[2 * jj], e[2 * jj + 1]);
      }
    }
  }

  // ---- online softmax for head g over this lane's 4 tokens {2tig, 2tig+1, 8+2tig, 9+2tig} ----
  float sc[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = i >> 1, e = i & 1;
    const float dot = sacc[r][e] + sacc[r][2 + e];
    sc[i] = fmaf(sk[i] * mu, dot, zk[i] * sumq);
    if constexpr (MASKED) {
      const bool live = (mask >> (8 * r + 2 * tig + e)) & 1u;
      if (!live) {
        sc[i] = -INFINITY;
        sv[i] = 0.f;
        zv[i] = 0.f;
      }
    }
  }
  float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
  const float m_new = fmaxf(st.m, mx);
  if (__any_sync(0xffffffffu, m_new > st.m)) {
    const float f = ex2(st.m - m_new);
    st.l *= f;
    st.zs *= f;
    const float f0 = __shfl_sync(0xffffffffu, f, (2 * tig) * 4);
    const float f1 = __shfl_sync(0xffffffffu, f, (2 * tig + 1) * 4);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      st.acc[mt][0] *= f0; st.acc[mt][1] *= f1; st.acc[mt][2] *= f0; st.acc[mt][3] *= f1;
    }
    st.m = m_new;
  }
  float wv[4], rs[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float s_e = (sv[i] == 0.f ? sigma_u : sv[i]) * inv_sigma_e;  // S_V / sigma_u * 2^E  (<= 2^E)
    rs[i] = rcp_approx(s_e);
    wv[i] = ex2(sc[i] - st.m) * s_e;
  }
  const uint32_t pb0 = pack_half2(wv[0], wv[1]);
  const uint32_t pb1 = pack_half2(wv[2], wv[3]);
  {
    const float2 w01 = __half22float2(*reinterpret_cast<const __half2 *>(&pb0));
    const float2 w23 = __half22float2(*reinterpret_cast<const __half2 *>(&pb1));
    const float p0 = w01.x * rs[0], p1 = w01.y * rs[1], p2 = w23.x * rs[2], p3 = w23.y * rs[3];
    st.l += (p0 + p1) + (p2 + p3);
    st.zs += fmaf(p0, zv[0], fmaf(p1, zv[1], fmaf(p2, zv[2], p3 * zv[3])));
  }

  // ---- output: O^T += V^T w, channels on M, tokens on K, heads on N ----
  if constexpr (BITS == 16) {
    const uint32_t ph0 = mul_half2(pb0, 32.f), ph1 = mul_half2(pb1, 32.f);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const uint32_t a0 = vw[2 * mt], a1 = vw[2 * mt + 1], a2 = vw[16 + 2 * mt], a3 = vw[16 + 2 * mt + 1];
      mma_f16(st.acc[mt], a0 & 0x00FF00FFu, a1 & 0x00FF00FFu, a2 & 0x00FF00FFu, a3 & 0x00FF00FFu, pb0, pb1);
      mma_f16(st.acc[mt], (a0 >> 5) & 0x07F807F8u, (a1 >> 5) & 0x07F807F8u, (a2 >> 5) & 0x07F807F8u,
              (a3 >> 5) & 0x07F807F8u, ph0, ph1);
    }
  } else {
#pragma unroll
    for (int w = 0; w < BITS; ++w) {
      uint32_t ea[F::N], eb[F::N];
      F::extract(vw[w], ea);
      F::extract(vw[BITS + w], eb);
#pragma unroll
      for (int jj = 0; jj < F::N / 2; ++jj)
        mma_f16(st.acc[(w * F::N) / 2 + jj], ea[2 * jj], ea[2 * jj + 1], eb[2 * jj], eb[2 * jj + 1], pb0, pb1);
    }
  }
}

// Log-sum-exp merge of the split partials of one slice (all its CTAs have published theirs);
// 128 threads = 128 channels.
__device__ __forceinline__ void combine_slice(const AttnParams &p, int slice, float *s_w) {
  const int tid = threadIdx.x;
  const int b = slice / p.kv_heads, hkv = slice % p.kv_heads;
  const int n_ctas = 1 + p.body_splits;
  const float *part = p.partials + (size_t)slice * n_ctas * kMaxGroup * kPartialStride;
  for (int h = 0; h < p.group; ++h) {
    // weights 2^(m_c - M) of the CTAs, computed once by the first warps and shared
    float M = kNegBig;
    for (int c = 0; c < n_ctas; ++c) M = fmaxf(M, __ldcg(part + ((size_t)c * kMaxGroup + h) * kPartialStride));
    __syncthreads();
    for (int c = tid; c < n_ctas; c += 128) s_w[c] = ex2(__ldcg(part + ((size_t)c * kMaxGroup + h) * kPartialStride) - M);
    __syncthreads();
    float num = 0.f, den = 0.f;
#pragma unroll 4
    for (int c = 0; c < n_ctas; ++c) {
      const float *pc = part + ((size_t)c * kMaxGroup + h) * kPartialStride;
      den = fmaf(s_w[c], __ldcg(pc + 1), den);
      num = fmaf(s_w[c], __ldcg(pc + 4 + tid), num);
    }
    p.out[((size_t)b * p.q_heads + hkv * p.group + h) * kHeadDim + tid] = num / den;
  }
}

// Everything one CTA does at width BITS: build the query fragments, run its tiles, merge its warps
// and write one partial (m, l, o[128]) per head.  `ring` is the CTA's dynamic shared memory: the
// per-warp cp.async stages while tiles stream, then the warps' outputs.
template <int BITS>
__device__ __forceinline__ void run_cta(const AttnParams &p, float (*s_q)[kHeadDim], float *s_stat, uint8_t *ring) {
  using F = Fmt<BITS>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tig = lane & 3;
  const int slice = blockIdx.y;
  const int b = slice / p.kv_heads, hkv = slice % p.kv_heads;
  const bool aux = (blockIdx.x == 0);

  // ---- Q'' = Q * lambda * sm_scale * log2(e)  (Eq. 9: the equalization scale migrates into Q) ----
  {
    const float lam = p.lambda[hkv * kHeadDim + tid];
    for (int h = 0; h < kMaxGroup; ++h) {
      float v = 0.f;
      if (h < p.group) {
        const uint16_t raw = p.Q[((size_t)b * p.q_heads + hkv * p.group + h) * kHeadDim + tid];
        v = __fmul_rn(__fmul_rn(__uint_as_float((uint32_t)raw << 16), lam), p.qk_scale);
      }
      s_q[h][tid] = v;
    }
  }
  __syncthreads();
  for (int h = warp; h < kMaxGroup; h += 4) {  // per-head max |q''| and sum q''
    const float4 v = *reinterpret_cast<const float4 *>(&s_q[h][lane * 4]);
    float mx = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
    float sm = (v.x + v.y) + (v.z + v.w);
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      sm += __shfl_xor_sync(0xffffffffu, sm, o);
    }
    if (lane == 0) {
      int e = 0;
      if (mx > 0.f) frexpf(mx, &e);  // mx = f * 2^e, f in [0.5, 1)
      s_stat[h] = (float)e;
      s_stat[8 + h] = sm;
    }
  }
  __syncthreads();
  const int e_g = (int)s_stat[g];
  const float sumq = s_stat[8 + g];
  const float mu = ldexpf(1.0f, 24 - F::E + e_g);

  uint32_t qa[8][4];
#pragma unroll
  for (int s = 0; s < 8; ++s) {
#pragma unroll
    for (int beta = 0; beta < 2; ++beta) {
      const int W = 2 * s + beta;
      const float scl = ldexpf(1.0f, F::E - F::pos(W % F::N) - e_g);
      const int c0 = 16 * s + 8 * beta + 2 * tig;
      const float x0 = s_q[g][c0] * scl, x1 = s_q[g][c0 + 1] * scl;
      const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
      const __half l0 = __float2half_rn(x0 - __half2float(h0)), l1 = __float2half_rn(x1 - __half2float(h1));
      const __half2 hi = __halves2half2(h0, h1), lo = __halves2half2(l0, l1);
      qa[s][2 * beta] = *reinterpret_cast<const uint32_t *>(&hi);
      qa[s][2 * beta + 1] = *reinterpret_cast<const uint32_t *>(&lo);
    }
  }

  // ---- unit of the V accumulators: a power of two >= every V scale of this slice at this width ----
  float sigma_u = 1.0f;
  {
    const float s16 = __uint_as_float(p.vmax_bits[slice]);
    if (s16 > 0.f) {
      int e;
      frexpf(s16, &e);
      sigma_u = ldexpf(1.0f, e + F::SIGMA_LOG2);
    }
  }
  const float inv_sigma_e = ldexpf(1.0f, F::E) / sigma_u;

  WarpState st;
  st.m = kNegBig; st.l = 0.f; st.zs = 0.f;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) st.acc[mt][0] = st.acc[mt][1] = st.acc[mt][2] = st.acc[mt][3] = 0.f;

  const uint8_t *slice_base = p.geom.base + (size_t)slice * p.geom.slice_stride;
  if (aux) {
    if constexpr (BITS == 16) {
      const int sink_tiles = (p.n_sink_eff + 15) >> 4;
      const int ring_tiles = p.geom.ring_tokens >> 4;
      const int n_win = p.n_tokens - p.win_start;
      const int first_slot = (p.win_start - p.geom.n_sink) % p.geom.ring_tokens;  // win_start >= n_sink when n_win > 0
      for (int it = warp; it < sink_tiles + ring_tiles; it += 4) {
        uint32_t mask = 0;
        const uint8_t *tile;
        if (it < sink_tiles) {
          const int live = min(16, p.n_sink_eff - 16 * it);
          mask = (1u << live) - 1u;
          tile = slice_base + (size_t)it * tile_bytes(16);
        } else {
          const int rt = it - sink_tiles;
          tile = slice_base + p.geom.ring_off + (size_t)rt * tile_bytes(16);
          if (n_win > 0) {
            for (int r = 0; r < 16; ++r) {
              int d = rt * 16 + r - first_slot;
              if (d < 0) d += p.geom.ring_tokens;
              if (d < n_win) mask |= 1u << r;
            }
          }
        }
        if (mask == 0xFFFFu) process_tile<16, false>(tile, mask, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
        else if (mask) process_tile<16, true>(tile, mask, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
      }
    }
  } else {
    const int split = blockIdx.x - 1;
    const int t0 = split * p.tiles_per_split;
    const int t1 = min(p.body_tiles, t0 + p.tiles_per_split);
    const uint8_t *body = slice_base + p.geom.body_off;
    const uint32_t tail_mask = (p.n_body & 15) ? (1u << (p.n_body & 15)) - 1u : 0xFFFFu;
    if constexpr (F::STAGES == 0) {
      for (int t = t0 + warp; t < t1; t += 4) {
        const uint8_t *tile = body + (size_t)t * tile_bytes(BITS);
        if (t == p.body_tiles - 1 && tail_mask != 0xFFFFu)
          process_tile<BITS, true>(tile, tail_mask, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
        else
          process_tile<BITS, false>(tile, 0xFFFFu, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
      }
    } else {
      // per-warp ring of STAGES tiles; tile i of this warp is body tile t0 + warp + 4 i
      constexpr int TB = tile_bytes(BITS);
      constexpr int S = F::STAGES;
      uint8_t *my_ring = ring + (size_t)warp * S * TB;
      const uint32_t ring_addr = (uint32_t)__cvta_generic_to_shared(my_ring);
      const int n_my = (t1 - t0 - warp + 3) >> 2;
      const uint8_t *src0 = body + (size_t)(t0 + warp) * TB + lane * 16;
      auto issue = [&](int i, int stage) {
        const uint8_t *src = src0 + (size_t)i * 4 * TB;
        const uint32_t dst = ring_addr + stage * TB + lane * 16;
#pragma unroll
        for (int c = 0; c < (TB / 16 + 31) / 32; ++c)
          if (c * 32 + lane < TB / 16) cp_async16(dst + c * 512, src + c * 512);
      };
#pragma unroll
      for (int i = 0; i < S - 1; ++i) {
        if (i < n_my) issue(i, i);
        cp_async_commit();
      }
      int stage = 0, fill = S - 1;
      for (int i = 0; i < n_my; ++i) {
        if (i + S - 1 < n_my) issue(i + S - 1, fill);
        cp_async_commit();
        cp_async_wait<S - 1>();
        __syncwarp();
        const uint8_t *tile = my_ring + stage * TB;
        if (t0 + warp + 4 * i == p.body_tiles - 1 && tail_mask != 0xFFFFu)
          process_tile<BITS, true>(tile, tail_mask, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
        else
          process_tile<BITS, false>(tile, 0xFFFFu, st, qa, mu, sumq, sigma_u, inv_sigma_e, lane);
        __syncwarp();
        fill = stage;
        stage = (stage + 1 == S) ? 0 : stage + 1;
      }
    }
  }

  // ---- warp epilogue: quad sums, real units, to shared memory (the ring is free now) ----
  st.l += __shfl_xor_sync(0xffffffffu, st.l, 1);
  st.l += __shfl_xor_sync(0xffffffffu, st.l, 2);
  st.zs += __shfl_xor_sync(0xffffffffu, st.zs, 1);
  st.zs += __shfl_xor_sync(0xffffffffu, st.zs, 2);
  __syncthreads();  // every warp is done with its stages; s_stat is reused below
  float(*s_o)[kMaxGroup][kHeadDim] = reinterpret_cast<float(*)[kMaxGroup][kHeadDim]>(ring);
  if (tig == 0) {
    s_stat[16 + warp * 8 + g] = st.m;
    s_stat[48 + warp * 8 + g] = st.l;
  }
  const float zs0 = __shfl_sync(0xffffffffu, st.zs, (2 * tig) * 4);
  const float zs1 = __shfl_sync(0xffffffffu, st.zs, (2 * tig + 1) * 4);
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int J = 2 * mt + rr;
      const float f = ldexpf(sigma_u, 24 - F::E - F::pos(J % F::N));
      const int ch = 16 * mt + 8 * rr + g;
      s_o[warp][2 * tig][ch] = fmaf(st.acc[mt][2 * rr], f, zs0);
      s_o[warp][2 * tig + 1][ch] = fmaf(st.acc[mt][2 * rr + 1], f, zs1);
    }
  }
  __syncthreads();

  // ---- merge the 4 warps, publish the CTA's partial ----
  float *part = p.partials + ((size_t)slice * (1 + p.body_splits) + blockIdx.x) * kMaxGroup * kPartialStride;
  for (int h = 0; h < p.group; ++h) {
    const float m0 = s_stat[16 + h], m1 = s_stat[24 + h], m2 = s_stat[32 + h], m3 = s_stat[40 + h];
    const float M = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
    const float w0 = ex2(m0 - M), w1 = ex2(m1 - M), w2 = ex2(m2 - M), w3 = ex2(m3 - M);
    const float o = w0 * s_o[0][h][tid] + w1 * s_o[1][h][tid] + w2 * s_o[2][h][tid] + w3 * s_o[3][h][tid];
    __stcg(part + h * kPartialStride + 4 + tid, o);
    if (tid == 0) {
      __stcg(part + h * kPartialStride, M);
      __stcg(part + h * kPartialStride + 1,
             w0 * s_stat[48 + h] + w1 * s_stat[56 + h] + w2 * s_stat[64 + h] + w3 * s_stat[72 + h]);
    }
  }

  // ---- the last CTA of the slice to get here merges the slice (ticket, nobody waits) ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned t = atomicAdd(p.tickets + slice, 1u);
    s_stat[79] = (t == (unsigned)p.body_splits) ? 1.f : 0.f;  // 1 + body_splits CTAs per slice
  }
  __syncthreads();
  if (s_stat[79] != 0.f) {
    __threadfence();
    combine_slice(p, slice, s_stat + 80);
    if (tid == 0) p.tickets[slice] = 0u;  // ready for the next launch (stream order)
  }
}

constexpr int attn_ring_bytes(int bits) {
  // per-warp stages while streaming; at least the 16 KB of warp outputs they are reused for
  return bits == 16 ? 4 * kMaxGroup * kHeadDim * 4
                    : (4 * (bits == 8 ? 3 : 4) * tile_bytes(bits) > 4 * kMaxGroup * kHeadDim * 4
                           ? 4 * (bits == 8 ? 3 : 4) * tile_bytes(bits)
                           : 4 * kMaxGroup * kHeadDim * 4);
}

template <int BODY_BITS>
__global__ void __launch_bounds__(128, 4) decode_attn_splitk_kernel(const AttnParams p) {
  __shared__ __align__(16) float s_q[kMaxGroup][kHeadDim];
  __shared__ float s_stat[80 + 72];  // head stats, warp stats, ticket flag, combine weights (<= 65 CTAs)
  extern __shared__ __align__(128) uint8_t ring[];
  if (blockIdx.x == 0) run_cta<16>(p, s_q, s_stat, ring);
  else run_cta<BODY_BITS>(p, s_q, s_stat, ring);
}

}  // namespace pmkvq

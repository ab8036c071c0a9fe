// Offline calibration of the equalization vector (Sec. 3.3): RoPE with positional interpolation
// (Eq. 12: the position index is multiplied by s inside the rotation, so a short calibration text
// sweeps the angles of a text s times longer) applied to pre-RoPE Keys, then the per-channel
// absolute maximum over all tokens and sequences of a KV head, lambda_i = max(amax_i, floor)^alpha
// (Eq. 10).  One pass over the Keys; the maxima meet in the output buffer through atomicMax on the
// bit patterns of non-negative floats, so the kernel needs no workspace.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "kernels_attn.cuh"
#include "kernels_cache.cuh"
#include "layout.cuh"

namespace pmkvq {

// amax_bits [kv_heads][128] must be zero before the launch.  Grid: one CTA per chunk of tokens;
// thread t owns channel pair (t % 64, t % 64 + 64) of vector (t / 64 + 2 j) of the token.
__global__ void __launch_bounds__(128) calib_absmax_kernel(const uint16_t *__restrict__ K, unsigned *amax_bits,
                                                           int n_tokens, int n_vec /* sequences x kv_heads */,
                                                           int kv_heads, int tokens_per_cta, double pos_scale,
                                                           double theta) {
  __shared__ float s_cos[64], s_sin[64];
  __shared__ unsigned s_max[8][kHeadDim];  // per kv head (at most 8 per pass), per channel
  const int tid = threadIdx.x, pair = tid & 63, sub = tid >> 6;
  const int t0 = blockIdx.x * tokens_per_cta, t1 = min(n_tokens, t0 + tokens_per_cta);
  const double inv_freq = pow(theta, -2.0 * pair / (double)kHeadDim);
  for (int h0 = 0; h0 < kv_heads; h0 += 8) {
    for (int i = tid; i < 8 * kHeadDim; i += 128) (&s_max[0][0])[i] = 0u;
    __syncthreads();
    for (int t = t0; t < t1; ++t) {
      if (tid < 64) {
        double s, c;
        sincos((double)t * pos_scale * inv_freq, &s, &c);
        s_cos[pair] = (float)c;
        s_sin[pair] = (float)s;
      }
      __syncthreads();
      const float c = s_cos[pair], s = s_sin[pair];
      for (int v = sub; v < n_vec; v += 2) {
        const int head = v % kv_heads;
        if (head < h0 || head >= h0 + 8) continue;
        const uint16_t *src = K + ((size_t)t * n_vec + v) * kHeadDim;
        const float x1 = __uint_as_float((uint32_t)src[pair] << 16), x2 = __uint_as_float((uint32_t)src[pair + 64] << 16);
        const float y1 = __fsub_rn(__fmul_rn(x1, c), __fmul_rn(x2, s));  // Eq. 11 with the scaled position
        const float y2 = __fadd_rn(__fmul_rn(x1, s), __fmul_rn(x2, c));
        atomicMax(&s_max[head - h0][pair], __float_as_uint(fabsf(y1)));
        atomicMax(&s_max[head - h0][pair + 64], __float_as_uint(fabsf(y2)));
      }
      __syncthreads();
    }
    for (int i = tid; i < 8 * kHeadDim; i += 128) {
      const int head = h0 + i / kHeadDim;
      if (head < kv_heads && (&s_max[0][0])[i]) atomicMax(amax_bits + (size_t)head * kHeadDim + (i % kHeadDim), (&s_max[0][0])[i]);
    }
    __syncthreads();
  }
}

// In place: bit pattern of amax -> lambda = max(amax, floor)^alpha (Eq. 10).
__global__ void calib_finish_kernel(float *lambda, int n, float floor_value, float alpha) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) lambda[i] = powf(fmaxf(lambda[i], floor_value), alpha);
}

// ---------------------------------------------------------------------------------------------
// alpha of Eq. 10 by grid search (Sec. 4.1.1): for every alpha of the grid, the squared error between the
// causal self-attention of the calibration tensors and the same operator on what the cache would hold
// at `bits` (Eq. 9: Queries times Lambda, Keys times Lambda^-1 quantized at 16 bit and taken down the
// Eq. 3 chain; Values quantized likewise).  Keys and Queries are rotated on the fly with the
// interpolated RoPE of Eq. 12 from a (cos, sin) table.
// ---------------------------------------------------------------------------------------------

// table[t][pair] = (cos, sin) of pos_scale * t * theta^(-2 pair / 128), rounded from fp64.
__global__ void rope_table_kernel(float2 *table, int n_tokens, double pos_scale, double theta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_tokens * 64) return;
  const int t = i >> 6, pair = i & 63;
  double s, c;
  sincos((double)t * pos_scale * pow(theta, -2.0 * pair / (double)kHeadDim), &s, &c);
  table[i] = make_float2((float)c, (float)s);
}

constexpr int kGridQueries = 64;            // queries of one CTA: four warps of 16
constexpr int kGridKeys = 32;               // keys per shared-memory tile
constexpr int kMaxAlphas = 64;
__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// A tile in shared memory: four planes (K hi, K lo, V hi, V lo) of kGridKeys rows of 128 fp16; a row takes 272
// bytes so that the eight 16-byte rows of an 8 x 8 ldmatrix tile fall into different banks.
constexpr int kGridRowBytes = 2 * kHeadDim + 16;
constexpr int kGridPlaneBytes = kGridKeys * kGridRowBytes;
constexpr int kGridStageBytes = 4 * kGridPlaneBytes;
constexpr int kGridSmemBytes = 2 * kGridStageBytes;  // two stages

// x = hi + lo with both parts fp16: 22 significant bits (an absolute 2^-25 below 1/8), which three tensor-core
// products hi*hi + hi*lo + lo*hi carry into the fp32 accumulator.
__device__ __forceinline__ void split_half(float x, __half &hi, __half &lo) {
  hi = __float2half_rn(x);
  lo = __float2half_rn(x - __half2float(hi));
}
__device__ __forceinline__ void split_half2(float x, float y, uint32_t &hi, uint32_t &lo) {
  __half hx, lx, hy, ly;
  split_half(x, hx, lx);
  split_half(y, hy, ly);
  const __half2 h = __halves2half2(hx, hy), l = __halves2half2(lx, ly);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// One token's 4 channels per lane (channels 4 lane .. 4 lane + 3): rotate by the token's angles.  The
// partner channel (+-64) sits in lane ^ 16.
__device__ __forceinline__ void rotate_token(float (&x)[4], const float2 *__restrict__ table_t, int lane) {
  const int pair0 = (lane & 15) * 4;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float other = __shfl_xor_sync(0xffffffffu, x[e], 16);
    const float2 cs = table_t[pair0 + e];
    // lanes 0..15 hold x1 (channel < 64): y1 = x1 c - x2 s;  lanes 16..31 hold x2: y2 = x1 s + x2 c
    x[e] = lane < 16 ? __fsub_rn(__fmul_rn(x[e], cs.x), __fmul_rn(other, cs.y))
                     : __fadd_rn(__fmul_rn(other, cs.y), __fmul_rn(x[e], cs.x));
  }
}

// Eq. 1-2 at 16 bit on one token's 128 channels spread over a warp, the Eq. 3 chain to `bits`, and back
// to real values: x <- S_b * code_b + Z.
__device__ __forceinline__ void quantize_dequantize_token(float (&x)[4], int bits) {
  float mn = fminf(fminf(x[0], x[1]), fminf(x[2], x[3]));
  float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  const float s16 = __fdiv_rn(__fsub_rn(mx, mn), 65535.0f);
  float sb = s16;
  for (int w = 8; w >= bits; w >>= 1) sb = __fmul_rn(sb, (float)((1 << w) + 1));
  const bool plain = s16 >= 0x1p-60f && s16 <= 0x1p60f;  // else: constant token (0 / 0 converts to code 0) or absurd range
  const float y = plain ? __frcp_rn(s16) : 0.f;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float d = __fsub_rn(x[e], mn);
    const int c = plain ? code_of_quotient(quotient_rn(d, s16, y)) : min(max(__float2int_rn(__fdiv_rn(d, s16)), 0), 65535);
    x[e] = fmaf((float)shift_chain((uint32_t)c, bits), sb, mn);
  }
}

__device__ __forceinline__ void load_bf16x4(const uint16_t *src, float (&x)[4]) {
  const uint2 raw = *reinterpret_cast<const uint2 *>(src);
  x[0] = __uint_as_float(raw.x << 16);
  x[1] = __uint_as_float(raw.x & 0xFFFF0000u);
  x[2] = __uint_as_float(raw.y << 16);
  x[3] = __uint_as_float(raw.y & 0xFFFF0000u);
}

// Four values of vector `vec` (channels 4 lane ..) as fp16 hi and lo parts: the hi plane [n_vectors][128] fp16
// is followed by the lo plane, together the 4 bytes per element of the fp32 buffer they replace.
__device__ __forceinline__ void store_split4(float *out, long long n_vectors, long long vec, int lane, const float (&x)[4]) {
  uint2 hi, lo;
  split_half2(x[0], x[1], hi.x, lo.x);
  split_half2(x[2], x[3], hi.y, lo.y);
  __half *planes = reinterpret_cast<__half *>(out);
  *reinterpret_cast<uint2 *>(planes + vec * kHeadDim + 4 * lane) = hi;
  *reinterpret_cast<uint2 *>(planes + (n_vectors + vec) * kHeadDim + 4 * lane) = lo;
}

// One pass's Keys and Values as the attention kernel reads them: [n_tokens][n_seq][kv_heads][128] as fp16 hi and
// lo planes (see store_split4).
// One warp per (token, sequence, KV head) vector, lane l on channels 4 l .. 4 l + 3.
//   alpha_index < 0  (the unquantized operator): k_out = rotated Keys, v_out = Values
//   alpha_index >= 0: k_out = dequantized Q_bits(rotated Keys * Lambda^-1), lambda = max(amax, floor)^alpha;
//                     v_out (if not null) = dequantized Q_bits(Values), which no alpha changes
__global__ void __launch_bounds__(128) alpha_grid_prep_kernel(const uint16_t *__restrict__ K, const uint16_t *__restrict__ V,
                                                              const float *__restrict__ amax, const float2 *__restrict__ table,
                                                              const float *__restrict__ alphas, int alpha_index,
                                                              long long n_vectors, int vec_per_token, int kv_heads, int bits,
                                                              float floor_value, float *__restrict__ k_out,
                                                              float *__restrict__ v_out) {
  const int lane = threadIdx.x & 31;
  const long long vec = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (vec >= n_vectors) return;
  const int t = (int)(vec / vec_per_token), kv_head = (int)(vec % kv_heads);
  float xk[4];
  load_bf16x4(K + vec * kHeadDim + 4 * lane, xk);
  rotate_token(xk, table + (size_t)t * 64, lane);
  if (alpha_index >= 0) {
    const float alpha = alphas[alpha_index];
    const float4 am = *reinterpret_cast<const float4 *>(amax + (size_t)kv_head * kHeadDim + 4 * lane);
    xk[0] = __fmul_rn(xk[0], __fdiv_rn(1.0f, powf(fmaxf(am.x, floor_value), alpha)));
    xk[1] = __fmul_rn(xk[1], __fdiv_rn(1.0f, powf(fmaxf(am.y, floor_value), alpha)));
    xk[2] = __fmul_rn(xk[2], __fdiv_rn(1.0f, powf(fmaxf(am.z, floor_value), alpha)));
    xk[3] = __fmul_rn(xk[3], __fdiv_rn(1.0f, powf(fmaxf(am.w, floor_value), alpha)));
    quantize_dequantize_token(xk, bits);
  }
  store_split4(k_out, n_vectors, vec, lane, xk);
  if (v_out) {
    float xv[4];
    load_bf16x4(V + vec * kHeadDim + 4 * lane, xv);
    if (alpha_index >= 0) quantize_dequantize_token(xv, bits);
    store_split4(v_out, n_vectors, vec, lane, xv);
  }
}

// One pass of causal self-attention on the tensor cores at fp32-like precision.  Grid: (query blocks, query
// heads, sequences); a CTA takes 64 queries, a warp 16 of them against all their keys.
// Q: bf16 [n_tokens][n_seq][kv_heads * group][128] before RoPE (rotated here, and scaled by lambda(alpha)
// when alpha_index >= 0, Eq. 9); k_in, v_in: this pass's tensors from alpha_grid_prep_kernel (fp16 hi and lo
// planes).  alpha_index < 0: the outputs go to o_ref [n_tokens][n_seq][q_heads][128]; otherwise the squared
// differences to o_ref are added to loss_sums[alpha_index] (fp64).
// Every operand of the two contractions is a sum of two fp16 numbers (queries and probabilities split in
// registers, keys and values by the prep kernel), and a product takes three mma.sync.m16n8k16 (hi hi, hi lo,
// lo hi; the lo lo term is below 2^-22 of the product): the loss is a small difference of two attention
// outputs, so plain fp16 or bf16 operands would drown it.  Key / Value tiles of 32 tokens arrive through a
// two-stage cp.async ring; ldmatrix (transposed for the Values) builds the B fragments.
__global__ void __launch_bounds__(128, 2) alpha_grid_attn_kernel(const uint16_t *__restrict__ Q, const float *__restrict__ k_in,
                                                                 const float *__restrict__ v_in, const float *__restrict__ amax,
                                                                 const float2 *__restrict__ table,
                                                                 const float *__restrict__ alphas, int alpha_index, int n_tokens,
                                                                 int n_seq, int kv_heads, int group, float floor_value,
                                                                 float *__restrict__ o_ref, double *loss_sums) {
  extern __shared__ __align__(16) uint8_t s_tiles[];  // [stage][K hi | K lo | V hi | V lo][32 keys][272 bytes]
  __shared__ float s_lam[kHeadDim];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, tig = lane & 3;
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;  // long rows first
  const int q_head = blockIdx.y, seq = blockIdx.z, kv_head = q_head / group, q_heads = kv_heads * group;
  const int q0 = qb * kGridQueries + 16 * warp;                   // first of the warp's queries
  const int q_last = min(n_tokens, (qb + 1) * kGridQueries) - 1;  // last live query of the CTA
  const size_t kv_row = (size_t)n_seq * kv_heads * kHeadDim;      // halfs from one token to the next
  const size_t plane = (size_t)n_tokens * kv_row;                 // halfs from the hi plane to the lo plane
  const __half *kv_base[4];
  kv_base[0] = reinterpret_cast<const __half *>(k_in) + ((size_t)seq * kv_heads + kv_head) * kHeadDim;
  kv_base[1] = kv_base[0] + plane;
  kv_base[2] = reinterpret_cast<const __half *>(v_in) + ((size_t)seq * kv_heads + kv_head) * kHeadDim;
  kv_base[3] = kv_base[2] + plane;
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)kHeadDim);
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(s_tiles);

  // tile j -> stage j & 1: thread i copies 16-byte pieces i, i + 128, ... of the 4 x 32 rows of 256 bytes
  auto issue = [&](int j) {
    const uint32_t dst = ring + (uint32_t)((j & 1) * kGridStageBytes);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const int piece = tid + 128 * c, pl = piece >> 9, row = (piece >> 4) & 31, col = piece & 15;
      const int t = min(j * kGridKeys + row, n_tokens - 1);  // rows behind the last token are masked below
      cp_async16(dst + (uint32_t)(pl * kGridPlaneBytes + row * kGridRowBytes + col * 16), kv_base[pl] + (size_t)t * kv_row + col * 8);
    }
  };
  const int n_tiles = q_last / kGridKeys + 1;
  issue(0);
  cp_async_commit();

  s_lam[tid] = alpha_index >= 0 ? powf(fmaxf(amax[(size_t)kv_head * kHeadDim + tid], floor_value), alphas[alpha_index]) : 1.0f;
  __syncthreads();

  // ---- the warp's queries as A fragments: rotated, equalized, pre-scaled, split; qh / ql[k-step][register] ----
  // register 0: row g, channels 16 ks + 2 tig, + 1; 1: row g + 8; 2: row g, channels + 8; 3: row g + 8, channels + 8
  uint32_t qh[8][4], ql[8][4];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int qi = min(q0 + g + 8 * rr, n_tokens - 1);  // a dead row repeats the last query; its output is dropped
    const uint16_t *src = Q + (((size_t)qi * n_seq + seq) * q_heads + q_head) * kHeadDim;
    const float2 *tab = table + (size_t)qi * 64;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
#pragma unroll
      for (int c8 = 0; c8 < 2; ++c8) {
        const int ch = 16 * ks + 8 * c8 + 2 * tig;  // channels ch, ch + 1 and their rotation partners + 64
        const uint32_t r1 = *reinterpret_cast<const uint32_t *>(src + ch), r2 = *reinterpret_cast<const uint32_t *>(src + ch + 64);
        float y1[2], y2[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float x1 = __uint_as_float(e ? (r1 & 0xFFFF0000u) : (r1 << 16));
          const float x2 = __uint_as_float(e ? (r2 & 0xFFFF0000u) : (r2 << 16));
          const float2 cs = tab[ch + e];
          y1[e] = __fsub_rn(__fmul_rn(x1, cs.x), __fmul_rn(x2, cs.y)) * s_lam[ch + e] * scale_log2;
          y2[e] = __fadd_rn(__fmul_rn(x1, cs.y), __fmul_rn(x2, cs.x)) * s_lam[ch + e + 64] * scale_log2;
        }
        split_half2(y1[0], y1[1], qh[ks][2 * c8 + rr], ql[ks][2 * c8 + rr]);
        split_half2(y2[0], y2[1], qh[ks + 4][2 * c8 + rr], ql[ks + 4][2 * c8 + rr]);
      }
  }

  float acc[16][4];          // O[16 queries][128]: n-block nb holds channels 8 nb + 2 tig, + 1 of rows g (0, 1) and g + 8 (2, 3)
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};  // rows g, g + 8 (l: this thread's columns only)
#pragma unroll
  for (int nb = 0; nb < 16; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
  // ldmatrix row addresses of this lane inside a plane: lane = 8 mat + row
  const int lm_row = lane & 7, lm_mat = lane >> 3;
  const uint32_t k_lane_off = (uint32_t)((((lm_mat >> 1) * 8 + lm_row) * kGridRowBytes) + (lm_mat & 1) * 16);  // keys of two n-blocks, channels k0 / k0 + 8
  const uint32_t v_lane_off = (uint32_t)((((lm_mat & 1) * 8 + lm_row) * kGridRowBytes) + (lm_mat >> 1) * 16);  // keys k0 / k0 + 8, channels of two n-blocks

  for (int j = 0; j < n_tiles; ++j) {
    __syncthreads();  // everyone is done with the stage that tile j + 1 will overwrite
    if (j + 1 < n_tiles) issue(j + 1);
    cp_async_commit();
    cp_async_wait<1>();  // tile j has landed (this thread's pieces)
    __syncthreads();     // ... and everyone else's
    const int k0 = j * kGridKeys;
    if (k0 > q0 + 15) continue;  // every key of the tile lies behind every query of this warp (the barriers above still run)
    const uint32_t st = ring + (uint32_t)((j & 1) * kGridStageBytes);
    // ---- S[16 queries][32 keys] = Q K^T ----
    float sc[4][4];
#pragma unroll
    for (int nb = 0; nb < 4; ++nb) sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int np = 0; np < 2; ++np) {  // n-blocks 2 np, 2 np + 1
        uint32_t bh[4], bl[4];
        const uint32_t a = st + k_lane_off + (uint32_t)(np * 16 * kGridRowBytes + ks * 32);
        ldsm_x4(a, bh);
        ldsm_x4(a + kGridPlaneBytes, bl);
        mma_f16(sc[2 * np], qh[ks], bh[0], bh[1]);
        mma_f16(sc[2 * np], qh[ks], bl[0], bl[1]);
        mma_f16(sc[2 * np], ql[ks], bh[0], bh[1]);
        mma_f16(sc[2 * np + 1], qh[ks], bh[2], bh[3]);
        mma_f16(sc[2 * np + 1], qh[ks], bl[2], bl[3]);
        mma_f16(sc[2 * np + 1], ql[ks], bh[2], bh[3]);
      }
    }
    // ---- causal mask, running maximum, probabilities ----
    const bool diagonal = k0 + kGridKeys - 1 > q0;  // some key of the tile may lie behind some query of the warp
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int qi = q0 + g + 8 * rr;
      float mx = -INFINITY;
#pragma unroll
      for (int nb = 0; nb < 4; ++nb)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          if (diagonal && k0 + 8 * nb + 2 * tig + e > qi) sc[nb][2 * rr + e] = -INFINITY;
          mx = fmaxf(mx, sc[nb][2 * rr + e]);
        }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      // key 0 is live for every query and sits in the first tile, so m is finite from the first tile on
      const float m_new = fmaxf(m[rr], mx);
      const float corr = ex2_fast(m[rr] - m_new);  // 0 on the first tile
      m[rr] = m_new;
      l[rr] *= corr;
#pragma unroll
      for (int nb = 0; nb < 16; ++nb) { acc[nb][2 * rr] *= corr; acc[nb][2 * rr + 1] *= corr; }
#pragma unroll
      for (int nb = 0; nb < 4; ++nb)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float pe = ex2_fast(sc[nb][2 * rr + e] - m_new);
          sc[nb][2 * rr + e] = pe;
          l[rr] += pe;
        }
    }
    // ---- O += P V: the probability fragments of two key n-blocks are the A fragment of one k-step ----
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      uint32_t ph[4], pl[4];
      split_half2(sc[2 * ks][0], sc[2 * ks][1], ph[0], pl[0]);
      split_half2(sc[2 * ks][2], sc[2 * ks][3], ph[1], pl[1]);
      split_half2(sc[2 * ks + 1][0], sc[2 * ks + 1][1], ph[2], pl[2]);
      split_half2(sc[2 * ks + 1][2], sc[2 * ks + 1][3], ph[3], pl[3]);
#pragma unroll
      for (int np = 0; np < 8; ++np) {  // channel n-blocks 2 np, 2 np + 1
        uint32_t bh[4], bl[4];
        const uint32_t a = st + 2 * kGridPlaneBytes + v_lane_off + (uint32_t)(ks * 16 * kGridRowBytes + np * 32);
        ldsm_x4_trans(a, bh);
        ldsm_x4_trans(a + kGridPlaneBytes, bl);
        mma_f16(acc[2 * np], ph, bh[0], bh[1]);
        mma_f16(acc[2 * np], ph, bl[0], bl[1]);
        mma_f16(acc[2 * np], pl, bh[0], bh[1]);
        mma_f16(acc[2 * np + 1], ph, bh[2], bh[3]);
        mma_f16(acc[2 * np + 1], ph, bl[2], bl[3]);
        mma_f16(acc[2 * np + 1], pl, bh[2], bh[3]);
      }
    }
  }
  cp_async_wait<0>();

  // ---- the pass's output: keep it (the unquantized pass) or compare with the kept one ----
  float err = 0.f;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    float ls = l[rr];
    ls += __shfl_xor_sync(0xffffffffu, ls, 1);
    ls += __shfl_xor_sync(0xffffffffu, ls, 2);
    const int qi = q0 + g + 8 * rr;
    if (qi < n_tokens) {
      const float inv_l = __fdiv_rn(1.0f, ls);
      float *kept = o_ref + (((size_t)qi * n_seq + seq) * q_heads + q_head) * kHeadDim + 2 * tig;
#pragma unroll
      for (int nb = 0; nb < 16; ++nb) {
        float2 o = make_float2(acc[nb][2 * rr] * inv_l, acc[nb][2 * rr + 1] * inv_l);
        if (alpha_index < 0) {
          *reinterpret_cast<float2 *>(kept + 8 * nb) = o;
        } else {
          const float2 r = *reinterpret_cast<const float2 *>(kept + 8 * nb);
          o.x -= r.x; o.y -= r.y;
          err = fmaf(o.x, o.x, err); err = fmaf(o.y, o.y, err);
        }
      }
    }
  }
  if (alpha_index >= 0) {
    double e = (double)err;
#pragma unroll
    for (int o = 16; o; o >>= 1) e += __shfl_xor_sync(0xffffffffu, e, o);
    if (lane == 0) atomicAdd(loss_sums + alpha_index, e);
  }
}

}  // namespace pmkvq

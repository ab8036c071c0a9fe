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

constexpr int kQPT = 4;                     // queries per thread
constexpr int kGridQueries = 16 * kQPT;     // queries of one CTA: 16 groups of kQPT queries, 8 threads per group
constexpr int kGridKeys = 32;     // keys per shared-memory tile
constexpr int kMaxAlphas = 64;
__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
constexpr int kGridSmemBytes = 2 * 2 * kGridKeys * kHeadDim * 4;  // two stages of a K tile and a V tile

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

// One pass's Keys and Values as the attention kernel reads them: fp32 [n_tokens][n_seq][kv_heads][128].
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
  *reinterpret_cast<float4 *>(k_out + vec * kHeadDim + 4 * lane) = make_float4(xk[0], xk[1], xk[2], xk[3]);
  if (v_out) {
    float xv[4];
    load_bf16x4(V + vec * kHeadDim + 4 * lane, xv);
    if (alpha_index >= 0) quantize_dequantize_token(xv, bits);
    *reinterpret_cast<float4 *>(v_out + vec * kHeadDim + 4 * lane) = make_float4(xv[0], xv[1], xv[2], xv[3]);
  }
}

// One pass of causal self-attention in fp32.  Grid: (query blocks, query heads, sequences).
// Q: bf16 [n_tokens][n_seq][kv_heads * group][128] before RoPE (rotated here, and scaled by lambda(alpha)
// when alpha_index >= 0, Eq. 9); k_in, v_in: this pass's tensors from alpha_grid_prep_kernel.
// alpha_index < 0: the outputs go to o_ref [n_tokens][n_seq][q_heads][128]; otherwise the squared
// differences to o_ref are added to loss_sums[alpha_index] (fp64).
// Thread (group, part) works on the group's kQPT consecutive queries and on channels 32 c + 4 part + e
// (c < 4, e < 4): a rotation pair (i, i + 64) stays in one thread, the 8 parts read one 128-byte run of a
// key row, every value read from shared memory feeds kQPT multiply-adds (one per query), and two keys are
// taken per turn so that their score chains, shuffles and exponentials overlap.  Key / Value tiles of 32
// tokens arrive through a two-stage cp.async ring.
__global__ void __launch_bounds__(128) alpha_grid_attn_kernel(const uint16_t *__restrict__ Q, const float *__restrict__ k_in,
                                                              const float *__restrict__ v_in, const float *__restrict__ amax,
                                                              const float2 *__restrict__ table,
                                                              const float *__restrict__ alphas, int alpha_index, int n_tokens,
                                                              int n_seq, int kv_heads, int group, float floor_value,
                                                              float *__restrict__ o_ref, double *loss_sums) {
  extern __shared__ __align__(16) float s_dyn[];  // [stage][K | V][32 keys][128]
  __shared__ float s_lam[kHeadDim];
  const int tid = threadIdx.x, lane = tid & 31;
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;  // long rows first
  const int q_head = blockIdx.y, seq = blockIdx.z, kv_head = q_head / group, q_heads = kv_heads * group;
  const int ql0 = (tid >> 3) * kQPT, part = tid & 7;  // first of the thread's queries inside the CTA
  const int q0 = qb * kGridQueries + ql0;
  const int q_last = min(n_tokens, (qb + 1) * kGridQueries) - 1;  // last live query of the CTA
  const size_t kv_row = (size_t)n_seq * kv_heads * kHeadDim;
  const float *k_base = k_in + ((size_t)seq * kv_heads + kv_head) * kHeadDim;
  const float *v_base = v_in + ((size_t)seq * kv_heads + kv_head) * kHeadDim;
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)kHeadDim);
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(s_dyn);
  constexpr int kStageFloats = 2 * kGridKeys * kHeadDim;

  // tile j -> stage j & 1: thread i copies 16-byte pieces i, i + 128, ... of the 32 x 512-byte rows
  auto issue = [&](int j) {
    const uint32_t dst = ring + (uint32_t)((j & 1) * kStageFloats * 4);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int piece = tid + 128 * c, row = piece >> 5, col = (piece & 31) * 4;
      const int t = min(j * kGridKeys + row, n_tokens - 1);  // rows behind the last token are masked below
      cp_async16(dst + (uint32_t)((row * kHeadDim + col) * 4), k_base + (size_t)t * kv_row + col);
      cp_async16(dst + (uint32_t)(((kGridKeys + row) * kHeadDim + col) * 4), v_base + (size_t)t * kv_row + col);
    }
  };
  const int n_tiles = q_last / kGridKeys + 1;
  issue(0);
  cp_async_commit();

  s_lam[tid] = alpha_index >= 0 ? powf(fmaxf(amax[(size_t)kv_head * kHeadDim + tid], floor_value), alphas[alpha_index]) : 1.0f;
  __syncthreads();
  // the thread's rotated, equalized, pre-scaled query channels: qe[n][4 c + e]
  float qe[kQPT][16], acc[kQPT][16], m[kQPT], l[kQPT];
#pragma unroll
  for (int n = 0; n < kQPT; ++n) {
    m[n] = -INFINITY;
    l[n] = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) { qe[n][i] = 0.f; acc[n][i] = 0.f; }
    const int qi = q0 + n;
    if (qi < n_tokens) {
      const uint16_t *src = Q + (((size_t)qi * n_seq + seq) * q_heads + q_head) * kHeadDim;
      const float2 *tab = table + (size_t)qi * 64;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float x1[4], x2[4];
        load_bf16x4(src + 32 * c + 4 * part, x1);
        load_bf16x4(src + 64 + 32 * c + 4 * part, x2);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int ch = 32 * c + 4 * part + e;
          const float2 cs = tab[ch];
          const float y1 = __fsub_rn(__fmul_rn(x1[e], cs.x), __fmul_rn(x2[e], cs.y));
          const float y2 = __fadd_rn(__fmul_rn(x1[e], cs.y), __fmul_rn(x2[e], cs.x));
          qe[n][4 * c + e] = y1 * s_lam[ch] * scale_log2;
          qe[n][4 * (c + 2) + e] = y2 * s_lam[ch + 64] * scale_log2;
        }
      }
    }
  }

  for (int j = 0; j < n_tiles; ++j) {
    __syncthreads();  // everyone is done with the stage that tile j + 1 will overwrite
    if (j + 1 < n_tiles) issue(j + 1);
    cp_async_commit();
    cp_async_wait<1>();  // tile j has landed (this thread's pieces)
    __syncthreads();     // ... and everyone else's
    const float(*s_k)[kHeadDim] = reinterpret_cast<const float(*)[kHeadDim]>(s_dyn + (j & 1) * kStageFloats);
    const float(*s_v)[kHeadDim] = s_k + kGridKeys;
    const int k0 = j * kGridKeys;
    const int k_hi = min(kGridKeys, q_last - k0 + 1);
    for (int kk = 0; kk < k_hi; kk += 2) {  // two keys per turn: their dependent chains overlap
      // (a second key beyond k_hi lies behind every query of the CTA and is masked below; its row exists)
      float s[2][kQPT];
#pragma unroll
      for (int n = 0; n < kQPT; ++n) s[0][n] = s[1][n] = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float4 ka = *reinterpret_cast<const float4 *>(&s_k[kk][32 * c + 4 * part]);
        const float4 kb = *reinterpret_cast<const float4 *>(&s_k[kk + 1][32 * c + 4 * part]);
#pragma unroll
        for (int n = 0; n < kQPT; ++n) {
          s[0][n] = fmaf(qe[n][4 * c], ka.x, s[0][n]); s[1][n] = fmaf(qe[n][4 * c], kb.x, s[1][n]);
          s[0][n] = fmaf(qe[n][4 * c + 1], ka.y, s[0][n]); s[1][n] = fmaf(qe[n][4 * c + 1], kb.y, s[1][n]);
          s[0][n] = fmaf(qe[n][4 * c + 2], ka.z, s[0][n]); s[1][n] = fmaf(qe[n][4 * c + 2], kb.z, s[1][n]);
          s[0][n] = fmaf(qe[n][4 * c + 3], ka.w, s[0][n]); s[1][n] = fmaf(qe[n][4 * c + 3], kb.w, s[1][n]);
        }
      }
#pragma unroll
      for (int o = 1; o <= 4; o <<= 1)
#pragma unroll
        for (int n = 0; n < kQPT; ++n) {
          s[0][n] += __shfl_xor_sync(0xffffffffu, s[0][n], o);
          s[1][n] += __shfl_xor_sync(0xffffffffu, s[1][n], o);
        }
      float p[2][kQPT];
#pragma unroll
      for (int n = 0; n < kQPT; ++n) {
        // causal mask (the eight threads of a group agree); key 0 is live for every query, so m is finite
        // from the first turn on
        const float sa = (k0 + kk <= q0 + n) ? s[0][n] : -INFINITY;
        const float sb = (k0 + kk + 1 <= q0 + n) ? s[1][n] : -INFINITY;
        const float mx = fmaxf(sa, sb);
        if (mx > m[n]) {
          const float corr = ex2_fast(m[n] - mx);  // 0 on the first key
          l[n] *= corr;
#pragma unroll
          for (int i = 0; i < 16; ++i) acc[n][i] *= corr;
          m[n] = mx;
        }
        p[0][n] = ex2_fast(sa - m[n]);
        p[1][n] = ex2_fast(sb - m[n]);
        l[n] += p[0][n] + p[1][n];
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float4 va = *reinterpret_cast<const float4 *>(&s_v[kk][32 * c + 4 * part]);
        const float4 vb = *reinterpret_cast<const float4 *>(&s_v[kk + 1][32 * c + 4 * part]);
#pragma unroll
        for (int n = 0; n < kQPT; ++n) {
          acc[n][4 * c] = fmaf(p[1][n], vb.x, fmaf(p[0][n], va.x, acc[n][4 * c]));
          acc[n][4 * c + 1] = fmaf(p[1][n], vb.y, fmaf(p[0][n], va.y, acc[n][4 * c + 1]));
          acc[n][4 * c + 2] = fmaf(p[1][n], vb.z, fmaf(p[0][n], va.z, acc[n][4 * c + 2]));
          acc[n][4 * c + 3] = fmaf(p[1][n], vb.w, fmaf(p[0][n], va.w, acc[n][4 * c + 3]));
        }
      }
    }
  }
  cp_async_wait<0>();

  // ---- the pass's output: keep it (the unquantized pass) or compare with the kept one ----
  float err = 0.f;
#pragma unroll
  for (int n = 0; n < kQPT; ++n) {
    if (q0 + n < n_tokens) {
      const float inv_l = __fdiv_rn(1.0f, l[n]);
      float *kept = o_ref + (((size_t)(q0 + n) * n_seq + seq) * q_heads + q_head) * kHeadDim + 4 * part;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float4 o = make_float4(acc[n][4 * c] * inv_l, acc[n][4 * c + 1] * inv_l, acc[n][4 * c + 2] * inv_l,
                               acc[n][4 * c + 3] * inv_l);
        if (alpha_index < 0) {
          *reinterpret_cast<float4 *>(kept + 32 * c) = o;
        } else {
          const float4 r = *reinterpret_cast<const float4 *>(kept + 32 * c);
          o.x -= r.x; o.y -= r.y; o.z -= r.z; o.w -= r.w;
          err = fmaf(o.x, o.x, err); err = fmaf(o.y, o.y, err); err = fmaf(o.z, o.z, err); err = fmaf(o.w, o.w, err);
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

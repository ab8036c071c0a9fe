// Offline calibration of the equalization vector (Sec. 3.3): RoPE with positional interpolation
// (Eq. 12: the position index is multiplied by s inside the rotation, so a short calibration text
// sweeps the angles of a text s times longer) applied to pre-RoPE Keys, then the per-channel
// absolute maximum over all tokens and sequences of a KV head, lambda_i = max(amax_i, floor)^alpha
// (Eq. 10).  One pass over the Keys; the maxima meet in the output buffer through atomicMax on the
// bit patterns of non-negative floats, so the kernel needs no workspace.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

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

}  // namespace pmkvq

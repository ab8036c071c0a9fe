// Fused dequantize + GQA decode attention over the packed mixed-precision cache (Eq. 9 + softmax
// attention), split over the sequence (flash-decoding) with a last-arriver combine.
//
// Work decomposition.  Every (batch, kv_head) slice is two runs of 16-token tiles: the INT16 run
// (sink tiles + window ring) and the body run at the block's current width.  A tile of the body
// weighs one unit, an INT16 tile `w16` units (their byte ratio), and every slice starts with a few
// empty units that stand for the fixed cost of a segment.  All units of all slices form one
// line that is cut into equal contiguous pieces, one per CTA of a persistent grid (one CTA of 16
// warps per SM), so every CTA streams the same number of bytes whatever the shape.  The part of a
// CTA's piece that lies in one slice is a "segment": its 16 warps draw the segment's tiles from a
// shared counter (INT16 tiles first, then body tiles, the accumulators changing units in between),
// so they finish together however the SM shares its issue slots among them; each warp keeps its
// own running (max, sum, accumulator), the warps are merged in shared memory and the segment
// publishes one partial (m, l, o[128]) per head.  The CTA that publishes the
// last partial of a slice (atomic ticket, nobody waits) merges the slice and writes the output.
//
// Two contraction paths share this decomposition.  The 4- and 2-bit body, which holds most bytes of a
// cache in its steady state, runs on tcgen05.mma with its code operands in tensor memory
// (kernels_attn_tc.cuh).  INT16 tiles (sink, window) and an 8- or 16-bit body run on warp-level
// mma.sync.m16n8k16 (f16 inputs, f32 accumulate) with register operands, the body tiles staged through a
// per-warp cp.async ring in shared memory (a tile is one contiguous run of bytes); in both paths packed
// codes become MMA operands with one logic operation per pair of codes - a code field left in place
// inside an fp16 bit pattern below bit 11 is the exact value code * 2^(pos-24) (fp16 subnormals and the
// first binade are linear in the bit pattern).
//   scores:  S[h, t]  = sum_i Q''[h, i] * c_K[t, i]      A = Q'' (rows 0-7: fp16 "hi" part of the 8 heads,
//                                                        rows 8-15: the "lo" remainder), B = K codes
//   output:  O^T[i,h] = sum_t c_V[t, i] * w[t, h]        A = V codes, B = w = p * S_V (one fp16)
// The per-token scale and zero-point never touch the codes: q.k = S_K (q.c) + Z_K sum(q) and
// sum_t p_t v_t = sum_t (p_t S_V,t) c_t + sum_t p_t Z_V,t.
//
// Online softmax with a lazy reference: probabilities are taken relative to a per-head reference m
// that is only moved (and the accumulators rescaled) when a score exceeds it by more than
// kMaxAhead, so the common case has no cross-lane traffic at all.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "kernels_cache.cuh"
#include "layout.cuh"
#include "tc05.cuh"

namespace pmkvq {

constexpr int kMaxGroup = 8;         // query heads per KV head handled by one MMA row block
constexpr int kPartialStride = 132;  // floats per (segment, head): m, l, 2 pad, o[128]
constexpr float kNegBig = -1.0e30f;
constexpr float kMaxAhead = 3.0f;    // a score may exceed the reference by this much (log2 units)
constexpr int kAttnWarps = 16;       // one CTA per SM; these warps share the CTA's INT16 / 8- / 16-bit tiles dynamically
constexpr int kAttnThreads = 32 * kAttnWarps;
constexpr int kParts = kAttnWarps + 3;  // partial results a segment merges: one per warp, three of the tensor-memory body

struct AttnParams {
  LayerGeom geom;
  const uint16_t *Q;          // bf16 [batch][q_heads][128]
  const float *lambda;        // [kv_heads][128] of this block
  const unsigned *vmax_bits;  // [n_slices] running max of the INT16 V scales (fp32 bit patterns)
  float *partials;            // [n_ctas + n_slices][8][kPartialStride]
  float *out;                 // fp32 [batch][q_heads][128]
  unsigned *tickets;          // [n_slices], zero between launches: partials of a slice published so far
  int kv_heads, group, q_heads, n_slices;
  int n_tokens, n_sink_eff, win_start, cur_bits;
  int n_body, body_tiles, aux_tiles, sink_tiles;
  int w16;                    // units of one INT16 tile
  int units_lead;             // empty units at the start of every slice: the fixed cost of one more segment
  long long units_aux, units_slice, units_total, units_per_cta;  // units_aux includes units_lead
  // Where this block's units sit on the line that is cut into CTA pieces.  A launch for one block has
  // origin 0 and weight 1; the all-blocks launch strings the blocks together, each unit weighing
  // `unit_weight` fine units (blocks of different widths cost different time per tile).
  long long line_origin;      // fine units before this block's first unit
  int unit_weight;            // fine units per unit
  int cta_origin;             // first CTA that touches this block (partials are numbered from it)
  float qk_scale;             // sm_scale * log2(e)
};

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void *gptr) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gptr) : "memory");
}
// the same at byte offset OFF of both addresses (an immediate: no address arithmetic per copy)
template <int OFF>
__device__ __forceinline__ void cp_async16_at(uint32_t smem_addr, const void *gptr) {
  asm volatile("cp.async.cg.shared.global [%0 + %2], [%1 + %2], 16;\n" ::"r"(smem_addr), "l"(gptr), "n"(OFF) : "memory");
}
template <int N, int I = 0>
__device__ __forceinline__ void cp_async_run(uint32_t smem_addr, const void *gptr) {  // N copies, 512 bytes apart
  if constexpr (I < N) {
    cp_async16_at<I * 512>(smem_addr, gptr);
    cp_async_run<N, I + 1>(smem_addr, gptr);
  }
}
// lane 0 takes the next ticket of a shared-memory counter; every lane gets it
__device__ __forceinline__ int claim_next(int *ctr, int lane) {
  int j = 0;
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(ctr);
  asm volatile(
      "{\n .reg .pred p;\n setp.eq.s32 p, %2, 0;\n @p atom.shared.add.u32 %0, [%1], 1;\n}\n"
      : "+r"(j)
      : "r"(addr), "r"(lane)
      : "memory");
  return __shfl_sync(0xffffffffu, j, 0);
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
__device__ __forceinline__ uint32_t high_bytes(uint32_t x) { return __byte_perm(x, 0u, 0x4341); }  // {b1, 0, b3, 0}

// Per width: bit position of code j of a half-word after extraction, the fp16 exponent budgets
// (Q fragments are scaled by 2^(EQ - pos - e_head) and stay below 2^EQ; w = p * S_V is scaled to at
// most 2^(EP + kMaxAhead)), log2 of the bound on S_b / S_16, and the staging ring (NT tiles are
// consumed per step, SLOTS steps are resident per warp; a warp holds SLOTS - 1 claimed steps, which
// is also how far apart the warps of a CTA can finish, so the ring is kept shallow: 16 warps per SM
// already keep about 70 KB in flight).
template <int BITS> struct Fmt;
template <> struct Fmt<2> {
  static constexpr int N = 8, EQ = 14, EP = 12, SIGMA_LOG2 = 15, NT = 2, SLOTS = 2;
  __host__ __device__ static constexpr int pos(int j) { return j < 5 ? 2 * j : 2 * j - 5; }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[8]) {
    const uint32_t xr = x >> 5;
    e[0] = x & 0x00030003u; e[1] = x & 0x000C000Cu; e[2] = x & 0x00300030u; e[3] = x & 0x00C000C0u;
    e[4] = x & 0x03000300u;
    e[5] = xr & 0x00600060u; e[6] = xr & 0x01800180u; e[7] = xr & 0x06000600u;
  }
};
template <> struct Fmt<4> {
  static constexpr int N = 4, EQ = 14, EP = 12, SIGMA_LOG2 = 13, NT = 2, SLOTS = 2;
  __host__ __device__ static constexpr int pos(int j) { return (j & 1) ? 4 : 0; }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[4]) {
    const uint32_t xr = x >> 8;
    e[0] = x & 0x000F000Fu; e[1] = x & 0x00F000F0u;
    e[2] = xr & 0x000F000Fu; e[3] = xr & 0x00F000F0u;
  }
};
template <> struct Fmt<8> {
  static constexpr int N = 2, EQ = 14, EP = 12, SIGMA_LOG2 = 9, NT = 1, SLOTS = 2;
  __host__ __device__ static constexpr int pos(int) { return 0; }
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t (&e)[2]) {
    e[0] = x & 0x00FF00FFu;
    e[1] = high_bytes(x);
  }
};
// 16 bit: a code is split into its two bytes.  Scores keep two accumulators (low bytes, high bytes)
// against the same Q fragments; for the output the high bytes sit at bit 3 (weight 8) and are
// multiplied by w * 32.  16-bit tiles are read straight from global memory.
template <> struct Fmt<16> {
  static constexpr int N = 1, EQ = 14, EP = 7, SIGMA_LOG2 = 0, NT = 1, SLOTS = 0;
  __host__ __device__ static constexpr int pos(int) { return 0; }
};

// The query fragments of a lane (8 k-steps x 4 registers) depend on the lane, not on the warp: the CTA
// keeps one copy in shared memory and a warp fetches a k-step's fragment right before it uses it
// (8 shared loads per step instead of 32 registers held for the whole segment).
struct QFrag {
  const uint4 *mine;  // entry (k-step s, this lane) at mine[32 s]
  __device__ __forceinline__ void load(int s, uint32_t (&q)[4]) const {
    const uint4 t = mine[32 * s];
    q[0] = t.x; q[1] = t.y; q[2] = t.z; q[3] = t.w;
  }
};

// 16-byte load of tile data: body tiles sit in shared memory, INT16 tiles are read from global
// memory past L1 (another kernel may have written them while this SM still holds old lines).
template <int BITS, class T>
__device__ __forceinline__ T ld_tile(const void *ptr) {
  if constexpr (BITS == 16) return __ldcg(reinterpret_cast<const T *>(ptr));
  else return *reinterpret_cast<const T *>(ptr);
}

struct WarpState {
  float m;          // reference (log2 units) of head g (this lane's quad)
  float2 l, zs;     // sum of probabilities and of p * Z_V, two partial sums each (packed arithmetic)
  float acc[8][4];  // O^T accumulators: [m-tile][channel row g / g+8 x head col 2tig / 2tig+1]
};

// First half of a step: the score dot products of NT consecutive 16-token tiles against the query
// fragments (no scale / zero-point yet), as pairs: dot2[2 nt + r] = tokens (2tig, 2tig+1) of half r.
template <int BITS, int NT>
__device__ __forceinline__ void qk_phase(const uint8_t *tile0, const QFrag &qa, int lane, float2 (&dot2)[2 * NT]) {
  using F = Fmt<BITS>;
  constexpr int TB = tile_bytes(BITS);
  constexpr int CHUNKS = BITS / 2;
  // ---- scores: S = Q'' K^T, heads on M (hi rows 0-7, lo rows 8-15), tokens on N ----
  if constexpr (BITS == 16) {
    const uint8_t *kp = tile0 + lane * 16;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      uint32_t kw[16];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 a = __ldcg(reinterpret_cast<const uint4 *>(kp + (4 * r + q) * 512));
        kw[4 * q] = a.x; kw[4 * q + 1] = a.y; kw[4 * q + 2] = a.z; kw[4 * q + 3] = a.w;
      }
      float lo[4] = {0.f, 0.f, 0.f, 0.f}, hi[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const uint32_t x0 = kw[2 * s], x1 = kw[2 * s + 1];
        uint32_t qf[4];
        qa.load(s, qf);
        mma_f16(lo, qf, x0 & 0x00FF00FFu, x1 & 0x00FF00FFu);
        mma_f16(hi, qf, high_bytes(x0), high_bytes(x1));
      }
      dot2[r] = make_float2(fmaf(256.f, hi[0] + hi[2], lo[0] + lo[2]), fmaf(256.f, hi[1] + hi[3], lo[1] + lo[3]));
    }
  } else {
    // the 2 NT (tile, token half) accumulators advance together: consecutive MMAs are independent
    uint32_t kw[NT][2 * BITS];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const uint8_t *kp = tile0 + nt * TB + lane * 16;
#pragma unroll
      for (int q = 0; q < CHUNKS; ++q) {
        const uint4 a = *reinterpret_cast<const uint4 *>(kp + q * 512);
        kw[nt][4 * q] = a.x; kw[nt][4 * q + 1] = a.y; kw[nt][4 * q + 2] = a.z; kw[nt][4 * q + 3] = a.w;
      }
    }
    float sacc[NT][2][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int r = 0; r < 2; ++r) sacc[nt][r][0] = sacc[nt][r][1] = sacc[nt][r][2] = sacc[nt][r][3] = 0.f;
#pragma unroll
    for (int w = 0; w < BITS; ++w) {
      uint32_t qf[F::N / 2][4];
#pragma unroll
      for (int jj = 0; jj < F::N / 2; ++jj) qa.load((w * F::N) / 2 + jj, qf[jj]);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          uint32_t e[F::N];
          F::extract(kw[nt][r * BITS + w], e);
#pragma unroll
          for (int jj = 0; jj < F::N / 2; ++jj) mma_f16(sacc[nt][r], qf[jj], e[2 * jj], e[2 * jj + 1]);
        }
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        dot2[2 * nt + r] = __fadd2_rn(make_float2(sacc[nt][r][0], sacc[nt][r][1]), make_float2(sacc[nt][r][2], sacc[nt][r][3]));
      }
  }
}

// Second part of a step: scale / zero-point and online softmax of the NT tiles' scores.  Leaves the
// weights w = p * S_V of this lane's tokens in pb (fp16 pairs, the B fragments of the output MMAs) and
// returns the factor by which everything accumulated so far for head g must be multiplied (1 unless the
// reference moved).  `mask` (NT == 1 only) has bit r set when token row r is live.
template <int BITS, int NT, bool MASKED>
__device__ __forceinline__ float softmax_phase(const uint8_t *tile0, uint32_t mask, WarpState &st,
                                               const float2 (&dot2)[2 * NT], float mu, float sumq, float inv_sigma_e,
                                               int lane, uint32_t (&pb)[2 * NT]) {
  using F = Fmt<BITS>;
  static_assert(!(MASKED && NT != 1), "masked tiles are processed one at a time");
  constexpr int TB = tile_bytes(BITS);
  constexpr int NS = 4 * NT;  // scores per lane
  float rescale = 1.0f;
  const int tig = lane & 3;

  // ---- per-token scale / zero-point of this lane's tokens {2tig, 2tig+1, 8+2tig, 9+2tig} of each tile ----
  // (the softmax arithmetic below runs on pairs of scores with the packed fp32x2 instructions)
  constexpr int NP = NS / 2;
  float2 sk[NP], zk[NP], sv[NP], zv[NP];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const float4 *mp = reinterpret_cast<const float4 *>(tile0 + nt * TB + meta_offset(BITS) + tig * 64);
    const float4 a = ld_tile<BITS, float4>(mp), b = ld_tile<BITS, float4>(mp + 1), c = ld_tile<BITS, float4>(mp + 2),
                 d = ld_tile<BITS, float4>(mp + 3);
    sk[2 * nt] = make_float2(a.x, a.y); sk[2 * nt + 1] = make_float2(a.z, a.w);
    zk[2 * nt] = make_float2(b.x, b.y); zk[2 * nt + 1] = make_float2(b.z, b.w);
    sv[2 * nt] = make_float2(c.x, c.y); sv[2 * nt + 1] = make_float2(c.z, c.w);
    zv[2 * nt] = make_float2(d.x, d.y); zv[2 * nt + 1] = make_float2(d.z, d.w);
  }

  // ---- true scores; the reference moves only when one of them runs ahead of it ----
  const float2 mu2 = make_float2(mu, mu), sumq2 = make_float2(sumq, sumq);
  float2 sc[NP];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < NP; ++j) {
    sc[j] = __ffma2_rn(__fmul2_rn(sk[j], mu2), dot2[j], __fmul2_rn(zk[j], sumq2));
    if constexpr (MASKED) {
      const int bit = 8 * (j & 1) + 2 * tig;
      if (!((mask >> bit) & 1u)) { sc[j].x = -INFINITY; sv[j].x = 0.f; zv[j].x = 0.f; }
      if (!((mask >> (bit + 1)) & 1u)) { sc[j].y = -INFINITY; sv[j].y = 0.f; zv[j].y = 0.f; }
    }
    mx = fmaxf(mx, fmaxf(sc[j].x, sc[j].y));
  }
  if (__any_sync(0xffffffffu, mx > st.m + kMaxAhead)) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(st.m, mx);
    const float f = ex2(st.m - m_new);
    st.l = __fmul2_rn(st.l, make_float2(f, f));
    st.zs = __fmul2_rn(st.zs, make_float2(f, f));
    rescale = f;
    st.m = m_new;
  }
  // w = p * S_V goes to the tensor cores as one fp16; the probability that enters the denominator and
  // the zero-point sum is that rounded w divided by the scale again, so numerator and denominator
  // see the same (slightly perturbed) probabilities and the rounding cancels where it matters most,
  // when a few tokens carry the whole softmax.
  {
    const float2 neg_m = make_float2(-st.m, -st.m), inv2 = make_float2(inv_sigma_e, inv_sigma_e);
#pragma unroll
    for (int j = 0; j < NP; ++j) {
      // The token's unit s_e = S_V / sigma_u * 2^EP is kept at or above 2^-10, so that w stays in fp16's normal
      // range whenever p matters: a constant V group (S_V = 0, all codes 0) and a token whose V scale lies
      // far below the slice's largest then enter the sums with their exact probability, and what the floor
      // adds to the output, at most p * 2^-22 sigma_u per code unit, is far below the tolerance.
      float2 s_e = __fmul2_rn(sv[j], inv2);
      s_e.x = fmaxf(s_e.x, 0x1p-10f); s_e.y = fmaxf(s_e.y, 0x1p-10f);
      const float2 rs = make_float2(rcp_approx(s_e.x), rcp_approx(s_e.y));
      const float2 arg = __fadd2_rn(sc[j], neg_m);
      const float2 w = __fmul2_rn(make_float2(ex2(arg.x), ex2(arg.y)), s_e);  // p * S_V / sigma_u * 2^EP
      pb[j] = pack_half2(w.x, w.y);
      const float2 p = __fmul2_rn(__half22float2(*reinterpret_cast<const __half2 *>(&pb[j])), rs);
      st.l = __fadd2_rn(st.l, p);
      st.zs = __ffma2_rn(p, zv[j], st.zs);
    }
  }
  return rescale;
}

// The accumulators of this lane hold heads 2tig and 2tig + 1 (columns): apply the heads' factors.
__device__ __forceinline__ void rescale_acc(float (&acc)[8][4], float f_of_my_head, int lane) {
  const int tig = lane & 3;
  const float f0 = __shfl_sync(0xffffffffu, f_of_my_head, (2 * tig) * 4);
  const float f1 = __shfl_sync(0xffffffffu, f_of_my_head, (2 * tig + 1) * 4);
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    acc[mt][0] *= f0; acc[mt][1] *= f1; acc[mt][2] *= f0; acc[mt][3] *= f1;
  }
}

// Last part of a step: O^T += V^T w for NT tiles, channels on M, tokens on K, heads on N.
template <int BITS, int NT>
__device__ __forceinline__ void pv_phase(const uint8_t *tile0, float (&acc)[8][4], const uint32_t (&pb)[2 * NT], int lane) {
  using F = Fmt<BITS>;
  constexpr int TB = tile_bytes(BITS);
  constexpr int CHUNKS = BITS / 2;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const uint8_t *vp = tile0 + nt * TB + v_part_offset(BITS) + lane * 16;
    uint32_t vw[2 * BITS];
#pragma unroll
    for (int q = 0; q < CHUNKS; ++q) {
      const uint4 a = ld_tile<BITS, uint4>(vp + q * 512);
      vw[4 * q] = a.x; vw[4 * q + 1] = a.y; vw[4 * q + 2] = a.z; vw[4 * q + 3] = a.w;
    }
    const uint32_t pb0 = pb[2 * nt], pb1 = pb[2 * nt + 1];
    if constexpr (BITS == 16) {
      const uint32_t ph0 = mul_half2(pb0, 32.f), ph1 = mul_half2(pb1, 32.f);
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        const uint32_t a0 = vw[2 * mt], a1 = vw[2 * mt + 1], a2 = vw[16 + 2 * mt], a3 = vw[16 + 2 * mt + 1];
        mma_f16(acc[mt], a0 & 0x00FF00FFu, a1 & 0x00FF00FFu, a2 & 0x00FF00FFu, a3 & 0x00FF00FFu, pb0, pb1);
        mma_f16(acc[mt], (a0 >> 5) & 0x07F807F8u, (a1 >> 5) & 0x07F807F8u, (a2 >> 5) & 0x07F807F8u,
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
          mma_f16(acc[(w * F::N) / 2 + jj], ea[2 * jj], ea[2 * jj + 1], eb[2 * jj], eb[2 * jj + 1], pb0, pb1);
      }
    }
  }
}

// Softmax and output of a step in one warp.
template <int BITS, int NT, bool MASKED>
__device__ __forceinline__ void softmax_pv_phase(const uint8_t *tile0, uint32_t mask, WarpState &st,
                                                 const float2 (&dot2)[2 * NT], float mu, float sumq, float inv_sigma_e,
                                                 int lane) {
  uint32_t pb[2 * NT];
  const float f = softmax_phase<BITS, NT, MASKED>(tile0, mask, st, dot2, mu, sumq, inv_sigma_e, lane, pb);
  if (__any_sync(0xffffffffu, f != 1.0f)) rescale_acc(st.acc, f, lane);
  pv_phase<BITS, NT>(tile0, st.acc, pb, lane);
}

// A whole step in one go (INT16 tiles, ragged ends).
template <int BITS, int NT, bool MASKED>
__device__ __forceinline__ void process_tiles(const uint8_t *tile0, uint32_t mask, WarpState &st, const QFrag &qa,
                                              float mu, float sumq, float inv_sigma_e, int lane) {
  float2 dot2[2 * NT];
  qk_phase<BITS, NT>(tile0, qa, lane, dot2);
  softmax_pv_phase<BITS, NT, MASKED>(tile0, mask, st, dot2, mu, sumq, inv_sigma_e, lane);
}

// ---- where the partials of a slice live ------------------------------------------------------
// Slice s covers units [s U, (s+1) U); the segment of CTA c in it publishes partial number (c - cta_origin) + s.
// A unit belongs to the CTA whose piece holds the unit's first fine unit (units_per_cta counts fine units).
__device__ __forceinline__ int unit_owner(const AttnParams &p, long long unit) {
  return (int)((p.line_origin + unit * p.unit_weight) / p.units_per_cta);
}
__device__ __forceinline__ void slice_ctas(const AttnParams &p, int slice, int &c_first, int &c_last) {
  const long long lo = (long long)slice * p.units_slice;
  c_first = unit_owner(p, lo + p.units_lead);  // a CTA that only touches the lead units has no segment
  c_last = unit_owner(p, lo + p.units_slice - 1);
}

// Log-sum-exp merge of the partials of one slice (all published).  Warp w merges head w;
// a lane owns 4 channels, and the weights of up to 32 partials at a time (one per lane).
__device__ __forceinline__ void combine_slice(const AttnParams &p, int slice) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = slice / p.kv_heads, hkv = slice % p.kv_heads;
  int cf, cl;
  slice_ctas(p, slice, cf, cl);
  const int n_parts = cl - cf + 1;
  const float *base = p.partials + (size_t)(cf - p.cta_origin + slice) * kMaxGroup * kPartialStride;
  for (int h = warp; h < p.group; h += kAttnWarps) {
    const float *ph = base + (size_t)h * kPartialStride;
    float M = kNegBig;
    for (int c = lane; c < n_parts; c += 32) M = fmaxf(M, __ldcg(ph + (size_t)c * kMaxGroup * kPartialStride));
#pragma unroll
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (int c0 = 0; c0 < n_parts; c0 += 32) {
      float w = 0.f;
      if (c0 + lane < n_parts) {
        const float2 ml = __ldcg(reinterpret_cast<const float2 *>(ph + (size_t)(c0 + lane) * kMaxGroup * kPartialStride));
        w = ex2(ml.x - M);
        den = fmaf(w, ml.y, den);
      }
      const int nb = min(32, n_parts - c0);
#pragma unroll 8
      for (int j = 0; j < nb; ++j) {
        const float wj = __shfl_sync(0xffffffffu, w, j);
        const float4 o4 = __ldcg(reinterpret_cast<const float4 *>(ph + (size_t)(c0 + j) * kMaxGroup * kPartialStride + 4) + lane);
        num.x = fmaf(wj, o4.x, num.x); num.y = fmaf(wj, o4.y, num.y);
        num.z = fmaf(wj, o4.z, num.z); num.w = fmaf(wj, o4.w, num.w);
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    const float inv = 1.0f / den;
    float4 *dst = reinterpret_cast<float4 *>(p.out + ((size_t)b * p.q_heads + hkv * p.group + h) * kHeadDim) + lane;
    *dst = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
  }
}

// Query fragment of head g for k-step s (channels 16 s .. 16 s + 15) at the code positions of width
// BITS, from Q'' in shared memory: {hi, lo} of channels (c0, c0 + 1) and of (c0 + 8, c0 + 9).
template <int BITS>
__device__ __forceinline__ uint4 q_fragment(const float (*s_q)[kHeadDim], int e_g, int g, int tig, int s) {
  using F = Fmt<BITS>;
  uint32_t r[4];
#pragma unroll
  for (int beta = 0; beta < 2; ++beta) {
    const int W = 2 * s + beta;
    const float scl = ldexpf(1.0f, F::EQ - F::pos(W % F::N) - e_g);
    const int c0 = 16 * s + 8 * beta + 2 * tig;
    const float x0 = s_q[g][c0] * scl, x1 = s_q[g][c0 + 1] * scl;
    const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
    const __half l0 = __float2half_rn(x0 - __half2float(h0)), l1 = __float2half_rn(x1 - __half2float(h1));
    const __half2 hi = __halves2half2(h0, h1), lo = __halves2half2(l0, l1);
    r[2 * beta] = *reinterpret_cast<const uint32_t *>(&hi);
    r[2 * beta + 1] = *reinterpret_cast<const uint32_t *>(&lo);
  }
  return make_uint4(r[0], r[1], r[2], r[3]);
}

// Fills the CTA's copy of the fragments at width BITS (all threads; a barrier must follow).
template <int BITS>
__device__ __forceinline__ void fill_q_fragments(uint4 *s_frag, const float (*s_q)[kHeadDim], const float *s_stat) {
  for (int i = threadIdx.x; i < 256; i += kAttnThreads) {  // entry (k-step i / 32, lane i % 32)
    const int l = i & 31, g = l >> 2;
    s_frag[i] = q_fragment<BITS>(s_q, (int)s_stat[g], g, l & 3, i >> 5);
  }
}

// ---- pieces of a segment that both contraction paths share --------------------------------------

// Q'' = Q * lambda * sm_scale * log2(e)  (Eq. 9: the equalization scale migrates into Q), per-head
// exponent of max |q''| and sum of q''.  Ends with a CTA-wide barrier.
__device__ __forceinline__ void build_query(const AttnParams &p, int b, int hkv, float (*s_q)[kHeadDim], float *s_stat) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < kMaxGroup * kHeadDim; i += kAttnThreads) {
    const int h = i >> 7, ch = i & 127;
    float v = 0.f;
    if (h < p.group) {
      const uint16_t raw = p.Q[((size_t)b * p.q_heads + hkv * p.group + h) * kHeadDim + ch];
      v = __fmul_rn(__fmul_rn(__uint_as_float((uint32_t)raw << 16), p.lambda[hkv * kHeadDim + ch]), p.qk_scale);
    }
    s_q[h][ch] = v;
  }
  __syncthreads();
  if (warp < kMaxGroup) {  // per-head max |q''| and sum q''
    const float4 v = *reinterpret_cast<const float4 *>(&s_q[warp][lane * 4]);
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
      s_stat[warp] = (float)e;
      s_stat[8 + warp] = sm;
    }
  }
  __syncthreads();
}

// unit of the V accumulators: a power of two >= every INT16 V scale of this slice
__device__ __forceinline__ float slice_sigma16(const AttnParams &p, int slice) {
  const float s16 = __uint_as_float(__ldcg(p.vmax_bits + slice));
  if (s16 > 0.f) {
    int e;
    frexpf(s16, &e);
    return ldexpf(1.0f, e);
  }
  return 1.0f;
}

// The INT16 tiles [a_lo, a_hi) of a slice (sink tiles, then the window ring), drawn from the shared
// counter s_ctr[0] by the warps of the CTA.
__device__ __forceinline__ void run_int16_tiles(const AttnParams &p, const uint8_t *slice_base, int a_lo, int a_hi,
                                                WarpState &st, const uint4 *s_frag, int *s_ctr, int e_g, float sumq,
                                                float sigma16, int lane) {
  using F16 = Fmt<16>;
  int it = a_lo + claim_next(s_ctr, lane);
  if (it >= a_hi) return;
  QFrag qa;
  qa.mine = s_frag + lane;
  const float mu = ldexpf(1.0f, 24 - F16::EQ + e_g);
  const float inv_sigma_e = ldexpf(1.0f, F16::EP) / sigma16;
  const int n_win = p.n_tokens - p.win_start;
  const int first_slot = n_win > 0 ? (p.win_start - p.geom.n_sink) % p.geom.ring_tokens : 0;
  do {
    uint32_t mask = 0;
    const uint8_t *tile;
    if (it < p.sink_tiles) {
      const int live = max(0, min(16, p.n_sink_eff - 16 * it));
      mask = (1u << live) - 1u;
      tile = slice_base + (size_t)it * tile_bytes(16);
    } else {
      const int rt = it - p.sink_tiles;
      tile = slice_base + p.geom.ring_off + (size_t)rt * tile_bytes(16);
      if (n_win > 0) {
        for (int r = 0; r < 16; ++r) {
          int d = rt * 16 + r - first_slot;
          if (d < 0) d += p.geom.ring_tokens;
          if (d < n_win) mask |= 1u << r;
        }
      }
    }
    if (mask == 0xFFFFu) process_tiles<16, 1, false>(tile, mask, st, qa, mu, sumq, inv_sigma_e, lane);
    else if (mask) process_tiles<16, 1, true>(tile, mask, st, qa, mu, sumq, inv_sigma_e, lane);
    it = a_lo + claim_next(s_ctr, lane);
  } while (it < a_hi);
}

// A warp's running state -> its partial (m, l, o[128]) per head in real units, slot `slot`.
// f_of(J) is the factor of accumulator column block J (channels 8 J + g).
template <class FactorOf>
__device__ __forceinline__ void store_warp_partial(const WarpState &st, FactorOf f_of, float (*s_o)[kMaxGroup][kHeadDim],
                                                   float *s_m, float *s_l, int slot, int lane) {
  const int g = lane >> 2, tig = lane & 3;
  float l_sum = st.l.x + st.l.y, zs_sum = st.zs.x + st.zs.y;
  l_sum += __shfl_xor_sync(0xffffffffu, l_sum, 1);
  l_sum += __shfl_xor_sync(0xffffffffu, l_sum, 2);
  zs_sum += __shfl_xor_sync(0xffffffffu, zs_sum, 1);
  zs_sum += __shfl_xor_sync(0xffffffffu, zs_sum, 2);
  if (tig == 0) {
    s_m[slot * 8 + g] = st.m;
    s_l[slot * 8 + g] = l_sum;
  }
  const float zs0 = __shfl_sync(0xffffffffu, zs_sum, (2 * tig) * 4);
  const float zs1 = __shfl_sync(0xffffffffu, zs_sum, (2 * tig + 1) * 4);
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const float f = f_of(2 * mt + rr);
      const int ch = 16 * mt + 8 * rr + g;
      s_o[slot][2 * tig][ch] = fmaf(st.acc[mt][2 * rr], f, zs0);
      s_o[slot][2 * tig + 1][ch] = fmaf(st.acc[mt][2 * rr + 1], f, zs1);
    }
  }
}

// Merges the segment's n_parts partials (all written, a CTA-wide barrier passed), publishes the segment's
// partial, and lets the CTA that publishes the slice's last partial merge the slice (nobody waits).
__device__ __forceinline__ void publish_segment(const AttnParams &p, int slice, int n_parts,
                                                const float (*s_o)[kMaxGroup][kHeadDim], const float *s_m, const float *s_l,
                                                int *s_ctr) {
  const int tid = threadIdx.x;
  float *part = p.partials + (size_t)((int)blockIdx.x - p.cta_origin + slice) * kMaxGroup * kPartialStride;
  for (int i = tid; i < p.group * kHeadDim; i += kAttnThreads) {
    const int h = i >> 7, ch = i & 127;
    float M = kNegBig;
    for (int w = 0; w < n_parts; ++w) M = fmaxf(M, s_m[w * 8 + h]);
    float o = 0.f, l = 0.f;
    for (int w = 0; w < n_parts; ++w) {
      const float wt = ex2(s_m[w * 8 + h] - M);
      o = fmaf(wt, s_o[w][h][ch], o);
      l = fmaf(wt, s_l[w * 8 + h], l);
    }
    __stcg(part + h * kPartialStride + 4 + ch, o);
    if (ch == 0) {
      __stcg(part + h * kPartialStride, M);
      __stcg(part + h * kPartialStride + 1, l);
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    int cf, cl;
    slice_ctas(p, slice, cf, cl);
    const unsigned t = atomicAdd(p.tickets + slice, 1u);
    s_ctr[2] = (t + 1u == (unsigned)(cl - cf + 1)) ? 1 : 0;
  }
  __syncthreads();
  if (s_ctr[2]) {
    __threadfence();
    combine_slice(p, slice);
    if (tid == 0) p.tickets[slice] = 0u;  // ready for the next launch (stream order)
  }
  __syncthreads();  // the segment's shared memory may be reused
}

// Ranges of a segment [u_lo, u_hi) (units relative to the slice): INT16 tiles [a_lo, a_hi) (a tile belongs to
// the segment that holds its first unit) and body tiles [t_lo, t_hi).
__device__ __forceinline__ void segment_ranges(const AttnParams &p, long long u_lo, long long u_hi, int &a_lo, int &a_hi,
                                               int &t_lo, int &t_hi) {
  a_lo = a_hi = t_lo = t_hi = 0;
  if (u_lo < p.units_aux) {
    a_lo = (int)((max(u_lo - p.units_lead, 0ll) + p.w16 - 1) / p.w16);
    a_hi = (int)((min(u_hi, p.units_aux) - p.units_lead + p.w16 - 1) / p.w16);
  }
  if (u_hi > p.units_aux) {
    t_lo = (int)(max(u_lo, p.units_aux) - p.units_aux);
    t_hi = (int)(u_hi - p.units_aux);
  }
}

// One segment on the warp-level MMA path: the part [u_lo, u_hi) (units relative to the slice) of one slice
// that this CTA owns.  Builds the slice's query, runs the INT16 tiles and then the body tiles (width
// BITS) of the range, merges the warps and publishes one partial per head.  The warps of the CTA draw
// work from two shared counters (INT16 tiles, then body steps of NT tiles), so they all finish together
// whatever share of the issue slots each of them gets.  `ring` is the CTA's dynamic shared memory: the
// per-warp cp.async stages while tiles stream, then the warps' outputs.
template <int BITS>
__device__ __forceinline__ void run_segment(const AttnParams &p, int slice, long long u_lo, long long u_hi,
                                            float (*s_q)[kHeadDim], float *s_stat, int *s_ctr, uint4 *s_frag,
                                            uint8_t *ring) {
  using F = Fmt<BITS>;
  using F16 = Fmt<16>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2;
  const int b = slice / p.kv_heads, hkv = slice % p.kv_heads;

  // (the previous segment ended with a CTA-wide barrier after its last use of s_q / s_stat / s_ctr / ring)
  if (tid == 0) s_ctr[0] = s_ctr[1] = 0;
  __syncthreads();
  int a_lo, a_hi, t_lo, t_hi;
  segment_ranges(p, u_lo, u_hi, a_lo, a_hi, t_lo, t_hi);
  const uint8_t *slice_base = p.geom.base + (size_t)slice * p.geom.slice_stride;

  // ---- body stream set-up: claim the first steps and start their copies before anything else ----
  constexpr int TB = tile_bytes(BITS);
  constexpr int NT = F::NT, S = F::SLOTS > 0 ? F::SLOTS : 1, SB = NT * TB;
  const uint8_t *body = slice_base + p.geom.body_off;
  const size_t stream_stride = p.geom.stream_stride;
  // A step is NT tiles.  With NT = 2 these are the tiles 16 G + s and 16 G + 8 + s: neighbours in stream s, one
  // contiguous run of 2 TB bytes (attention does not care about the order of the tokens).  The first and
  // the last group of 16 tiles of a segment may reach beyond [t_lo, t_hi): such tiles are left out.
  const int g_lo = t_lo >> 4;
  const int n_steps = t_hi <= t_lo ? 0 : (NT == 2 ? 8 * (((t_hi - 1) >> 4) - g_lo + 1) : t_hi - t_lo);
  auto step_tile = [&](int j, int k) { return NT == 2 ? 16 * (g_lo + (j >> 3)) + (j & 7) + 8 * k : t_lo + j; };
  auto live = [&](int t) { return t >= t_lo && t < t_hi; };
  uint8_t *my_ring = ring + (size_t)warp * S * SB;
  const uint32_t ring_addr = (uint32_t)__cvta_generic_to_shared(my_ring);
  auto claim = [&](int which) { return claim_next(s_ctr + which, lane); };
  auto issue = [&](int j, int slot) {
    constexpr int CPT = TB / 16;  // 16-byte chunks per tile: lane l copies chunks l, l + 32, ...
    const int ta = step_tile(j, 0);
    const uint8_t *src = body + body_tile_offset(ta, BITS, stream_stride) + lane * 16;
    const uint32_t dst = ring_addr + slot * SB + lane * 16;
    if (NT == 2 && (NT * CPT) % 32 == 0 && live(ta) && live(ta + 8)) {  // the whole step, every lane the same number of chunks
      cp_async_run<NT * CPT / 32>(dst, src);
    } else {
#pragma unroll
      for (int k = 0; k < NT; ++k) {
        if (live(step_tile(j, k))) {
          cp_async_run<CPT / 32>(dst + k * TB, src + k * TB);
          if (CPT % 32 != 0 && lane < CPT % 32) cp_async16_at<(CPT / 32) * 512>(dst + k * TB, src + k * TB);
        }
      }
    }
  };
  int pending[S];  // steps claimed and in flight, oldest first (>= n_steps: none)
  if constexpr (F::SLOTS > 0) {
#pragma unroll
    for (int i = 0; i < S - 1; ++i) {
      pending[i] = n_steps > 0 ? claim(1) : 0;
      if (pending[i] < n_steps) issue(pending[i], i);
      cp_async_commit();
    }
  }

  build_query(p, b, hkv, s_q, s_stat);
  const int e_g = (int)s_stat[g];
  const float sumq = s_stat[8 + g];
  fill_q_fragments<16>(s_frag, s_q, s_stat);
  if constexpr (BITS != 16) fill_q_fragments<BITS>(s_frag + 256, s_q, s_stat);
  __syncthreads();
  const float sigma16 = slice_sigma16(p, slice);

  WarpState st;
  st.m = kNegBig; st.l = make_float2(0.f, 0.f); st.zs = make_float2(0.f, 0.f);
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) st.acc[mt][0] = st.acc[mt][1] = st.acc[mt][2] = st.acc[mt][3] = 0.f;

  // ---- INT16 tiles (sink + window ring) ----
  if (a_hi > a_lo) {
    run_int16_tiles(p, slice_base, a_lo, a_hi, st, s_frag, s_ctr, e_g, sumq, sigma16, lane);
    if constexpr (BITS != 16) {
      // accumulator units change with the width: INT16 units -> body units (exact powers of two)
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          const float f = ldexpf(1.0f, F::EP - F16::EP + F::pos((2 * mt + rr) % F::N) - F::SIGMA_LOG2);
          st.acc[mt][2 * rr] *= f;
          st.acc[mt][2 * rr + 1] *= f;
        }
      }
    }
  }

  // ---- body tiles ----
  const float sigma_u = sigma16 * ldexpf(1.0f, F::SIGMA_LOG2);
  if (n_steps > 0) {
    QFrag qa;
    qa.mine = (BITS != 16 ? s_frag + 256 : s_frag) + lane;
    const float mu = ldexpf(1.0f, 24 - F::EQ + e_g);
    const float inv_sigma_e = ldexpf(1.0f, F::EP) / sigma_u;
    const uint32_t tail_mask = (p.n_body & 15) ? (1u << (p.n_body & 15)) - 1u : 0xFFFFu;
    const int tail_tile = tail_mask != 0xFFFFu ? p.body_tiles - 1 : -1;  // the one tile with dead rows
    if constexpr (F::SLOTS == 0) {
      for (int t = t_lo + claim(1); t < t_hi; t = t_lo + claim(1)) {
        const uint8_t *tile = body + body_tile_offset(t, BITS, stream_stride);
        if (t == tail_tile) process_tiles<BITS, 1, true>(tile, tail_mask, st, qa, mu, sumq, inv_sigma_e, lane);
        else process_tiles<BITS, 1, false>(tile, 0xFFFFu, st, qa, mu, sumq, inv_sigma_e, lane);
      }
    } else {
      int slot = 0, fill = S - 1;
      while (pending[0] < n_steps) {
        const int nxt = claim(1);
        if (nxt < n_steps) issue(nxt, fill);
        cp_async_commit();
        cp_async_wait<S - 1>();
        __syncwarp();
        const uint8_t *tile = my_ring + slot * SB;
        const int t = step_tile(pending[0], 0);
        if (NT == 2 && live(t) && live(t + 8) && t != tail_tile && t + 8 != tail_tile) {
          process_tiles<BITS, NT, false>(tile, 0xFFFFu, st, qa, mu, sumq, inv_sigma_e, lane);
        } else {
#pragma unroll
          for (int k = 0; k < NT; ++k) {
            const int tk = step_tile(pending[0], k);
            if (!live(tk)) continue;
            if (tk == tail_tile)
              process_tiles<BITS, 1, true>(tile + k * TB, tail_mask, st, qa, mu, sumq, inv_sigma_e, lane);
            else
              process_tiles<BITS, 1, false>(tile + k * TB, 0xFFFFu, st, qa, mu, sumq, inv_sigma_e, lane);
          }
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i + 2 < S; ++i) pending[i] = pending[i + 1];
        pending[S - 2] = nxt;
        fill = slot;
        slot = (slot + 1 == S) ? 0 : slot + 1;
      }
    }
  }
  if constexpr (F::SLOTS > 0) cp_async_wait<0>();

  // ---- warp epilogue: quad sums, real units, to shared memory (the ring is free now) ----
  __syncthreads();  // every warp is done with its stages
  float(*s_o)[kMaxGroup][kHeadDim] = reinterpret_cast<float(*)[kMaxGroup][kHeadDim]>(ring);
  float *s_m = s_stat + 16, *s_l = s_stat + 16 + kParts * kMaxGroup;
  store_warp_partial(st, [&](int J) { return ldexpf(sigma_u, 24 - F::EP - F::pos(J % F::N)); }, s_o, s_m, s_l, warp, lane);
  __syncthreads();
  publish_segment(p, slice, kAttnWarps, s_o, s_m, s_l, s_ctr);
}

}  // namespace pmkvq
#include "kernels_attn_tc.cuh"
namespace pmkvq {

// Dynamic shared memory of a CTA that may run the tensor-memory path.
constexpr int kSmemStages = kStages * kStageBytes;
constexpr int kSmemQOperand = kSmemStages;
constexpr int kSmemWBuf = kSmemQOperand + kQOperandBytes;
constexpr int kSmemParts = kSmemWBuf + kTcGroups * kWBufBytes;
constexpr int kSmemTcTotal = kSmemParts + kParts * kMaxGroup * kHeadDim * 4;

// One segment with a 4- or 2-bit body.  The INT16 tiles run as above, on the warps' own accumulators, and
// every warp parks its partial in shared memory; the body then runs through the tensor-memory pipeline
// and leaves one more partial.
template <int BITS>
__device__ __forceinline__ void run_segment_tc(const AttnParams &p, int slice, long long u_lo, long long u_hi,
                                               float (*s_q)[kHeadDim], float *s_stat, int *s_ctr, uint4 *s_frag,
                                               TcCtx &tc) {
  using F16 = Fmt<16>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2;
  const int b = slice / p.kv_heads, hkv = slice % p.kv_heads;
  if (tid == 0) s_ctr[0] = s_ctr[1] = 0;
  __syncthreads();
  int a_lo, a_hi, t_lo, t_hi;
  segment_ranges(p, u_lo, u_hi, a_lo, a_hi, t_lo, t_hi);
  const uint8_t *slice_base = p.geom.base + (size_t)slice * p.geom.slice_stride;

  build_query(p, b, hkv, s_q, s_stat);
  if (a_hi > a_lo) fill_q_fragments<16>(s_frag, s_q, s_stat);
  if (t_hi > t_lo) {
    fill_q_operand<BITS>(tc.q_operand, s_q, s_stat);
    tc05::fence_async_smem();
  }
  __syncthreads();
  const float sigma16 = slice_sigma16(p, slice);
  float(*s_o)[kMaxGroup][kHeadDim] = reinterpret_cast<float(*)[kMaxGroup][kHeadDim]>(tc.part_o);
  float *s_m = s_stat + 16, *s_l = s_stat + 16 + kParts * kMaxGroup;

  if (warp < kAttnWarps) {
    WarpState st;
    st.m = kNegBig; st.l = make_float2(0.f, 0.f); st.zs = make_float2(0.f, 0.f);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) st.acc[mt][0] = st.acc[mt][1] = st.acc[mt][2] = st.acc[mt][3] = 0.f;
    if (a_hi > a_lo) run_int16_tiles(p, slice_base, a_lo, a_hi, st, s_frag, s_ctr, (int)s_stat[g], s_stat[8 + g], sigma16, lane);
    store_warp_partial(st, [&](int J) { return ldexpf(sigma16, 24 - F16::EP - F16::pos(J % F16::N)); }, s_o, s_m, s_l, warp, lane);
  }
  if (t_hi > t_lo) {
    tc_body<BITS>(p, tc, slice_base + p.geom.body_off, t_lo, t_hi, s_stat, sigma16, s_m, s_l, kAttnWarps);
  } else if (tid < kTcGroups * kHeadDim) {
    const int slot = kAttnWarps + (tid >> 7), c = tid & 127;
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) s_o[slot][h][c] = 0.f;
    if (c < kMaxGroup) { s_m[slot * 8 + c] = kNegBig; s_l[slot * 8 + c] = 0.f; }
  }
  __syncthreads();
  publish_segment(p, slice, kParts, s_o, s_m, s_l, s_ctr);
}

// Dynamic shared memory of the warp-level MMA path at body width BITS: per-warp stages while streaming;
// at least the warps' outputs they are reused for.
template <int BITS>
constexpr int attn_ring_bytes() {
  constexpr int out_bytes = kAttnWarps * kMaxGroup * kHeadDim * 4;
  constexpr int ring = kAttnWarps * Fmt<BITS>::SLOTS * Fmt<BITS>::NT * tile_bytes(BITS);
  return ring > out_bytes ? ring : out_bytes;
}
// ... of the one-block kernel on either path
template <int BITS, bool ROWS>
constexpr int attn_smem_bytes() {
  if constexpr (BITS <= 4 && ROWS) return kSmemTcTotal;
  else return attn_ring_bytes<BITS>();
}

// CTA set-up of the tensor-memory path: barriers and tensor memory.  Ends with a CTA-wide barrier.
__device__ __forceinline__ void tc_setup(TcShared *sh, TcCtx &tc, uint8_t *ring, unsigned *error_word) {
  const int tid = threadIdx.x, warp = tid >> 5;
  tc.sh = sh;
  tc.stages = ring;
  tc.q_operand = ring + kSmemQOperand;
  tc.wbuf = ring + kSmemWBuf;
  tc.part_o = reinterpret_cast<float *>(ring + kSmemParts);
  tc.error_word = error_word;
  tc.gi = 0; tc.gc = 0;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      tc05::mbar_init(tc05::smem_u32(&sh->full[s]), 1);
      tc05::mbar_init(tc05::smem_u32(&sh->stage_free[s]), 4);
    }
    for (int b = 0; b < kTcGroups; ++b) {
      tc05::mbar_init(tc05::smem_u32(&sh->ak_full[b]), 4);
      tc05::mbar_init(tc05::smem_u32(&sh->av_full[b]), 4);
      tc05::mbar_init(tc05::smem_u32(&sh->w_full[b]), 4);
      tc05::mbar_init(tc05::smem_u32(&sh->bar_s[b]), 1);
      tc05::mbar_init(tc05::smem_u32(&sh->bar_o[b]), 1);
      sh->pv_fresh[b] = 1;
    }
    sh->abort = 0;
    tc05::mbar_init_fence();
  }
  if (warp == 0) tc05::tmem_alloc(tc05::smem_u32(&sh->tmem_base), kTmemCols);
  tc05::fence_before_sync();
  __syncthreads();
  tc05::fence_after_sync();
  tc.tmem_base = sh->tmem_base;
}
__device__ __forceinline__ void tc_teardown(TcCtx &tc) {
  tc05::fence_before_sync();
  __syncthreads();
  if (*reinterpret_cast<volatile int *>(&tc.sh->abort)) {
    // a wait gave up: copies into this CTA's shared memory may still be in flight; give them about a
    // millisecond (a bounded delay) to land before the CTA goes away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) {}
    __syncthreads();
  }
  if ((threadIdx.x >> 5) == 0) tc05::tmem_dealloc(tc.tmem_base, kTmemCols);
}

template <int BODY_BITS, bool ROWS>
__global__ void __launch_bounds__(kAttnThreads, 1) decode_attn_splitk_kernel(const AttnParams p, unsigned *error_word) {
  __shared__ __align__(16) float s_q[kMaxGroup][kHeadDim];
  __shared__ float s_stat[16 + 2 * kParts * kMaxGroup];  // head stats, per-partial (m, l)
  __shared__ int s_ctr[4];                                // work counters (INT16 tiles, body tiles), combine flag
  __shared__ uint4 s_frag[512];                           // query fragments at INT16 and at the body width
  __shared__ TcShared s_tc;
  extern __shared__ __align__(128) uint8_t ring[];
  TcCtx tc;
  constexpr bool tensor_path = BODY_BITS <= 4 && ROWS;
  if constexpr (tensor_path) tc_setup(&s_tc, tc, ring, error_word);
  const long long u_begin = (long long)blockIdx.x * p.units_per_cta;
  const long long u_end = min(u_begin + p.units_per_cta, p.units_total);
  for (long long u = u_begin; u < u_end;) {
    const int slice = (int)(u / p.units_slice);
    const long long base = (long long)slice * p.units_slice;
    const long long hi = min(u_end - base, p.units_slice);
    if (hi > p.units_lead) {
      if constexpr (tensor_path) run_segment_tc<BODY_BITS>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, tc);
      else run_segment<BODY_BITS>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, ring);
    }
    u = base + hi;
  }
  if constexpr (tensor_path) tc_teardown(tc);
}

// ---------------------------------------------------------------------------------------------
// All blocks of a decode step in one launch.  The blocks' units are strung together on one line (a
// tile of a wider block weighs more fine units, in proportion to the time it takes) and the line is
// cut into one piece per CTA, so launch ramp, tail and most segment set-ups are paid once per step
// instead of once per block.  Per-block quantities are derived on the device from the block's token
// count and width; geometry comes from the table the cache keeps in device memory.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxFusedLayers = 128;
struct FusedParams {
  const LayerGeom *geoms;     // [layers]
  const uint16_t *Q;          // bf16 [layers][batch][q_heads][128]
  const float *lambda;        // [layers][kv_heads][128]
  const unsigned *vmax_bits;  // [layers][n_slices]
  float *partials;            // per block, partial_stride floats apart
  float *out;                 // fp32 [layers][batch][q_heads][128]
  unsigned *tickets;          // [layers][n_slices]
  unsigned *error_word;       // bits set by a wait that ran out
  size_t partial_stride;
  int layers, kv_heads, group, q_heads, n_slices, batch;
  int n_sink, window, evict_chunk, sink_tiles, ring_tiles;
  int rows;                   // 1: tensor-memory path (row tiles at 4 and 2 bit)
  float qk_scale;
  long long per_cta, total;              // fine units
  long long start[kMaxFusedLayers + 1];  // fine units before each block
  int n_tokens[kMaxFusedLayers];
  unsigned char bits[kMaxFusedLayers], lead[kMaxFusedLayers], weight[kMaxFusedLayers];
};

__device__ __forceinline__ void fused_layer_params(const FusedParams &fp, int l, AttnParams &p) {
  const int n = fp.n_tokens[l], bits = fp.bits[l];
  p.geom = fp.geoms[l];
  p.Q = fp.Q + (size_t)l * fp.batch * fp.q_heads * kHeadDim;
  p.lambda = fp.lambda + (size_t)l * fp.kv_heads * kHeadDim;
  p.vmax_bits = fp.vmax_bits + (size_t)l * fp.n_slices;
  p.partials = fp.partials + (size_t)l * fp.partial_stride;
  p.out = fp.out + (size_t)l * fp.batch * fp.q_heads * kHeadDim;
  p.tickets = fp.tickets + (size_t)l * fp.n_slices;
  p.kv_heads = fp.kv_heads; p.group = fp.group; p.q_heads = fp.q_heads; p.n_slices = fp.n_slices;
  p.n_tokens = n;
  p.n_sink_eff = min(n, fp.n_sink);
  const int excess = n - fp.n_sink - fp.window;
  p.n_body = excess <= 0 ? 0 : excess / fp.evict_chunk * fp.evict_chunk;
  p.win_start = p.n_sink_eff + p.n_body;
  p.cur_bits = bits;
  p.body_tiles = (p.n_body + 15) / 16;
  p.sink_tiles = fp.sink_tiles;
  p.aux_tiles = fp.sink_tiles + fp.ring_tiles;
  p.w16 = (tile_bytes(16) + tile_bytes(bits) - 1) / tile_bytes(bits);
  p.units_lead = fp.lead[l];
  p.units_aux = p.units_lead + (long long)p.aux_tiles * p.w16;
  p.units_slice = p.units_aux + p.body_tiles;
  p.units_total = p.units_slice * fp.n_slices;
  p.units_per_cta = fp.per_cta;
  p.line_origin = fp.start[l];
  p.unit_weight = fp.weight[l];
  p.cta_origin = (int)(fp.start[l] / fp.per_cta);
  p.qk_scale = fp.qk_scale;
}

template <bool ROWS>
__global__ void __launch_bounds__(kAttnThreads, 1) decode_attn_fused_kernel(const __grid_constant__ FusedParams fp) {
  __shared__ __align__(16) float s_q[kMaxGroup][kHeadDim];
  __shared__ float s_stat[16 + 2 * kParts * kMaxGroup];
  __shared__ int s_ctr[4];
  __shared__ uint4 s_frag[512];
  __shared__ TcShared s_tc;
  extern __shared__ __align__(128) uint8_t ring[];
  TcCtx tc;
  constexpr bool tensor_path = ROWS;  // the cache was created for the tensor-memory path
  if constexpr (tensor_path) tc_setup(&s_tc, tc, ring, fp.error_word);
  const long long f_begin = (long long)blockIdx.x * fp.per_cta;
  const long long f_end = min(f_begin + fp.per_cta, fp.total);
  int l = 0;
  for (long long f = f_begin; f < f_end;) {
    while (l + 1 < fp.layers && fp.start[l + 1] <= f) ++l;  // the block this fine unit belongs to
    AttnParams p;
    fused_layer_params(fp, l, p);
    const long long f_hi = min(f_end, fp.start[l + 1]);
    // units of this block whose first fine unit lies in [f, f_hi)
    const int w = p.unit_weight;
    long long u = (f - p.line_origin + w - 1) / w;
    const long long u_end = (f_hi - p.line_origin + w - 1) / w;
    while (u < u_end) {
      const int slice = (int)(u / p.units_slice);
      const long long base = (long long)slice * p.units_slice;
      const long long hi = min(u_end - base, p.units_slice);
      if (hi > p.units_lead) {
        switch (p.cur_bits) {
          case 16: run_segment<16>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, ring); break;
          case 8: run_segment<8>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, ring); break;
          case 4:
            if constexpr (tensor_path) run_segment_tc<4>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, tc);
            else run_segment<4>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, ring);
            break;
          default:
            if constexpr (tensor_path) run_segment_tc<2>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, tc);
            else run_segment<2>(p, slice, u - base, hi, s_q, s_stat, s_ctr, s_frag, ring);
            break;
        }
      }
      u = base + hi;
    }
    f = f_hi;
  }
  if constexpr (tensor_path) tc_teardown(tc);
}

template <bool ROWS>
constexpr int attn_fused_smem_bytes() {
  int m = ROWS ? kSmemTcTotal : 0;
  m = attn_ring_bytes<16>() > m ? attn_ring_bytes<16>() : m;
  m = attn_ring_bytes<8>() > m ? attn_ring_bytes<8>() : m;
  m = attn_ring_bytes<4>() > m ? attn_ring_bytes<4>() : m;
  m = attn_ring_bytes<2>() > m ? attn_ring_bytes<2>() : m;
  return m;
}

}  // namespace pmkvq

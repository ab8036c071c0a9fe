// Cache-maintenance kernels: quantize-on-append (Eq. 1-2 at 16 bit, Keys equalized per Eq. 9),
// window eviction and the progressive reduce (Eq. 3).  All integer / IEEE-fp32 work is written
// with explicit round-to-nearest intrinsics so that codes, scales and zero-points have exactly
// one bit pattern.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "layout.cuh"

namespace pmkvq {

// Where one block's slices live inside the arena.
struct LayerGeom {
  uint8_t *base;        // first slice of this block
  size_t slice_stride;  // bytes between (batch, kv_head) slices
  size_t ring_off;      // byte offset of the INT16 window ring inside a slice
  size_t body_off;      // byte offset of the body inside a slice
  size_t stream_stride; // bytes between the eight interleaved streams of the body
  int n_sink;           // leading INT16 tokens (stored in tiles at offset 0)
  int ring_tokens;      // ring capacity in tokens (multiple of 16)
  int shift_variant;    // ShiftVariant of this cache
  int rows;             // 1: the 4- and 2-bit body uses row tiles (tensor-memory attention path)
};

struct TokenDest {
  uint8_t *tile;
  int row;
  int bits;
};

// Tile, row and width of absolute token t, given the first window token `win_start`
// (= n_sink + n_body) and the body width.
__device__ __forceinline__ TokenDest token_dest(const LayerGeom &g, uint8_t *slice, int t, int win_start,
                                                int cur_bits) {
  TokenDest d;
  if (t < g.n_sink) {
    d.tile = slice + (size_t)(t >> 4) * tile_bytes(16);
    d.row = t & 15;
    d.bits = 16;
  } else if (t < win_start) {
    const int j = t - g.n_sink;
    d.tile = slice + g.body_off + body_tile_offset(j >> 4, cur_bits, g.stream_stride);
    d.row = j & 15;
    d.bits = cur_bits;
  } else {
    const int rp = (t - g.n_sink) % g.ring_tokens;
    d.tile = slice + g.ring_off + (size_t)(rp >> 4) * tile_bytes(16);
    d.row = rp & 15;
    d.bits = 16;
  }
  return d;
}

// Scale after the chain 16 -> ... -> bits: S_b = (2^b + 1) S_2b, one fp32 rounding per step (Sec. 3.1).
__device__ __forceinline__ float chain_scale(float s16, int bits, int variant = kShiftEquivalent) {
  float s = s16;
  for (int w = 8; w >= bits; w >>= 1) s = __fmul_rn(s, (float)((1 << w) + (variant == kShiftModified ? 0 : 1)));
  return s;
}
// One halving of the metadata of one token: (S_2b, Z_2b) -> (S_b, Z_b), each step one fp32 rounding.
__device__ __forceinline__ void halve_meta(float &s, float &z, int b, int variant) {
  if (variant == kShiftModified) {
    const float sb = __fmul_rn(s, (float)(1 << b));
    z = __fadd_rn(z, __fmul_rn(__fsub_rn(sb, s), 0.5f));
    s = sb;
  } else {
    s = __fmul_rn(s, (float)((1 << b) + 1));
  }
}
// Zero-point after the chain 16 -> ... -> bits (it only moves under the modified right shift).
__device__ __forceinline__ float chain_zero(float z16, float s16, int bits, int variant) {
  float s = s16, z = z16;
  if (variant == kShiftModified)
    for (int w = 8; w >= bits; w >>= 1) halve_meta(s, z, w, variant);
  return z;
}

// Write one token's 128 codes (given as INT16 codes in shared memory) into a tile at `bits`,
// applying the Eq. 3 chain; one warp, every half-word of the token is written by one lane.
template <int BITS>
__device__ __forceinline__ void store_token_w(uint8_t *part, int row, const uint16_t *codes16, int is_value, int lane,
                                              int variant) {
  constexpr int bits = BITS;  // a compile-time width turns the index arithmetic below into shifts
  constexpr int n = 16 / bits;
  const int r = row >> 3;
  for (int hw = lane; hw < 8 * bits; hw += 32) {
    const int w = hw >> 3, sub = hw & 7;
    int owner, h, chan0, chan_step = 8;
    if (is_value) {  // sub = g ; channels 8*J + g
      h = row & 1;
      owner = sub * 4 + ((row & 7) >> 1);
      chan0 = sub;
    } else {  // sub = tig + 4*h ; channels 8*W + 2*tig + h
      const int tig = sub & 3;
      h = sub >> 2;
      owner = (row & 7) * 4 + tig;
      chan0 = 2 * tig + h;
    }
    uint32_t val = 0;
    for (int j = 0; j < n; ++j) {
      const int ch = chan_step * (w * n + j) + chan0;
      val |= shift_chain(codes16[ch], bits, variant) << (j * bits);
    }
    int byte_off, bit_off;
    lane_slot(bits, owner, r, w * n, h, byte_off, bit_off);
    *reinterpret_cast<uint16_t *>(part + byte_off) = (uint16_t)val;
  }
}

// Row tiles (4 and 2 bit), K part: the token's 16*BITS bytes are its own; lane w builds word w.
template <int BITS>
__device__ __forceinline__ void store_key_row(uint8_t *k_part, int row, const uint16_t *codes16, int lane, int variant) {
  constexpr int per_word = 32 / BITS, n_words = 4 * BITS;
  if (lane < n_words) {
    uint32_t val = 0;
#pragma unroll
    for (int i = 0; i < per_word; ++i)
      val |= shift_chain(codes16[per_word * lane + i], BITS, variant) << (16 * (i & 1) + BITS * (i >> 1));
    *reinterpret_cast<uint32_t *>(k_part + row * 16 * BITS + 4 * lane) = val;
  }
}
// Row tiles, V part: a half-word of a channel's row holds the codes of 16/BITS tokens, so a token is
// inserted by read-modify-write; lane l handles channels l, l+32, l+64, l+96.  Only ONE warp at a time may
// insert tokens into a given tile (the callers below let the first token of a tile do the tile's others).
template <int BITS>
__device__ __forceinline__ void insert_value_row(uint8_t *v_part, int row, const uint16_t *codes16, int lane, int variant) {
  int bo, sh;
  row_slot(BITS, row, bo, sh);
  constexpr uint32_t mask = (1u << BITS) - 1u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int ch = lane + 32 * j;
    uint16_t *hw = reinterpret_cast<uint16_t *>(v_part + ch * 2 * BITS + bo);
    const uint32_t v = *hw;
    *hw = (uint16_t)((v & ~(mask << sh)) | (shift_chain(codes16[ch], BITS, variant) << sh));
  }
}

__device__ __forceinline__ void store_token(uint8_t *part, int bits, int row, const uint16_t *codes16, int is_value,
                                            int lane, int variant, bool rows) {
  switch (bits) {
    case 16: store_token_w<16>(part, row, codes16, is_value, lane, variant); break;
    case 8: store_token_w<8>(part, row, codes16, is_value, lane, variant); break;
    case 4:
      if (!rows) store_token_w<4>(part, row, codes16, is_value, lane, variant);
      else if (is_value) insert_value_row<4>(part, row, codes16, lane, variant);
      else store_key_row<4>(part, row, codes16, lane, variant);
      break;
    default:
      if (!rows) store_token_w<2>(part, row, codes16, is_value, lane, variant);
      else if (is_value) insert_value_row<2>(part, row, codes16, lane, variant);
      else store_key_row<2>(part, row, codes16, lane, variant);
      break;
  }
}

// Read one token's INT16 codes from a 16-bit tile into shared memory; one warp.
__device__ __forceinline__ void load_token16(const uint8_t *part, int row, uint16_t *codes16, int is_value, int lane) {
  for (int ch = lane; ch < kHeadDim; ch += 32) {
    int byte_off, bit_off;
    if (is_value) v_slot(16, false, row, ch, byte_off, bit_off);
    else k_slot(16, false, row, ch, byte_off, bit_off);
    codes16[ch] = *reinterpret_cast<const uint16_t *>(part + byte_off);
  }
}

// ---------------------------------------------------------------------------------------------
// Quantize-on-append.  One warp per (new token, slice, K|V).  Eq. 1-2 with b = 16 on the 128
// channels of the token; Keys are first multiplied by Lambda^-1 (Eq. 9).  The token goes to the
// sink, straight to the body (bulk appends; Eq. 3 chain to the body width) or to the window ring.
// ---------------------------------------------------------------------------------------------
// RN(d / s), the correctly rounded fp32 quotient, for 0 <= d and a scale in [2^-60, 2^60], from the
// correctly rounded reciprocal y = RN(1 / s) that a token computes once.  q0 = RN(d y) is within two units
// in the last place; the residual d - q s is exact in one fused multiply-add (no underflow in this range
// unless the quotient is below 2^-20, where any result still rounds to code 0), so the first correction
// gives a faithful quotient and the second, by Markstein's theorem on correcting a faithful quotient with a
// correctly rounded reciprocal, the correctly rounded one.  5 instructions against the ~15 of a division.
__device__ __forceinline__ float quotient_rn(float d, float s, float y) {
  float q = __fmul_rn(d, y);
  float r = __fmaf_rn(-q, s, d);
  q = __fmaf_rn(r, y, q);
  r = __fmaf_rn(-q, s, d);
  return __fmaf_rn(r, y, q);
}
// round-half-to-even of a quotient: adding 2^23 leaves the rounded integer in the low mantissa bits.  No
// clamp is needed: d <= max - min and S = RN((max - min) / 65535) >= (max - min) / 65535 (1 - 2^-24) bound
// the correctly rounded quotient by 65535 (1 + 2^-23), which is below 65535.5.
__device__ __forceinline__ int code_of_quotient(float q) {
  return __float_as_int(__fadd_rn(q, 8388608.0f)) - 0x4B000000;
}

// Eq. 1-2 at 16 bit on one token's 128 channels (Keys first times Lambda^-1, Eq. 9), by one warp: lane l
// holds channels 4l..4l+3.  Writes the codes to `codes` (shared memory) and returns S; Z goes to `zero`.
__device__ __forceinline__ float quantize_token16(uint2 raw, const float *__restrict__ inv_lambda_head, uint16_t *codes,
                                                  int lane, float &zero);
__device__ __forceinline__ float quantize_token16(const uint16_t *__restrict__ src, const float *__restrict__ inv_lambda_head,
                                                  uint16_t *codes, int lane, float &zero) {
  return quantize_token16(*reinterpret_cast<const uint2 *>(src + lane * 4), inv_lambda_head, codes, lane, zero);
}
__device__ __forceinline__ float quantize_token16(uint2 raw, const float *__restrict__ inv_lambda_head, uint16_t *codes,
                                                  int lane, float &zero) {
  float x[4];
  x[0] = __uint_as_float(raw.x << 16);
  x[1] = __uint_as_float(raw.x & 0xFFFF0000u);
  x[2] = __uint_as_float(raw.y << 16);
  x[3] = __uint_as_float(raw.y & 0xFFFF0000u);
  if (inv_lambda_head) {
    const float4 il = *reinterpret_cast<const float4 *>(inv_lambda_head + lane * 4);
    x[0] = __fmul_rn(x[0], il.x);
    x[1] = __fmul_rn(x[1], il.y);
    x[2] = __fmul_rn(x[2], il.z);
    x[3] = __fmul_rn(x[3], il.w);
  }
  float mn = fminf(fminf(x[0], x[1]), fminf(x[2], x[3]));
  float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  const float scale = __fdiv_rn(__fsub_rn(mx, mn), 65535.0f);
  if (scale >= 0x1p-60f && scale <= 0x1p60f) {  // one scale per token: the branch is uniform in the warp
    const float y = __frcp_rn(scale);
#pragma unroll
    for (int e = 0; e < 4; ++e) codes[lane * 4 + e] = (uint16_t)code_of_quotient(quotient_rn(__fsub_rn(x[e], mn), scale, y));
  } else {  // constant tokens (0 / 0 converts to code 0) and scales far outside any real tensor's range
#pragma unroll
    for (int e = 0; e < 4; ++e)
      codes[lane * 4 + e] = (uint16_t)min(max(__float2int_rn(__fdiv_rn(__fsub_rn(x[e], mn), scale)), 0), 65535);
  }
  zero = mn;
  return scale;
}

// Writes the metadata of one stored token (S, Z of K or of V after the chain to `bits`).
__device__ __forceinline__ void store_meta(uint8_t *tile, int bits, int row, int is_value, float s16, float z16, int variant,
                                           bool rows) {
  float *meta = reinterpret_cast<float *>(tile + meta_offset(bits));
  meta[meta_slot(bits, rows, is_value ? 2 : 0, row) >> 2] = chain_scale(s16, bits, variant);
  meta[meta_slot(bits, rows, is_value ? 3 : 1, row) >> 2] = chain_zero(z16, s16, bits, variant);
}

// One warp per (new token, slice, K|V) of the new tokens i0 .. i0 + n_cnt - 1.  Values that go straight
// into a row tile of the body (4 and 2 bit) are inserted by read-modify-write of half-words that the
// tile's tokens share, so the first such token of a tile inside the launch's range does the tile's
// other tokens of the range too, one after the other, and their own warps leave.
__device__ __forceinline__ void append_one(long long wid, uint16_t *codes, int lane, const uint16_t *__restrict__ K,
                                           const uint16_t *__restrict__ V, const float *__restrict__ inv_lambda,
                                           unsigned *vmax_bits, const LayerGeom &geom, int n_slices, int kv_heads,
                                           int n_old, int win_start, int cur_bits, int i0 = 0, int n_cnt = 1) {
  const int is_value = (int)(wid & 1);
  const long long ts = wid >> 1;
  const int slice = (int)(ts % n_slices);
  int i = i0 + (int)(ts / n_slices);  // index among the new tokens
  uint8_t *slice_base = geom.base + (size_t)slice * geom.slice_stride;
  int t = n_old + i, last = t;
  const bool shared_rows = is_value && t >= geom.n_sink && t < win_start && row_layout(cur_bits, geom.rows != 0);
  if (shared_rows) {
    const int j = t - geom.n_sink;
    if (i != i0 && (j & 15) != 0) return;  // an earlier token of this tile does this one
    last = min(min(n_old + i0 + n_cnt, win_start), geom.n_sink + (j | 15) + 1) - 1;
  }
  for (; t <= last; ++t, ++i) {
    const uint16_t *src = (is_value ? V : K) + ((size_t)i * n_slices + slice) * kHeadDim;
    float mn;
    const float scale = quantize_token16(src, is_value ? nullptr : inv_lambda + (size_t)(slice % kv_heads) * kHeadDim,
                                         codes, lane, mn);
    __syncwarp();
    const TokenDest d = token_dest(geom, slice_base, t, win_start, cur_bits);
    store_token(d.tile + (is_value ? v_part_offset(d.bits) : 0), d.bits, d.row, codes, is_value, lane, geom.shift_variant,
                geom.rows != 0);
    if (lane == 0) {
      store_meta(d.tile, d.bits, d.row, is_value, scale, mn, geom.shift_variant, geom.rows != 0);
      if (is_value) atomicMax(vmax_bits + slice, __float_as_uint(scale));  // scale >= 0: uint order = float order
    }
    __syncwarp();
  }
}

__global__ void __launch_bounds__(128) append_kernel(const uint16_t *__restrict__ K, const uint16_t *__restrict__ V,
                                                     const float *__restrict__ inv_lambda, unsigned *vmax_bits,
                                                     LayerGeom geom, int n_new, int n_slices, int kv_heads,
                                                     int n_old, int win_start, int cur_bits, int i0) {
  // new tokens i0 .. i0 + n_new - 1 of the K / V arrays, one by one
  __shared__ uint16_t s_codes[4][kHeadDim];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wid = (long long)blockIdx.x * 4 + warp;
  if (wid >= (long long)n_new * n_slices * 2) return;
  append_one(wid, s_codes[warp], lane, K, V, inv_lambda, vmax_bits, geom, n_slices, kv_heads, n_old, win_start, cur_bits, i0,
             n_new);
}

// Bulk appends (prefill): body tiles that consist of new tokens only are built whole, one warp per
// (tile, slice, K|V).  Every lane loads exactly the elements whose codes the tile layout makes it own
// (K part: tokens {g, g+8} x channels {8W + 2 tig + h}; V part: tokens {2 tig + 8r + h} x channels
// {8J + g}), so a token's minimum and maximum meet inside a quad (K) or across the eight lanes of equal
// tig (V), the codes are packed in registers (Eq. 3 chain to the body width included) and leave as the
// lane's own 16-byte chunks: coalesced 128-bit stores, no shared memory.  The strided 2- and 4-byte
// loads of one warp cover whole 4 KB of input; the sectors they share are served by L1.

// Eq. 1-2 at 16 bit on N values of one token that a lane holds, given the token's min and max; the
// values are replaced by their codes at `BITS` (Eq. 3 chain).  Returns the INT16 scale.
template <int BITS, int N>
__device__ __forceinline__ float quantize_owned(float (&x)[N], float mn, float mx, int variant) {
  const float scale = __fdiv_rn(__fsub_rn(mx, mn), 65535.0f);
  if (scale >= 0x1p-60f && scale <= 0x1p60f) {  // one scale per token: the branch is uniform in the warp
    // two values per instruction (packed fp32 pairs, each component rounded to nearest like the scalar form):
    // x - mn as x + (-mn), the residual d - q s as q (-s) + d
    static_assert(N % 2 == 0, "values are taken in pairs");
    const float y = __frcp_rn(scale);
    const float2 y2 = make_float2(y, y), ns2 = make_float2(-scale, -scale), nmn2 = make_float2(-mn, -mn);
#pragma unroll
    for (int i = 0; i < N; i += 2) {
      const float2 d = __fadd2_rn(make_float2(x[i], x[i + 1]), nmn2);
      float2 q = __fmul2_rn(d, y2);
      float2 r = __ffma2_rn(q, ns2, d);
      q = __ffma2_rn(r, y2, q);
      r = __ffma2_rn(q, ns2, d);
      q = __ffma2_rn(r, y2, q);
      const float2 c = __fadd2_rn(q, make_float2(8388608.0f, 8388608.0f));  // code_of_quotient, both at once
      if constexpr (BITS == 16) {  // the code is the low half of the sum's bit pattern; the packing keeps only that
        x[i] = c.x;
        x[i + 1] = c.y;
      } else {
        x[i] = __uint_as_float(shift_chain((uint32_t)(__float_as_int(c.x) - 0x4B000000), BITS, variant));
        x[i + 1] = __uint_as_float(shift_chain((uint32_t)(__float_as_int(c.y) - 0x4B000000), BITS, variant));
      }
    }
  } else {  // constant tokens (0 / 0 converts to code 0) and scales far outside any real tensor's range
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const int c = min(max(__float2int_rn(__fdiv_rn(__fsub_rn(x[i], mn), scale)), 0), 65535);
      x[i] = __uint_as_float(shift_chain((uint32_t)c, BITS, variant));
    }
  }
  return scale;
}

// Lane-words of one token pair: word w holds codes idx = w n + j (n = 16 / BITS) of the token (or
// channel) in half 0 and of its partner in half 1.  lo / hi: the 16 codes (as bit patterns) of the halves,
// `step` entries apart.
template <int BITS>
__device__ __forceinline__ void pack_words(const float *lo, const float *hi, int step, uint32_t *words) {
  constexpr int n = 16 / BITS;
  if constexpr (BITS == 16) {  // one code per half; only the low 16 bits of a pattern are the code
#pragma unroll
    for (int w = 0; w < 16; ++w) words[w] = __byte_perm(__float_as_uint(lo[w * step]), __float_as_uint(hi[w * step]), 0x5410);
  } else {
#pragma unroll
    for (int w = 0; w < BITS; ++w) {
      uint32_t a = 0, b = 0;
#pragma unroll
      for (int j = 0; j < n; ++j) {
        a |= __float_as_uint(lo[(w * n + j) * step]) << (j * BITS);
        b |= __float_as_uint(hi[(w * n + j) * step]) << (j * BITS);
      }
      words[w] = a | (b << 16);
    }
  }
}

// The lane's words lw = r BITS .. r BITS + BITS - 1 (lane-word lw sits in chunk lw / 4 at word lw % 4).
template <int BITS>
__device__ __forceinline__ void store_words(uint8_t *part, int r, int lane, const uint32_t *words) {
  if constexpr (BITS >= 4) {
#pragma unroll
    for (int q = 0; q < BITS / 4; ++q)
      *reinterpret_cast<uint4 *>(part + ((r * (BITS / 4) + q) * 32 + lane) * 16) =
          make_uint4(words[4 * q], words[4 * q + 1], words[4 * q + 2], words[4 * q + 3]);
  } else {
    *reinterpret_cast<uint2 *>(part + lane * 16 + r * 8) = make_uint2(words[0], words[1]);
  }
}

constexpr int kStageRowBytes = 272;  // a staged bf16 row of 128 channels plus 16 bytes: the owner-mapped reads below hit 32 different banks
template <int BITS>
__device__ __forceinline__ void append_tile_half(const uint16_t *__restrict__ src, size_t row_stride,
                                                 const float *__restrict__ il, uint8_t *dst_tile, int is_value,
                                                 unsigned *vmax_slot, int lane, int variant, uint8_t *stage) {
  const int g = lane >> 2, tig = lane & 3;
  uint32_t words[BITS];
  // the tile's 16 rows of 256 bytes come in with eight coalesced 16-byte loads per lane, all in flight at once
  {
    uint4 v[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int id = lane + 32 * c;
      v[c] = *reinterpret_cast<const uint4 *>(src + (size_t)(id >> 4) * row_stride + (id & 15) * 8);
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int id = lane + 32 * c;
      *reinterpret_cast<uint4 *>(stage + (id >> 4) * kStageRowBytes + (id & 15) * 16) = v[c];
    }
    __syncwarp();
  }
  if (!is_value) {
#pragma unroll 1
    for (int r = 0; r < 2; ++r) {  // token g + 8 r
      float x[32];                 // [2 W + h]
      const uint8_t *row = stage + (g + 8 * r) * kStageRowBytes + 4 * tig;
#pragma unroll
      for (int W = 0; W < 16; ++W) {
        const uint32_t raw = *reinterpret_cast<const uint32_t *>(row + 16 * W);
        const float2 l2 = __ldg(reinterpret_cast<const float2 *>(il + 8 * W + 2 * tig));  // Lambda^-1, L1-resident
        const float2 xl = __fmul2_rn(make_float2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xFFFF0000u)), l2);
        x[2 * W] = xl.x;
        x[2 * W + 1] = xl.y;
      }
      float mn = x[0], mx = x[0];
#pragma unroll
      for (int i = 1; i < 32; ++i) { mn = fminf(mn, x[i]); mx = fmaxf(mx, x[i]); }
#pragma unroll
      for (int o = 1; o <= 2; o <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      const float s16 = quantize_owned<BITS>(x, mn, mx, variant);
      pack_words<BITS>(x, x + 1, 2, words);  // halves of a word: channels h = 0, 1 of the token
      store_words<BITS>(dst_tile, r, lane, words);
      // metadata record g / 2 holds tokens {2t, 2t+1, 8+2t, 9+2t} at entries {0, 1, 2, 3}
      if (tig == 0) {
        float *rec = reinterpret_cast<float *>(dst_tile + meta_offset(BITS) + (g >> 1) * 64) + 2 * r + (g & 1);
        rec[0] = chain_scale(s16, BITS, variant);
        rec[4] = chain_zero(mn, s16, BITS, variant);
      }
    }
  } else {
    float smax = 0.f;
#pragma unroll 1
    for (int r = 0; r < 2; ++r) {  // tokens 2 tig + 8 r + h, h = 0, 1
      float x[2][16];              // [h][J]
      const uint8_t *row = stage + (2 * tig + 8 * r) * kStageRowBytes + 2 * g;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int J = 0; J < 16; ++J)
          x[h][J] = __uint_as_float((uint32_t)*reinterpret_cast<const uint16_t *>(row + h * kStageRowBytes + 16 * J) << 16);
      float S[2], Z[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float mn = x[h][0], mx = x[h][0];
#pragma unroll
        for (int i = 1; i < 16; ++i) { mn = fminf(mn, x[h][i]); mx = fmaxf(mx, x[h][i]); }
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
          mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        S[h] = quantize_owned<BITS>(x[h], mn, mx, variant);
        Z[h] = mn;
        smax = fmaxf(smax, S[h]);
      }
      pack_words<BITS>(x[0], x[1], 1, words);  // halves of a word: tokens h = 0, 1 of one channel
      store_words<BITS>(dst_tile + v_part_offset(BITS), r, lane, words);
      if (g == 0) {  // record tig: S_V at bytes 32.., Z_V at 48.., entries 2 r + h
        float *rec = reinterpret_cast<float *>(dst_tile + meta_offset(BITS) + tig * 64 + 32) + 2 * r;
        *reinterpret_cast<float2 *>(rec) = make_float2(chain_scale(S[0], BITS, variant), chain_scale(S[1], BITS, variant));
        *reinterpret_cast<float2 *>(rec + 4) =
            make_float2(chain_zero(Z[0], S[0], BITS, variant), chain_zero(Z[1], S[1], BITS, variant));
      }
    }
    smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 1));  // the four tig groups hold different tokens
    smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 2));
    if (lane == 0) atomicMax(vmax_slot, __float_as_uint(smax));  // scale >= 0: uint order = float order
  }
}

// The same for row tiles (4 and 2 bit).  Lane 4 r' + q quantizes channels [32 q, 32 q + 32) of token
// 8 rr + r' (two rounds rr); a token's minimum and maximum meet inside a quad.  Keys leave as the token's own
// words.  Values are transposed through `scratch` (16 x 128 code bytes of this warp): afterwards lane l
// builds the words of channels l, l + 32, l + 64, l + 96, whose halves interleave the tile's tokens.
template <int BITS>
__device__ __forceinline__ void append_tile_half_row(const uint16_t *__restrict__ src, size_t row_stride,
                                                     const float *__restrict__ il, uint8_t *dst_tile, int is_value,
                                                     unsigned *vmax_slot, int lane, int variant, uint8_t *scratch) {
  constexpr int per_word = 32 / BITS, words_per_lane = 32 / per_word;
  const int rq = lane >> 2, q = lane & 3;
  float smax = 0.f;
#pragma unroll 1
  for (int rr = 0; rr < 2; ++rr) {
    const int row = 8 * rr + rq;
    float x[32];
    const uint4 *rp = reinterpret_cast<const uint4 *>(src + (size_t)row * row_stride + 32 * q);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint4 raw = rp[c];
      const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        x[8 * c + 2 * e] = __uint_as_float(w4[e] << 16);
        x[8 * c + 2 * e + 1] = __uint_as_float(w4[e] & 0xFFFF0000u);
      }
    }
    if (!is_value) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float4 l4 = __ldg(reinterpret_cast<const float4 *>(il + 32 * q) + c);  // Lambda^-1, L1-resident
        x[4 * c] = __fmul_rn(x[4 * c], l4.x); x[4 * c + 1] = __fmul_rn(x[4 * c + 1], l4.y);
        x[4 * c + 2] = __fmul_rn(x[4 * c + 2], l4.z); x[4 * c + 3] = __fmul_rn(x[4 * c + 3], l4.w);
      }
    }
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) { mn = fminf(mn, x[i]); mx = fmaxf(mx, x[i]); }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const float s16 = quantize_owned<BITS>(x, mn, mx, variant);
    if (!is_value) {
      uint32_t words[words_per_lane];
#pragma unroll
      for (int w = 0; w < words_per_lane; ++w) {
        uint32_t a = 0;
#pragma unroll
        for (int i = 0; i < per_word; ++i) a |= __float_as_uint(x[per_word * w + i]) << (16 * (i & 1) + BITS * (i >> 1));
        words[w] = a;
      }
      uint8_t *dst = dst_tile + row * 16 * BITS + q * 4 * words_per_lane;
      if constexpr (words_per_lane == 2) *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1]);
      else *reinterpret_cast<uint4 *>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
    } else {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t b4[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          b4[e] = __float_as_uint(x[16 * c + 4 * e]) | (__float_as_uint(x[16 * c + 4 * e + 1]) << 8) |
                  (__float_as_uint(x[16 * c + 4 * e + 2]) << 16) | (__float_as_uint(x[16 * c + 4 * e + 3]) << 24);
        *reinterpret_cast<uint4 *>(scratch + row * kHeadDim + 32 * q + 16 * c) = make_uint4(b4[0], b4[1], b4[2], b4[3]);
      }
      smax = fmaxf(smax, s16);
    }
    if (q == 0) {
      float *rec = reinterpret_cast<float *>(dst_tile + meta_offset(BITS) + row * 16) + (is_value ? 2 : 0);
      *reinterpret_cast<float2 *>(rec) = make_float2(chain_scale(s16, BITS, variant), chain_zero(mn, s16, BITS, variant));
    }
  }
  if (is_value) {
    __syncwarp();
    constexpr int words_per_ch = BITS / 2;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int ch = lane + 32 * j;
      uint32_t words[words_per_ch];
#pragma unroll
      for (int w = 0; w < words_per_ch; ++w) {
        uint32_t a = 0;
#pragma unroll
        for (int i = 0; i < per_word; ++i) a |= (uint32_t)scratch[(per_word * w + i) * kHeadDim + ch] << (16 * (i & 1) + BITS * (i >> 1));
        words[w] = a;
      }
      uint8_t *dst = dst_tile + v_part_offset(BITS) + ch * 2 * BITS;
      if constexpr (words_per_ch == 1) *reinterpret_cast<uint32_t *>(dst) = words[0];
      else *reinterpret_cast<uint2 *>(dst) = make_uint2(words[0], words[1]);
    }
#pragma unroll
    for (int o = 1; o <= 16; o <<= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, o));
    if (lane == 0) atomicMax(vmax_slot, __float_as_uint(smax));  // scale >= 0: uint order = float order
    __syncwarp();
  }
}

__global__ void __launch_bounds__(128, 8) append_tiles_kernel(const uint16_t *__restrict__ K, const uint16_t *__restrict__ V,
                                                           const float *__restrict__ inv_lambda, unsigned *vmax_bits,
                                                           LayerGeom geom, int n_slices, int kv_heads, int n_old,
                                                           int tile_lo, int n_tiles, int bits) {
  __shared__ __align__(16) uint8_t s_scratch[4][kTileTokens * kStageRowBytes];  // the warp's staged input rows, or its code bytes (row tiles)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wid = (long long)blockIdx.x * 4 + warp;
  if (wid >= (long long)n_tiles * n_slices * 2) return;
  const int is_value = (int)(wid & 1);
  const int slice = (int)((wid >> 1) % n_slices);
  const int tile = tile_lo + (int)((wid >> 1) / n_slices);
  const int i0 = geom.n_sink + tile * kTileTokens - n_old;  // index of the tile's first token among the new ones
  const size_t row_stride = (size_t)n_slices * kHeadDim;
  const uint16_t *src = (is_value ? V : K) + ((size_t)i0 * n_slices + slice) * kHeadDim;
  const float *il = inv_lambda + (size_t)(slice % kv_heads) * kHeadDim;
  uint8_t *dst_tile = geom.base + (size_t)slice * geom.slice_stride + geom.body_off + body_tile_offset(tile, bits, geom.stream_stride);
  switch (bits) {
    case 16: append_tile_half<16>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]); break;
    case 8: append_tile_half<8>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]); break;
    case 4:
      if (geom.rows) append_tile_half_row<4>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]);
      else append_tile_half<4>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]);
      break;
    default:
      if (geom.rows) append_tile_half_row<2>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]);
      else append_tile_half<2>(src, row_stride, il, dst_tile, is_value, vmax_bits + slice, lane, geom.shift_variant, s_scratch[warp]);
      break;
  }
}

// ---------------------------------------------------------------------------------------------
// Window eviction.  One warp per (evicted token, slice, K|V): the INT16 token leaves the ring and
// enters the body at the body width through the Eq. 3 chain (16 -> 8 -> ... -> cur_bits).  Values that
// enter a row tile share half-words with the tile's other tokens: the first evicted token of a tile does
// the tile's other evicted tokens too, and their own warps leave (see append_one).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void evict_one(long long wid, uint16_t *codes, int lane, const LayerGeom &geom, int n_slices,
                                          int first_token, int n_evict, int cur_bits) {
  const int is_value = (int)(wid & 1);
  const long long ts = wid >> 1;
  const int slice = (int)(ts % n_slices);
  int t = first_token + (int)(ts / n_slices), last = t;
  uint8_t *slice_base = geom.base + (size_t)slice * geom.slice_stride;
  if (is_value && row_layout(cur_bits, geom.rows != 0)) {
    const int j = t - geom.n_sink;
    if (t != first_token && (j & 15) != 0) return;
    last = min(first_token + n_evict, geom.n_sink + (j | 15) + 1) - 1;
  }
  for (; t <= last; ++t) {
    const int rp = (t - geom.n_sink) % geom.ring_tokens;
    const uint8_t *src_tile = slice_base + geom.ring_off + (size_t)(rp >> 4) * tile_bytes(16);
    const int src_row = rp & 15;
    load_token16(src_tile + (is_value ? v_part_offset(16) : 0), src_row, codes, is_value, lane);
    const float *smeta = reinterpret_cast<const float *>(src_tile + meta_offset(16));
    const float s16 = smeta[meta_slot(16, false, is_value ? 2 : 0, src_row) >> 2];
    const float z = smeta[meta_slot(16, false, is_value ? 3 : 1, src_row) >> 2];
    __syncwarp();
    const int j = t - geom.n_sink;
    uint8_t *dst_tile = slice_base + geom.body_off + body_tile_offset(j >> 4, cur_bits, geom.stream_stride);
    store_token(dst_tile + (is_value ? v_part_offset(cur_bits) : 0), cur_bits, j & 15, codes, is_value, lane,
                geom.shift_variant, geom.rows != 0);
    if (lane == 0) store_meta(dst_tile, cur_bits, j & 15, is_value, s16, z, geom.shift_variant, geom.rows != 0);
    __syncwarp();
  }
}

__global__ void __launch_bounds__(128) evict_kernel(LayerGeom geom, int n_slices, int first_token, int n_evict,
                                                    int cur_bits) {
  __shared__ uint16_t s_codes[4][kHeadDim];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wid = (long long)blockIdx.x * 4 + warp;
  if (wid >= (long long)n_evict * n_slices * 2) return;
  evict_one(wid, s_codes[warp], lane, geom, n_slices, first_token, n_evict, cur_bits);
}

// One decode step's cache update in a single launch: the tokens that leave the window (warps
// [0, 2 n_evict n_slices)) and the one new token (the rest).  Only valid when no evicted token
// shares its ring slot with the new token (single-token appends: the ring is larger than window +
// evict_chunk) and the new token does not enter a body tile that an evicted token enters too (the host
// sends the one configuration where that happens, window = 0 with evict_chunk > 1, through two launches).
__global__ void __launch_bounds__(128) append_decode_kernel(const uint16_t *__restrict__ K,
                                                            const uint16_t *__restrict__ V,
                                                            const float *__restrict__ inv_lambda, unsigned *vmax_bits,
                                                            LayerGeom geom, int n_slices, int kv_heads, int n_old,
                                                            int win_start, int cur_bits, int first_evicted, int n_evict) {
  __shared__ uint16_t s_codes[4][kHeadDim];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long wid = (long long)blockIdx.x * 4 + warp;
  const long long n_ev = (long long)n_evict * n_slices * 2;
  if (wid < n_ev) {
    evict_one(wid, s_codes[warp], lane, geom, n_slices, first_evicted, n_evict, cur_bits);
  } else if (wid < n_ev + 2ll * n_slices) {
    append_one(wid - n_ev, s_codes[warp], lane, K, V, inv_lambda, vmax_bits, geom, n_slices, kv_heads, n_old, win_start,
               cur_bits);
  }
}

// ---------------------------------------------------------------------------------------------
// One decode step's cache update for ALL blocks in a single launch.  The blocks' geometry is a
// table in device memory (written once when the cache is created); their token counts and widths
// travel as kernel arguments.  Per block the warps are laid out as in append_decode_kernel, with
// room for evict_chunk evictions whether or not this step has any.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxStepLayers = 128;
struct StepParams {
  int n_old[kMaxStepLayers];               // tokens cached in each block before this step
  unsigned char cur_bits[kMaxStepLayers];  // body width of each block
};

__global__ void __launch_bounds__(128) append_step_kernel(const uint16_t *__restrict__ K, const uint16_t *__restrict__ V,
                                                          const float *__restrict__ inv_lambda, unsigned *vmax_bits,
                                                          const LayerGeom *__restrict__ geoms, const StepParams sp,
                                                          int layers, int n_slices, int kv_heads, int n_sink, int window,
                                                          int evict_chunk) {
  __shared__ uint16_t s_codes[4][kHeadDim];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long per_layer = 2ll * (evict_chunk + 1) * n_slices;
  const long long gw = (long long)blockIdx.x * 4 + warp;
  const int layer = (int)(gw / per_layer);
  if (layer >= layers) return;
  const long long w = gw - (long long)layer * per_layer;
  const LayerGeom geom = geoms[layer];
  const int n_old = sp.n_old[layer], n_after = n_old + 1, cur_bits = sp.cur_bits[layer];
  auto body_at = [&](int n) {
    const int excess = n - n_sink - window;
    return excess <= 0 ? 0 : excess / evict_chunk * evict_chunk;
  };
  const int old_ws = min(n_old, n_sink) + body_at(n_old), new_ws = min(n_after, n_sink) + body_at(n_after);
  const int ev_first = max(old_ws, n_sink), n_evict = max(0, min(new_ws, n_old) - ev_first);
  const long long ev_room = 2ll * evict_chunk * n_slices;
  if (w < ev_room) {
    if (w < 2ll * n_evict * n_slices) evict_one(w, s_codes[warp], lane, geom, n_slices, ev_first, n_evict, cur_bits);
  } else {
    const size_t in_off = (size_t)layer * n_slices * kHeadDim;
    append_one(w - ev_room, s_codes[warp], lane, K + in_off, V + in_off, inv_lambda + (size_t)layer * kv_heads * kHeadDim,
               vmax_bits + (size_t)layer * n_slices, geom, n_slices, kv_heads, n_old, new_ws, cur_bits);
  }
}

// ---------------------------------------------------------------------------------------------
// Progressive reduce 2B -> B (Eq. 3) of one tile, by one warp: two adjacent words at 2B bits become
// one word at B bits.  Everything is read and transformed before the first store, so the output may
// overlap this tile's own input.
// ---------------------------------------------------------------------------------------------
// Eq. 3 (or the plain right shift of the ablations) on all codes of two adjacent words at 2B bits, packed into
// one word at B bits: half h of the result holds the codes of half h of in0 in its low byte-half and those
// of in1 above them.  The narrow widths work on several fields of a register at once: the product
// (c + 8) 241 of an 8-bit code fits the code's own 16-bit lane, so one multiply-add serves two codes; the eight
// 4-bit codes of a word are served by one add in place (halve_nibbles_in_place).
template <int B, bool SHR>
__device__ __forceinline__ uint32_t merge_words(uint32_t in0, uint32_t in1);

// the plain right shift of the ablations: 8 codes of 4 bit -> 8 codes of 2 bit in bits 0-7, 16-23
__device__ __forceinline__ uint32_t shift_nibbles(uint32_t x) {
  const uint32_t ya = (x >> 2) & 0x03030303u, yb = (x >> 6) & 0x03030303u;  // even / odd fields, one per byte
  return ((ya | (ya >> 4)) & 0x00330033u) | (((yb << 2) | (yb >> 2)) & 0x00CC00CCu);
}
template <bool SHR>
__device__ __forceinline__ uint32_t halve_bytes(uint32_t x) {  // 4 codes of 8 bit -> 4 codes of 4 bit in bits 0-7, 16-23
  const uint32_t a = x & 0x00FF00FFu, b = (x >> 8) & 0x00FF00FFu;  // first / second code of each half
  uint32_t ya, yb;
  if (SHR) {
    ya = (a >> 4) & 0x000F000Fu;
    yb = (b >> 4) & 0x000F000Fu;
  } else {  // (241 (c + 8)) >> 12 per 16-bit lane: 241 * 263 = 63383 stays inside the lane
    ya = ((a * 241u + 0x07880788u) >> 12) & 0x000F000Fu;
    yb = ((b * 241u + 0x07880788u) >> 12) & 0x000F000Fu;
  }
  return ya | (yb << 4);
}
// 4 -> 2 bit without spreading the codes out: Eq. 3 at b = 2, (13 (c + 2)) >> 6, is [c >= 3] + [c >= 8] + [c >= 13]
// for the sixteen 4-bit codes.  The result's high bit is the code's bit 3; its low bit is the carry of
// (c & 7) + 5 - 2 [c >= 8] into bit 3 ((c & 7) >= 3 below 8, (c & 7) >= 5 from 8 on), a sum that stays inside 3..12,
// so all eight fields of a word are served by one add with no carry between them.
__device__ __forceinline__ uint32_t halve_nibbles_in_place(uint32_t x) {  // -> 2-bit results at the bottom of every nibble
  const uint32_t h2 = (x >> 2) & 0x22222222u;
  const uint32_t s = (x & 0x77777777u) + 0x55555555u - h2;
  return ((s >> 3) & 0x11111111u) | h2;
}
// The four results of each half (fields at the bottom of the nibbles) gathered into 8 adjacent bits, at bits 6-13
// (half 0) and 22-29 (half 1): y * 5 puts an even nibble's result right below its odd neighbour's (bits 2-5 of
// every byte), * 17 puts byte 0's four bits right below byte 1's.  The fields never overlap, so the products are
// ORs of shifted copies, done on the multiply-add pipe, which this kernel leaves idle otherwise.
__device__ __forceinline__ uint32_t gather_nibble_results(uint32_t y) { return ((y * 5u) & 0x3C3C3C3Cu) * 17u; }
template <> __device__ __forceinline__ uint32_t merge_words<2, false>(uint32_t in0, uint32_t in1) {
  return __byte_perm(gather_nibble_results(halve_nibbles_in_place(in0)) >> 6, gather_nibble_results(halve_nibbles_in_place(in1)) >> 6,
                     0x6240);
}
template <> __device__ __forceinline__ uint32_t merge_words<2, true>(uint32_t in0, uint32_t in1) { return shift_nibbles(in0) | (shift_nibbles(in1) << 8); }
template <> __device__ __forceinline__ uint32_t merge_words<4, false>(uint32_t in0, uint32_t in1) { return halve_bytes<false>(in0) | (halve_bytes<false>(in1) << 8); }
template <> __device__ __forceinline__ uint32_t merge_words<4, true>(uint32_t in0, uint32_t in1) { return halve_bytes<true>(in0) | (halve_bytes<true>(in1) << 8); }
// 16 -> 8 bit: the product (c + 128) * 65281 needs all 32 bits; the new code is its top byte
template <> __device__ __forceinline__ uint32_t merge_words<8, false>(uint32_t in0, uint32_t in1) {
  const uint32_t p00 = (in0 & 0xFFFFu) * 65281u + 0x7F8080u, p01 = (in0 >> 16) * 65281u + 0x7F8080u;
  const uint32_t p10 = (in1 & 0xFFFFu) * 65281u + 0x7F8080u, p11 = (in1 >> 16) * 65281u + 0x7F8080u;
  return __byte_perm(__byte_perm(p00, p10, 0x0073), __byte_perm(p01, p11, 0x0073), 0x5410);  // {p00.3, p10.3, p01.3, p11.3}
}
template <> __device__ __forceinline__ uint32_t merge_words<8, true>(uint32_t in0, uint32_t in1) {
  return __byte_perm(__byte_perm(in0, in1, 0x0051), __byte_perm(in0, in1, 0x0073), 0x5410);  // the high byte of each code
}

// One lane-owned tile at 2B bits in a lane's registers: B 16-byte chunks per part, and the lane's 8 bytes of metadata.
template <int B>
struct TileRegs {
  uint4 v[2][B];
  float2 m;
};
template <int B>
__device__ __forceinline__ void load_tile_regs(const uint8_t *in, int lane, TileRegs<B> &t) {
#pragma unroll
  for (int part = 0; part < 2; ++part)
#pragma unroll
    for (int q = 0; q < B; ++q) t.v[part][q] = *reinterpret_cast<const uint4 *>(in + part * code_part_bytes(2 * B) + (q * 32 + lane) * 16);
  t.m = *reinterpret_cast<const float2 *>(in + meta_offset(2 * B) + lane * 8);
}
// Eq. 3 on the loaded tile and its stores at B bits.
template <int B, bool SHR>
__device__ __forceinline__ void finish_tile_regs(const TileRegs<B> &t, uint8_t *out, int lane, int variant) {
  constexpr int OUT_WORDS = 2 * B;                      // words per lane per part at B bits
  constexpr int OUT_CHUNKS = (OUT_WORDS + 3) / 4;
#pragma unroll
  for (int part = 0; part < 2; ++part) {
    uint32_t w[B * 4], o[OUT_CHUNKS * 4];
#pragma unroll
    for (int q = 0; q < B; ++q) {
      w[4 * q + 0] = t.v[part][q].x; w[4 * q + 1] = t.v[part][q].y; w[4 * q + 2] = t.v[part][q].z; w[4 * q + 3] = t.v[part][q].w;
    }
    // out lane-word r*B + w'  <-  in lane-words r*2B + 2w', r*2B + 2w' + 1
#pragma unroll
    for (int lw = 0; lw < OUT_WORDS; ++lw) {
      const int r = lw / B, wp = lw % B;
      o[lw] = merge_words<B, SHR>(w[r * 2 * B + 2 * wp], w[r * 2 * B + 2 * wp + 1]);
    }
    uint8_t *dst = out + part * code_part_bytes(B);
    if constexpr (OUT_WORDS >= 4) {
#pragma unroll
      for (int q = 0; q < OUT_CHUNKS; ++q)
        *reinterpret_cast<uint4 *>(dst + (q * 32 + lane) * 16) = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
    } else {
      *reinterpret_cast<uint4 *>(dst + lane * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  float2 m = t.m;
  const int kind = ((2 * lane) & 15) >> 2;  // 0 S_K, 1 Z_K, 2 S_V, 3 Z_V
  // a zero-point lane finds the scales of its two tokens two lanes below (16 bytes earlier)
  const float s_x = __shfl_up_sync(0xffffffffu, m.x, 2), s_y = __shfl_up_sync(0xffffffffu, m.y, 2);
  if ((kind & 1) == 0) {
    float unused = 0.f;
    halve_meta(m.x, unused, B, variant);
    halve_meta(m.y, unused, B, variant);
  } else if (variant == kShiftModified) {
    float sx = s_x, sy = s_y;
    halve_meta(sx, m.x, B, variant);
    halve_meta(sy, m.y, B, variant);
  }
  *reinterpret_cast<float2 *>(out + meta_offset(B) + lane * 8) = m;
}
// The tiles lo + warp, lo + warp + n_warps, ... below hi of a wave, by one warp: the loads of a warp's next tile
// are in flight while it works on the current one (every output of a wave lies below every input of the wave).
template <int B, bool SHR>
__device__ __forceinline__ void reduce_wave_tiles(uint8_t *base, int lo, int hi, int warp, int n_warps, int lane, int variant) {
  int j = lo + warp;
  if (j >= hi) return;
  TileRegs<B> a, b;  // two tiles take turns, so no tile is ever copied from one set of registers to another
  load_tile_regs<B>(base + (size_t)j * tile_bytes(2 * B), lane, a);
  while (true) {
    const bool more_b = j + n_warps < hi;
    if (more_b) load_tile_regs<B>(base + (size_t)(j + n_warps) * tile_bytes(2 * B), lane, b);
    finish_tile_regs<B, SHR>(a, base + (size_t)j * tile_bytes(B), lane, variant);
    if (!more_b) break;
    j += n_warps;
    const bool more_a = j + n_warps < hi;
    if (more_a) load_tile_regs<B>(base + (size_t)(j + n_warps) * tile_bytes(2 * B), lane, a);
    finish_tile_regs<B, SHR>(b, base + (size_t)j * tile_bytes(B), lane, variant);
    if (!more_a) break;
    j += n_warps;
  }
}

// CTA_WIDE: the warps of a CTA work on consecutive tiles at once; a CTA-wide barrier (reached by every
// warp, `active` or not) separates all their loads from all their stores.
template <int B, bool SHR>
__device__ __forceinline__ void reduce_tile_v(const uint8_t *in, uint8_t *out, int lane, int variant, bool active, bool cta_wide) {
  constexpr int IN_CHUNKS = B;                          // 16-byte chunks per lane per part at 2B bits
  constexpr int OUT_WORDS = 2 * B;                      // words per lane per part at B bits
  constexpr int OUT_CHUNKS = (OUT_WORDS + 3) / 4;
  uint32_t o[2][OUT_CHUNKS * 4];
  float2 m = make_float2(0.f, 0.f);
  if (active) {
#pragma unroll
  for (int part = 0; part < 2; ++part) {
    const uint8_t *src = in + part * code_part_bytes(2 * B);
    uint32_t w[IN_CHUNKS * 4];
#pragma unroll
    for (int q = 0; q < IN_CHUNKS; ++q) {
      const uint4 v = *reinterpret_cast<const uint4 *>(src + (q * 32 + lane) * 16);
      w[4 * q + 0] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
    }
    // out lane-word r*B + w'  <-  in lane-words r*2B + 2w', r*2B + 2w' + 1
#pragma unroll
    for (int lw = 0; lw < OUT_WORDS; ++lw) {
      const int r = lw / B, wp = lw % B;
      o[part][lw] = merge_words<B, SHR>(w[r * 2 * B + 2 * wp], w[r * 2 * B + 2 * wp + 1]);
    }
  }
  m = *reinterpret_cast<const float2 *>(in + meta_offset(2 * B) + lane * 8);
  const int kind = ((2 * lane) & 15) >> 2;  // 0 S_K, 1 Z_K, 2 S_V, 3 Z_V
  // a zero-point lane finds the scales of its two tokens two lanes below (16 bytes earlier)
  const float s_x = __shfl_up_sync(0xffffffffu, m.x, 2), s_y = __shfl_up_sync(0xffffffffu, m.y, 2);
  if ((kind & 1) == 0) {
    float unused = 0.f;
    halve_meta(m.x, unused, B, variant);
    halve_meta(m.y, unused, B, variant);
  } else if (variant == kShiftModified) {
    float sx = s_x, sy = s_y;
    halve_meta(sx, m.x, B, variant);
    halve_meta(sy, m.y, B, variant);
  }
  }
  // every lane (every warp of the CTA) holds its transformed data: the input is dead from here on
  if (cta_wide) __syncthreads();
  else __syncwarp();
  if (!active) return;
#pragma unroll
  for (int part = 0; part < 2; ++part) {
    uint8_t *dst = out + part * code_part_bytes(B);
#pragma unroll
    for (int q = 0; q < OUT_CHUNKS; ++q) {
      *reinterpret_cast<uint4 *>(dst + (q * 32 + lane) * 16) =
          make_uint4(o[part][4 * q], o[part][4 * q + 1], o[part][4 * q + 2], o[part][4 * q + 3]);
    }
  }
  *reinterpret_cast<float2 *>(out + meta_offset(B) + lane * 8) = m;
}

template <int B>
__device__ __forceinline__ void reduce_tile(const uint8_t *in, uint8_t *out, int lane, int variant, bool active, bool cta_wide) {
  if (variant == kShiftEquivalent) reduce_tile_v<B, false>(in, out, lane, variant, active, cta_wide);
  else reduce_tile_v<B, true>(in, out, lane, variant, active, cta_wide);
}

// Row tile at 4 bit -> row tile at 2 bit: in both parts the words of a row pair up (a token row has 16
// words, a channel row 2), so the tile is a flat array of word pairs; a lane takes four words at a time.
template <bool SHR>
__device__ __forceinline__ void reduce_tile_row(const uint8_t *in, uint8_t *out, int lane, int variant, bool active, bool cta_wide) {
  uint2 o[2][2];
  float4 m = make_float4(0.f, 0.f, 0.f, 0.f);
  if (active) {
#pragma unroll
    for (int part = 0; part < 2; ++part)
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint4 v = *reinterpret_cast<const uint4 *>(in + part * code_part_bytes(4) + (q * 32 + lane) * 16);
        o[part][q] = make_uint2(merge_words<2, SHR>(v.x, v.y), merge_words<2, SHR>(v.z, v.w));
      }
    if (lane < 16) {
      m = *reinterpret_cast<const float4 *>(in + meta_offset(4) + lane * 16);
      halve_meta(m.x, m.y, 2, variant);
      halve_meta(m.z, m.w, 2, variant);
    }
  }
  if (cta_wide) __syncthreads();  // every warp of the CTA holds its transformed tile: the inputs are dead from here on
  else __syncwarp();
  if (!active) return;
#pragma unroll
  for (int part = 0; part < 2; ++part)
#pragma unroll
    for (int q = 0; q < 2; ++q) *reinterpret_cast<uint2 *>(out + part * code_part_bytes(2) + (q * 32 + lane) * 8) = o[part][q];
  if (lane < 16) *reinterpret_cast<float4 *>(out + meta_offset(2) + lane * 16) = m;
}

// Lane-owned tile at 8 bit -> row tile at 4 bit.  The 4-bit codes go through `scratch` (16 x 128 code
// bytes of this warp, one part at a time), from which the lanes gather the row words.
template <bool SHR>
__device__ __forceinline__ void reduce_tile_to_row(const uint8_t *in, uint8_t *out, int lane, int variant, bool active,
                                                   bool cta_wide, uint8_t *scratch) {
  const int g = lane >> 2, tig = lane & 3;
  uint4 ko[4];       // K part: this lane's 16 bytes of rows lane / 2 (+ 0, 1 ... see below)
  uint2 vo[4];       // V part: channels lane, lane + 32, ...
  float m[8];        // metadata records
  if (active) {
#pragma unroll
    for (int part = 0; part < 2; ++part) {
      const uint8_t *src = in + part * code_part_bytes(8);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 v = *reinterpret_cast<const uint4 *>(src + (q * 32 + lane) * 16);
        const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int lw = 4 * q + e, r = lw >> 3, w = lw & 7;
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const uint32_t c8 = (w4[e] >> (16 * h + 8 * j)) & 0xFFu;
              const uint32_t c4 = SHR ? c8 >> 4 : shift_step(c8, 4);
              const int idx = 2 * w + j;
              const int row = part == 0 ? g + 8 * r : 2 * tig + 8 * r + h;
              const int ch = part == 0 ? 8 * idx + 2 * tig + h : 8 * idx + g;
              scratch[row * kHeadDim + ch] = (uint8_t)c4;
            }
        }
      }
      __syncwarp();
      if (part == 0) {
        // K rows: 16 rows x 16 words; lane l builds words 4 (l & 3) .. + 3 of rows (l >> 2) and (l >> 2) + 8
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          const int row = (lane >> 2) + 8 * rr;
          uint32_t wd[4];
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            const uint2 b = *reinterpret_cast<const uint2 *>(scratch + row * kHeadDim + 8 * (4 * (lane & 3) + w));
            uint32_t a = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t c = ((i < 4 ? b.x : b.y) >> (8 * (i & 3))) & 0xFu;
              a |= c << (16 * (i & 1) + 4 * (i >> 1));
            }
            wd[w] = a;
          }
          ko[rr] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int ch = lane + 32 * j;
          uint32_t wd[2];
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            uint32_t a = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) a |= (uint32_t)scratch[(8 * w + i) * kHeadDim + ch] << (16 * (i & 1) + 4 * (i >> 1));
            wd[w] = a;
          }
          vo[j] = make_uint2(wd[0], wd[1]);
        }
      }
      __syncwarp();
    }
    // metadata: lane-owned records {S_K[4], Z_K[4], S_V[4], Z_V[4]} per tig -> rows; lane l < 16 takes token row l
    if (lane < 16) {
      const float *mi = reinterpret_cast<const float *>(in + meta_offset(8));
#pragma unroll
      for (int kind = 0; kind < 4; ++kind) m[kind] = mi[meta_slot(8, false, kind, lane) >> 2];
      halve_meta(m[0], m[1], 4, variant);
      halve_meta(m[2], m[3], 4, variant);
    }
  }
  if (cta_wide) __syncthreads();  // every warp of the CTA holds its transformed tile: the inputs are dead from here on
  else __syncwarp();
  if (!active) return;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr)
    *reinterpret_cast<uint4 *>(out + ((lane >> 2) + 8 * rr) * 64 + 16 * (lane & 3)) = ko[rr];
#pragma unroll
  for (int j = 0; j < 4; ++j) *reinterpret_cast<uint2 *>(out + v_part_offset(4) + (lane + 32 * j) * 8) = vo[j];
  if (lane < 16) *reinterpret_cast<float4 *>(out + meta_offset(4) + lane * 16) = make_float4(m[0], m[1], m[2], m[3]);
}

// The whole body of a block in one launch: one CTA per (stream, slice) compacts its stream in place.  Inside
// a stream tile j moves from j tile_bytes(2B) to j tile_bytes(B).  The CTA first takes tiles [0, W), one per
// warp, with a CTA-wide barrier between their loads and their stores; then waves [lo, hi) with
// hi tile_bytes(B) <= lo tile_bytes(2B): every output of a wave lies below every input of the wave, so the
// warps run through the wave's tiles without meeting, and a barrier between waves keeps a wave's stores
// behind the earlier waves' loads.  The waves grow geometrically (x 1.8 - 1.9).
// Warps per CTA: enough tiles in flight per stream to cover the memory latency, and few enough registers
// that every (stream, slice) CTA of the common shapes is resident at once.  4 -> 2 bit keeps two tiles per warp
// in registers (80 registers at 6 warps); measured at 64 slices x 32K tokens, 6 warps 84 us,
// 5 warps 85, 8 warps (64 registers, spilling) 90, 4 warps 89; a cp.async ring of 2-4 tiles per warp in shared
// memory instead of the registers changed nothing (88 us at 8 warps): the three widths all sit on
// 14 us + bytes / 6.4 TB/s, the 14 us being the launch, the short first waves and the uneven end.
template <int B> __host__ __device__ constexpr int reduce_warps() { return B == 2 ? 6 : 8; }
template <int B> __host__ __device__ constexpr int reduce_min_ctas() { return 4; }
template <int B>
__device__ __forceinline__ void reduce_one_tile(const LayerGeom &geom, const uint8_t *in, uint8_t *out, int lane, bool active,
                                                bool cta_wide, uint8_t *scratch) {
  const bool shr = geom.shift_variant != kShiftEquivalent;
  if (B == 8 || !geom.rows) {
    reduce_tile<B>(in, out, lane, geom.shift_variant, active, cta_wide);
  } else if constexpr (B == 4) {
    if (shr) reduce_tile_to_row<true>(in, out, lane, geom.shift_variant, active, cta_wide, scratch);
    else reduce_tile_to_row<false>(in, out, lane, geom.shift_variant, active, cta_wide, scratch);
  } else {
    if (shr) reduce_tile_row<true>(in, out, lane, geom.shift_variant, active, cta_wide);
    else reduce_tile_row<false>(in, out, lane, geom.shift_variant, active, cta_wide);
  }
}

template <int B>
__global__ void __launch_bounds__(reduce_warps<B>() * 32, reduce_min_ctas<B>()) reduce_stream_kernel(LayerGeom geom, int n_tiles) {
  constexpr int kReduceWarps = reduce_warps<B>();
  __shared__ __align__(16) uint8_t s_scratch[B == 4 ? kReduceWarps : 1][B == 4 ? kTileTokens * kHeadDim : 16];
  const int stream = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint8_t *base = geom.base + (size_t)blockIdx.y * geom.slice_stride + geom.body_off + (size_t)stream * geom.stream_stride;
  const int cnt = (n_tiles - stream + kStreams - 1) / kStreams;  // tiles of this stream
  uint8_t *scratch = s_scratch[B == 4 ? warp : 0];
  if (cnt <= 0) return;
  reduce_one_tile<B>(geom, base + (size_t)warp * tile_bytes(2 * B), base + (size_t)warp * tile_bytes(B), lane, warp < cnt, true, scratch);
  for (int lo = kReduceWarps; lo < cnt;) {
    const int hi = min(cnt, (int)((long long)lo * tile_bytes(2 * B) / tile_bytes(B)));
    __syncthreads();  // the stores of this wave may land on inputs of the tiles before it
    if (B == 2 && !geom.rows) {  // few registers per tile at this width: a warp keeps its next tile's loads in flight
      if (geom.shift_variant == kShiftEquivalent) reduce_wave_tiles<B, false>(base, lo, hi, warp, kReduceWarps, lane, geom.shift_variant);
      else reduce_wave_tiles<B, true>(base, lo, hi, warp, kReduceWarps, lane, geom.shift_variant);
    } else {
      for (int j = lo + warp; j < hi; j += kReduceWarps)
        reduce_one_tile<B>(geom, base + (size_t)j * tile_bytes(2 * B), base + (size_t)j * tile_bytes(B), lane, true, false, scratch);
    }
    lo = hi;
  }
}

}  // namespace pmkvq

// Decode attention over the 4- and 2-bit body of a slice on the fifth-generation tensor cores.
//
// Included by kernels_attn.cuh (which holds the work decomposition, the INT16 tile path and the split-K
// combine).  A body block is 128 consecutive tokens = the eight tiles at one index of a slice's eight
// streams.  The CTA's three warpgroups each take every third block of the segment; per block a warpgroup
//
//   1. waits for the block's tiles (eight cp.async.bulk copies that complete on an mbarrier, issued one
//      block ahead by one thread);
//   2. K: thread t unpacks the 128 codes of token t into fp16 bit patterns (a code field left in place
//      below bit 11 of an fp16 is exactly code * 2^(pos-24); one AND per pair of codes) and stores them as
//      row t of the A operand in tensor memory (tcgen05.st);
//   3. one thread issues S[token, head] = A_K . Q''^T: 8 tcgen05.mma (128 x 16 x 16, fp16 in, fp32
//      accumulators in tensor memory), B = the query fragments in shared memory (rows 0-7 the fp16 "hi"
//      part of up to 8 heads, rows 8-15 the "lo" remainder), then tcgen05.commit onto an mbarrier;
//   4. V: thread c unpacks channel c's codes of the 128 tokens into row c of the second A operand while
//      the score MMAs run;
//   5. thread t reads its token's 16 score sums (tcgen05.ld), applies scale and zero-point
//      (q.k = S_K (q.c) + Z_K sum(q)), takes p = 2^(s - m) against the warpgroup's reference m and writes
//      w = p * S_V (fp16 hi + lo per head) as row t of the MN-major B operand of the output MMA;
//   6. one thread issues O^T[channel, head] += A_V . w: one tcgen05.mma per live tile of the block.
//
// The reference m only moves when some score of a block exceeds it by more than kMaxAhead (found with one
// barrier-wide OR per block); then the warpgroup takes the block's maxima, rescales its accumulators in
// tensor memory and its running sums, and goes on.  Each warpgroup ends a segment with one partial
// (m, l, o[128]) per head, merged with the INT16 tiles' per-warp partials like any other split.
//
// Every mbarrier wait has an iteration limit; a wait that runs out sets a CTA-wide abort flag and an
// error word in global memory, after which the CTA skips its remaining waits, runs through its barriers,
// frees its tensor memory and returns (the results of that launch are then meaningless and the host
// reports PMKVQ_ERR_DEVICE_WAIT).
#pragma once

namespace pmkvq {

constexpr int kWarpgroups = 3;
constexpr int kTmemCols = 512;
constexpr int kTmemColsPerWg = 160;        // A_K 64 | A_V 64 | D_S 16 | D_O 16
constexpr int kStageTiles = kBlockTiles;   // one block per stage
constexpr int kStagesPerWg = 2;
constexpr int kWBufBytes = 4096;           // [hi | lo][128 tokens][8 heads] fp16: columns h and 8 + h of the weights
constexpr int kQOperandBytes = 4096;       // [n-group 2][k-chunk 16][8 rows][8 channels] fp16
constexpr int kEPV = 12;                   // w = p * S_V / sigma_u * 2^(kEPV - pos) stays below 2^16

// Shared-memory bookkeeping of the tensor-core path (static).
struct TcShared {
  unsigned long long bar_full[kWarpgroups][kStagesPerWg];
  unsigned long long bar_s[kWarpgroups];
  unsigned long long bar_o[kWarpgroups];
  uint32_t tmem_base;
  int abort;
  float wmax[kWarpgroups][4][kMaxGroup];   // per warp block maxima (slow path)
  float sums[kWarpgroups][4][2 * kMaxGroup];
};

// Per-thread view: tensor-memory base, barrier parities (one bit each), error word.
struct TcCtx {
  TcShared *sh;
  uint8_t *stages;    // [kWarpgroups][kStagesPerWg][8 tiles of the widest row width]
  uint8_t *q_operand; // kQOperandBytes
  uint8_t *wbuf;      // [kWarpgroups] kWBufBytes
  float *part_o;      // [kParts][8][128]
  unsigned *error_word;
  uint32_t tmem_base;
  uint32_t ph_full;   // bit s: parity of the next wait on bar_full[wg][s]
  uint32_t ph_s, ph_o;
};

constexpr int kStageBytes = kStageTiles * tile_bytes(4);

__device__ __forceinline__ void wg_sync(int wg) { asm volatile("bar.sync %0, 128;\n" ::"r"(wg + 1) : "memory"); }
// barrier over the warpgroup that also ORs a predicate
__device__ __forceinline__ bool wg_any(int wg, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(wg + 1 + kWarpgroups)
      : "memory");
  return r != 0;
}

// A wait that gives up: marks the CTA as aborted and leaves a trace for the host.
__device__ __forceinline__ void tc_wait(TcCtx &tc, uint32_t bar, uint32_t parity, unsigned code) {
  if (*reinterpret_cast<volatile int *>(&tc.sh->abort)) return;
  if (!tc05::mbar_wait(bar, parity)) {
    tc.sh->abort = 1;
    atomicOr(tc.error_word, code);
  }
}

template <int BITS> struct RowFmt;
template <> struct RowFmt<2> {
  static constexpr int SIGMA_LOG2 = 15;
  __host__ __device__ static constexpr int pos(int f) { return 2 * (f & 3); }                // f = field 0..7
  __host__ __device__ static constexpr int field(int idx) { return (idx & 15) >> 1; }        // of channel / token index
  // one word (16 codes) -> 8 tensor-memory columns (column f = fields f of the two halves)
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t *e) {
    const uint32_t xr = x >> 8;
    e[0] = x & 0x00030003u; e[1] = x & 0x000C000Cu; e[2] = x & 0x00300030u; e[3] = x & 0x00C000C0u;
    e[4] = xr & 0x00030003u; e[5] = xr & 0x000C000Cu; e[6] = xr & 0x00300030u; e[7] = xr & 0x00C000C0u;
  }
};
template <> struct RowFmt<4> {
  static constexpr int SIGMA_LOG2 = 13;
  __host__ __device__ static constexpr int pos(int f) { return (f & 1) ? 4 : 0; }            // f = field 0..3
  __host__ __device__ static constexpr int field(int idx) { return (idx & 7) >> 1; }
  // one word (8 codes) -> 4 columns
  __device__ static __forceinline__ void extract(uint32_t x, uint32_t *e) {
    const uint32_t xr = x >> 8;
    e[0] = x & 0x000F000Fu; e[1] = x & 0x00F000F0u;
    e[2] = xr & 0x000F000Fu; e[3] = xr & 0x00F000F0u;
  }
};

// The B operand of the score MMAs: Q'' of the slice's heads at the code positions of width BITS, K-major,
// no swizzle: element (n, k) at (n / 8) * 2048 + (k / 8) * 128 + (n % 8) * 16 + (k % 8) * 2; rows n < 8 hold
// the fp16 "hi" part of head n, rows n >= 8 the "lo" remainder of head n - 8.  MMA k index = channel.
template <int BITS>
__device__ __forceinline__ void fill_q_operand(uint8_t *dst, const float (*s_q)[kHeadDim], const float *s_stat) {
  using F = RowFmt<BITS>;
  for (int i = threadIdx.x; i < kMaxGroup * kHeadDim; i += kAttnThreads) {
    const int h = i >> 7, k = i & 127;
    const float x = s_q[h][k] * ldexpf(1.0f, 14 - F::pos(F::field(k)) - (int)s_stat[h]);
    const __half hi = __float2half_rn(x);
    const __half lo = __float2half_rn(x - __half2float(hi));
    const int off = (k >> 3) * 128 + h * 16 + (k & 7) * 2;
    *reinterpret_cast<__half *>(dst + off) = hi;
    *reinterpret_cast<__half *>(dst + 2048 + off) = lo;
  }
}

// One warpgroup's walk over its blocks of the segment's body tiles [t_lo, t_hi).  Leaves the warpgroup's
// partial in slot `slot` of (s_m, s_l, part_o).
template <int BITS>
__device__ __forceinline__ void tc_body(const AttnParams &p, TcCtx &tc, const uint8_t *body, int t_lo, int t_hi,
                                        const float *s_stat, float sigma16, float *s_m, float *s_l, int slot) {
  using F = RowFmt<BITS>;
  constexpr int TB = tile_bytes(BITS);
  constexpr int ROW_BYTES = 16 * BITS;      // a token's K codes
  constexpr int CH_BYTES = 2 * BITS;        // a channel's V codes of one tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = warp >> 2, quad = warp & 3;
  const int tw = threadIdx.x & 127;         // token row of a block (scores) and channel (output)
  const int my_tile = tw >> 4, my_row = tw & 15;
  TcShared *sh = tc.sh;
  const uint32_t t_lane = (uint32_t)(quad * 32) << 16;
  const uint32_t tA_K = tc.tmem_base + wg * kTmemColsPerWg, tA_V = tA_K + 64, tD_S = tA_K + 128, tD_O = tA_K + 144;
  uint8_t *stage_base = tc.stages + (size_t)wg * kStagesPerWg * kStageBytes;
  uint8_t *wbuf = tc.wbuf + wg * kWBufBytes;
  const uint32_t bar_full0 = tc05::smem_u32(&sh->bar_full[wg][0]);
  const uint32_t bar_s = tc05::smem_u32(&sh->bar_s[wg]), bar_o = tc05::smem_u32(&sh->bar_o[wg]);
  const uint32_t q_addr = tc05::smem_u32(tc.q_operand), w_addr = tc05::smem_u32(wbuf);
  constexpr uint32_t idesc_qk = tc05::idesc_f16(128, 16, 0), idesc_pv = tc05::idesc_f16(128, 16, 1);

  const int kb0 = t_lo >> 3, kb1 = (t_hi - 1) >> 3;
  // issue the copies of block kb into stage s (warp 0 of the warpgroup; lane i copies tile i)
  auto issue_block = [&](int kb, int s) {
    const int lo_i = max(t_lo - 8 * kb, 0), hi_i = min(t_hi - 8 * kb, 8);
    const uint32_t bar = bar_full0 + 8 * s;
    if (lane == 0) tc05::mbar_arrive_expect_tx(bar, (uint32_t)((hi_i - lo_i) * TB));
    __syncwarp();
    if (lane >= lo_i && lane < hi_i)
      tc05::bulk_g2s(tc05::smem_u32(stage_base + (size_t)s * kStageBytes + lane * TB),
                     body + (size_t)lane * p.geom.stream_stride + (size_t)kb * TB, TB, bar);
  };

  // per-head constants
  float2 mu2[4], sumq2[4], m2[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    mu2[j] = make_float2(ldexpf(1.0f, 24 - 14 + (int)s_stat[2 * j]), ldexpf(1.0f, 24 - 14 + (int)s_stat[2 * j + 1]));
    sumq2[j] = make_float2(s_stat[8 + 2 * j], s_stat[8 + 2 * j + 1]);
    m2[j] = make_float2(kNegBig, kNegBig);
  }
  float2 l2[4], zs2[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) l2[j] = zs2[j] = make_float2(0.f, 0.f);
  const float sigma_u = sigma16 * ldexpf(1.0f, F::SIGMA_LOG2);
  // the weight of this thread's token row in the output MMA carries the row's code position
  const float w_unit = ldexpf(1.0f, kEPV - F::pos(F::field(my_row))) / sigma_u;

  if (quad == 0 && kb0 + wg <= kb1) issue_block(kb0 + wg, 0);
  // The tensor core adds into its fp32 accumulators without rounding to nearest, and the sums of codes
  // times weights are all of one sign: left to grow over thousands of MMAs the loss shows in the output,
  // which is the small difference of that sum and the zero-point sum.  So every kEpochBlocks blocks the
  // accumulators of this thread's channel move into registers (ov) and the tensor-memory sums restart.
  constexpr int kEpochBlocks = 16;
  float ov[8];
#pragma unroll
  for (int h = 0; h < 8; ++h) ov[h] = 0.f;
  bool first = true;  // the tensor-memory accumulators hold nothing yet
  int it = 0, since = 0;
  for (int kb = kb0 + wg; kb <= kb1; kb += kWarpgroups, ++it) {
    const int s = it & 1;
    const int lo_i = max(t_lo - 8 * kb, 0), hi_i = min(t_hi - 8 * kb, 8);
    const uint8_t *blk = stage_base + (size_t)s * kStageBytes;
    tc_wait(tc, bar_full0 + 8 * s, (tc.ph_full >> s) & 1u, 1u);
    tc.ph_full ^= 1u << s;

    // ---- K: token row -> tensor memory ----
    {
      const uint8_t *kp = blk + my_tile * TB + my_row * ROW_BYTES;
      constexpr int HALF_CHUNKS = ROW_BYTES / 32;  // 16-byte chunks per half row
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t r[32];
#pragma unroll
        for (int c = 0; c < HALF_CHUNKS; ++c) {
          const uint4 v = *reinterpret_cast<const uint4 *>(kp + (half * HALF_CHUNKS + c) * 16);
          const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) F::extract(w4[e], r + (4 * c + e) * (32 / (4 * HALF_CHUNKS)));
        }
        tc05::tmem_st32(tA_K + t_lane + 32 * half, r);
      }
    }
    tc05::wait_st();
    tc05::fence_before_sync();
    wg_sync(wg);
    if (tw == 0) {
      tc05::fence_after_sync();
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        tc05::mma_f16_ts(tD_S, tA_K + 8 * ks, tc05::smem_desc(q_addr + 256 * ks, 128, 2048), idesc_qk, ks > 0 ? 1u : 0u);
      tc05::mma_commit(bar_s);
    }
    // the other stage was last read in the previous block, which every thread has left: refill it
    if (quad == 0 && kb + kWarpgroups <= kb1) issue_block(kb + kWarpgroups, s ^ 1);

    // ---- V: channel row -> tensor memory (after the previous block's output MMAs have read it) ----
    {
      uint32_t r[64];
      const uint8_t *vp = blk + v_part_offset(BITS) + tw * CH_BYTES;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if constexpr (BITS == 2) {
          F::extract(*reinterpret_cast<const uint32_t *>(vp + i * TB), r + 8 * i);
        } else {
          const uint2 v = *reinterpret_cast<const uint2 *>(vp + i * TB);
          F::extract(v.x, r + 8 * i);
          F::extract(v.y, r + 8 * i + 4);
        }
      }
      if (it > 0) {
        tc_wait(tc, bar_o, tc.ph_o, 4u);
        tc.ph_o ^= 1u;
        tc05::fence_after_sync();
        if (since == kEpochBlocks) {
          uint32_t o[16];
          tc05::tmem_ld16(tD_O + t_lane, o);
          tc05::wait_ld();
#pragma unroll
          for (int h = 0; h < 8; ++h) ov[h] += fmaf(__uint_as_float(o[8 + h]), 0x1p-11f, __uint_as_float(o[h]));
          first = true;
          since = 0;
        }
      }
      tc05::tmem_st32(tA_V + t_lane, r);
      tc05::tmem_st32(tA_V + t_lane + 32, r + 32);
    }

    // ---- scores of this thread's token ----
    tc_wait(tc, bar_s, tc.ph_s, 2u);
    tc.ph_s ^= 1u;
    tc05::fence_after_sync();
    uint32_t sraw[16];
    tc05::tmem_ld16(tD_S + t_lane, sraw);
    tc05::wait_ld();
    const bool alive = my_tile >= lo_i && my_tile < hi_i && ((8 * kb + my_tile) * 16 + my_row) < p.n_body;
    float4 meta = *reinterpret_cast<const float4 *>(blk + my_tile * TB + meta_offset(BITS) + my_row * 16);  // S_K Z_K S_V Z_V
    if (!alive) meta = make_float4(0.f, 0.f, 0.f, 0.f);  // a dead row holds arbitrary bytes
    float2 dot[4], a2[4], arg[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      dot[j] = __fadd2_rn(make_float2(__uint_as_float(sraw[2 * j]), __uint_as_float(sraw[2 * j + 1])),
                          make_float2(__uint_as_float(sraw[8 + 2 * j]), __uint_as_float(sraw[8 + 2 * j + 1])));
      a2[j] = __fmul2_rn(mu2[j], make_float2(meta.x, meta.x));
      const float2 b = __ffma2_rn(make_float2(meta.y, meta.y), sumq2[j], make_float2(-m2[j].x, -m2[j].y));
      arg[j] = __ffma2_rn(a2[j], dot[j], b);
      if (!alive) arg[j] = make_float2(-INFINITY, -INFINITY);
    }
    float amax = fmaxf(fmaxf(fmaxf(arg[0].x, arg[0].y), fmaxf(arg[1].x, arg[1].y)),
                       fmaxf(fmaxf(arg[2].x, arg[2].y), fmaxf(arg[3].x, arg[3].y)));
    if (wg_any(wg, amax > kMaxAhead)) {
      // ---- the reference moves: block maxima of the true scores, new reference, rescale ----
      float2 sc[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        sc[j] = __ffma2_rn(a2[j], dot[j], __fmul2_rn(make_float2(meta.y, meta.y), sumq2[j]));
        if (!alive) sc[j] = make_float2(kNegBig, kNegBig);
        float mx = sc[j].x, my = sc[j].y;
#pragma unroll
        for (int o = 16; o; o >>= 1) {
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
          my = fmaxf(my, __shfl_xor_sync(0xffffffffu, my, o));
        }
        if (lane == 0) { sh->wmax[wg][quad][2 * j] = mx; sh->wmax[wg][quad][2 * j + 1] = my; }
      }
      wg_sync(wg);
      float f[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float nx = m2[j].x, ny = m2[j].y;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          nx = fmaxf(nx, sh->wmax[wg][q][2 * j]);
          ny = fmaxf(ny, sh->wmax[wg][q][2 * j + 1]);
        }
        f[2 * j] = ex2(m2[j].x - nx);
        f[2 * j + 1] = ex2(m2[j].y - ny);
        m2[j] = make_float2(nx, ny);
        l2[j] = __fmul2_rn(l2[j], make_float2(f[2 * j], f[2 * j + 1]));
        zs2[j] = __fmul2_rn(zs2[j], make_float2(f[2 * j], f[2 * j + 1]));
        ov[2 * j] *= f[2 * j];
        ov[2 * j + 1] *= f[2 * j + 1];
        arg[j] = __fadd2_rn(sc[j], make_float2(-nx, -ny));
        if (!alive) arg[j] = make_float2(-INFINITY, -INFINITY);
      }
      if (!first) {  // the output accumulators of channel row tw (every earlier output MMA has completed)
        uint32_t o[16];
        tc05::tmem_ld16(tD_O + t_lane, o);
        tc05::wait_ld();
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          o[h] = __float_as_uint(__uint_as_float(o[h]) * f[h]);
          o[8 + h] = __float_as_uint(__uint_as_float(o[8 + h]) * f[h]);
        }
        tc05::tmem_st16(tD_O + t_lane, o);
      }
      wg_sync(wg);  // wmax may be rewritten by the next slow path
    }

    // ---- probabilities and weights: w = p * S_V goes to the output MMA as fp16 hi + lo (22 bits), in
    //      columns h and 8 + h of the B operand; the sums take p itself ----
    {
      // a constant V group has S_V = 0 and all codes 0: any finite unit will do for it
      const float s_e = meta.z == 0.f ? w_unit : meta.z * w_unit;
      uint32_t whi[4], wlo[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 e = make_float2(ex2(arg[j].x), ex2(arg[j].y));
        const float2 w = __fmul2_rn(e, make_float2(s_e, s_e));
        whi[j] = pack_half2(w.x, w.y);
        const float2 back = __half22float2(*reinterpret_cast<const __half2 *>(&whi[j]));
        const float2 rest = __fmul2_rn(__fadd2_rn(w, make_float2(-back.x, -back.y)), make_float2(2048.f, 2048.f));
        wlo[j] = pack_half2(rest.x, rest.y);
        l2[j] = __fadd2_rn(l2[j], e);
        zs2[j] = __ffma2_rn(e, make_float2(meta.w, meta.w), zs2[j]);
      }
      *reinterpret_cast<uint4 *>(wbuf + tw * 16) = make_uint4(whi[0], whi[1], whi[2], whi[3]);
      *reinterpret_cast<uint4 *>(wbuf + 2048 + tw * 16) = make_uint4(wlo[0], wlo[1], wlo[2], wlo[3]);
    }
    tc05::fence_async_smem();
    tc05::wait_st();
    tc05::fence_before_sync();
    wg_sync(wg);
    if (tw == 0) {
      tc05::fence_after_sync();
      for (int j = lo_i; j < hi_i; ++j)
        tc05::mma_f16_ts(tD_O, tA_V + 8 * j, tc05::smem_desc(w_addr + 256 * j, 128, 2048), idesc_pv,
                         (first && j == lo_i) ? 0u : 1u);
      tc05::mma_commit(bar_o);
    }
    first = false;
    ++since;
  }

  // ---- the warpgroup's partial: (m, l, o[128]) per head ----
  if (it > 0) {
    tc_wait(tc, bar_o, tc.ph_o, 4u);
    tc.ph_o ^= 1u;
    tc05::fence_after_sync();
    uint32_t o[16];
    tc05::tmem_ld16(tD_O + t_lane, o);
    tc05::wait_ld();
    const float f_out = ldexpf(sigma_u, 24 - kEPV);
#pragma unroll
    for (int h = 0; h < 8; ++h) ov[h] = (ov[h] + fmaf(__uint_as_float(o[8 + h]), 0x1p-11f, __uint_as_float(o[h]))) * f_out;
  }
  // sums over the warpgroup's 128 token rows
  float red[16];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    red[2 * j] = l2[j].x; red[2 * j + 1] = l2[j].y;
    red[8 + 2 * j] = zs2[j].x; red[8 + 2 * j + 1] = zs2[j].y;
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) {
#pragma unroll
    for (int o = 16; o; o >>= 1) red[i] += __shfl_xor_sync(0xffffffffu, red[i], o);
  }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < 16; ++i) sh->sums[wg][quad][i] = red[i];
  }
  tc05::fence_before_sync();
  wg_sync(wg);
  float (*po)[kHeadDim] = reinterpret_cast<float (*)[kHeadDim]>(tc.part_o + (size_t)slot * kMaxGroup * kHeadDim);
#pragma unroll
  for (int h = 0; h < 8; ++h) {
    const float zs = sh->sums[wg][0][8 + h] + sh->sums[wg][1][8 + h] + sh->sums[wg][2][8 + h] + sh->sums[wg][3][8 + h];
    po[h][tw] = ov[h] + zs;
  }
  if (tw == 0) {
#pragma unroll
    for (int h = 0; h < 8; ++h) {
      s_m[slot * 8 + h] = (h & 1) ? m2[h >> 1].y : m2[h >> 1].x;
      s_l[slot * 8 + h] = sh->sums[wg][0][h] + sh->sums[wg][1][h] + sh->sums[wg][2][h] + sh->sums[wg][3][h];
    }
  }
}

}  // namespace pmkvq

// Decode attention over the 4- and 2-bit body of a slice on the fifth-generation tensor cores.
//
// Included by kernels_attn.cuh (which holds the work decomposition, the INT16 tile path and the split-K
// combine).  The body tiles [t_lo, t_hi) of a segment are taken stream by stream (tile t lives in stream
// t mod 8, and softmax attention does not care about the order of the tokens): in every stream the
// segment's tiles are one contiguous run of bytes, which is cut into MMA blocks of up to 8 tiles = 128
// tokens, one cp.async.bulk copy each (10 KB at 2 bit, 18 KB at 4 bit) into a ring of kStages stages in
// shared memory.  Block n belongs to warpgroup n mod 3.  Warps meet only on mbarriers (no CTA-wide barrier
// inside the loop):
//
//   warps 0-11     three block warpgroups of 128 threads.  For its block, thread t
//                  - unpacks the 128 codes of token t into fp16 bit patterns (a code field left in place
//                    below bit 11 of an fp16 is exactly code * 2^(pos-24); one AND per pair of codes) and
//                    stores them as row t of the score MMA's A operand in tensor memory (tcgen05.st);
//                  - does the same for channel t's codes of the block's tokens: row t of the output MMA's
//                    A operand (while the score MMAs run);
//                  - reads its token's 16 score sums (tcgen05.ld), applies scale and zero-point
//                    (q.k = S_K (q.c) + Z_K sum(q)), takes p = 2^(s - m) against its warpgroup's
//                    reference m and writes w = p * S_V (fp16 hi + lo per head) as row t of the MN-major
//                    B operand of the output MMA; it keeps the sums of p and p * Z_V.
//   warp 12        the copies, as far ahead as the ring has free stages;
//   warp 13        the score MMAs S[token, head] = A_K . Q''^T of every block, in block order: 8 tcgen05.mma
//                  (128 x 16 x 16, fp16 in, fp32 accumulators in tensor memory), B = the query fragments in
//                  shared memory (rows 0-7 the fp16 "hi" part of up to 8 heads, rows 8-15 the "lo"
//                  remainder), and tcgen05.commit onto the warpgroup's mbarrier;
//   warps 14, 15   the output MMAs O^T[channel, head] += A_V . w of alternate blocks, one tcgen05.mma per
//                  live tile, into the block's warpgroup's own accumulators.
//
// A_K, A_V, the score accumulators, the weight buffer and the output accumulators exist three times, one
// set per warpgroup (480 of the 512 columns of tensor memory).  A reference m only moves when some score
// of a block exceeds it by more than kTcMaxAhead (one OR over the warpgroup per block); the warpgroup
// then takes the block's maxima plus some headroom, rescales its accumulators in tensor memory and its
// running sums, and goes on.  A segment ends with one partial (m, l, o[128]) per head and warpgroup,
// merged with the INT16 tiles' per-warp partials like any split.
//
// Every mbarrier wait first tests its barrier without blocking, then polls with a time hint (the waiting
// warp sleeps in hardware instead of spinning through the issue slots of the working warps) under an
// iteration limit; a wait that runs out sets a CTA-wide abort flag and an error word in global memory,
// after which the CTA skips its remaining waits, runs through its loops, gives copies still in flight a
// bounded time to land, frees its tensor memory and returns (the results of that launch are then
// meaningless and the host reports PMKVQ_ERR_DEVICE_WAIT).
#pragma once

namespace pmkvq {

constexpr int kTcGroups = 3;               // warpgroups that each take every third block through K, V and softmax
constexpr int kTmemCols = 512;             // A_K 3 x 64 | A_V 3 x 64 | D_S 3 x 16 | D_O 3 x 16
constexpr int kTmemAK = 0, kTmemAV = 192, kTmemDS = 384, kTmemDO = 432;
constexpr int kStages = 6;                 // chunks in flight in shared memory
constexpr int kStageBytes = 8 * tile_bytes(4);    // 18 432: a chunk is 8 tiles = one MMA block at either width
constexpr int kWBufBytes = 4096;           // [hi | lo][128 tokens][8 heads] fp16: columns h and 8 + h of the weights
constexpr int kQOperandBytes = 4096;       // [n-group 2][k-chunk 16][8 rows][8 channels] fp16
constexpr int kEPV = 7;                    // w = p * S_V / sigma_u * 2^(kEPV - pos) stays below 2^16 for p <= 2^kTcMaxAhead
constexpr float kTcMaxAhead = 8.0f;        // a score may exceed the reference by this much (log2 units)
constexpr float kTcHeadroom = 4.0f;        // a new reference is set this far above the maxima seen
// warps 0-11 are the three block warpgroups; three single warps serve them
constexpr int kWarpCopy = 12, kWarpMmaS = 13, kWarpMmaO = 14;

// Shared-memory bookkeeping of the tensor-core path (static).
struct TcShared {
  unsigned long long full[kStages];           // the stage's copy has landed
  unsigned long long stage_free[kStages];     // the block's warpgroup is done with the stage (4 warp arrivals)
  unsigned long long ak_full[kTcGroups];      // the block's K operand is in tensor memory (4 warp arrivals)
  unsigned long long av_full[kTcGroups];      // the block's V operand is in tensor memory (4 warp arrivals)
  unsigned long long w_full[kTcGroups];       // the block's weights are in shared memory (4 warp arrivals)
  unsigned long long bar_s[kTcGroups], bar_o[kTcGroups];  // score / output MMAs of the warpgroup's block are complete
  uint32_t tmem_base;
  int abort;
  int pv_fresh[kTcGroups];                    // the block's first output MMA overwrites the accumulators
  float wmax[kTcGroups][4][kMaxGroup];        // per-warp block maxima (when a reference moves)
  float sums[kTcGroups][4][2 * kMaxGroup];
};

// Per-thread view: tensor-memory base, the CTA's running block and chunk counts (barrier parities follow).
struct TcCtx {
  TcShared *sh;
  uint8_t *stages;    // [kStages][kStageBytes]
  uint8_t *q_operand; // kQOperandBytes
  uint8_t *wbuf;      // [2] kWBufBytes
  float *part_o;      // [kParts][8][128]
  unsigned *error_word;
  uint32_t tmem_base;
  uint32_t gi, gc;    // body blocks / chunks this CTA has pushed through the pipeline so far (all segments)
};

// barriers over one block warpgroup (128 threads); `any` also ORs a predicate
__device__ __forceinline__ bool swg_any(int sw, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(1 + 2 * sw)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void swg_sync(int sw) { asm volatile("bar.sync %0, 128;\n" ::"r"(2 + 2 * sw) : "memory"); }

// A wait that gives up: marks the CTA as aborted and leaves a trace for the host.
__device__ __forceinline__ void tc_wait(TcCtx &tc, const unsigned long long *bar, uint32_t parity, unsigned code) {
  const uint32_t addr = tc05::smem_u32(bar);
  if (tc05::mbar_test_wait(addr, parity & 1u)) return;  // the common case costs one barrier operation
  if (*reinterpret_cast<volatile int *>(&tc.sh->abort)) return;
  const bool ok = tc05::mbar_wait(addr, parity & 1u);
  if (!ok) {
    tc.sh->abort = 1;
    atomicOr(tc.error_word, code);
  }
}
// A wait that nothing will ever satisfy, with a short limit: shows that a bounded wait gives up, reports it
// and lets the kernel end normally (the context stays usable).  One thread.
__global__ void bounded_wait_selftest_kernel(unsigned *word, unsigned limit) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = tc05::smem_u32(&bar);
  tc05::mbar_init(b, 1);
  tc05::mbar_init_fence();
  if (!tc05::mbar_wait(b, 0u, limit)) atomicOr(word, 1u);
}

// one arrival per warp, after all its lanes are done
__device__ __forceinline__ void warp_arrive(const unsigned long long *bar, int lane) {
  __syncwarp();
  if (lane == 0) tc05::mbar_arrive(tc05::smem_u32(bar));
}
template <int BITS> struct RowFmt;
template <> struct RowFmt<2> {
  static constexpr int SIGMA_LOG2 = 15, CHUNK_TILES = 8;
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
  static constexpr int SIGMA_LOG2 = 13, CHUNK_TILES = 8;
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

// Walks the blocks of the segment's body tiles [t_lo, t_hi) in the order every role uses: streams 0..7,
// in each stream the run of tiles j with t_lo <= s + 8 j < t_hi in chunks of CHUNK tiles, in each chunk
// blocks of up to 8 tiles.  on_chunk(chunk index, stream, first stream-tile j, tiles) comes before the
// chunk's blocks; on_block(block index, chunk index, stream, first stream-tile j of the block, tile offset
// inside the chunk, live tiles, last block of its chunk).
template <int CHUNK, class OnChunk, class OnBlock>
__device__ __forceinline__ void tc_walk(int t_lo, int t_hi, OnChunk on_chunk, OnBlock on_block) {
  int blk = 0, chunk = 0;
  for (int s = 0; s < kStreams; ++s) {
    const int j_lo = t_lo > s ? (t_lo - s + 7) >> 3 : 0, j_hi = t_hi > s ? (t_hi - s + 7) >> 3 : 0;
    for (int c0 = j_lo; c0 < j_hi; c0 += CHUNK, ++chunk) {
      const int tiles = min(CHUNK, j_hi - c0);
      on_chunk(chunk, s, c0, tiles);
      for (int sb = 0; sb < tiles; sb += 8, ++blk) on_block(blk, chunk, s, c0 + sb, sb, min(8, tiles - sb), sb + 8 >= tiles);
    }
  }
}

// The body tiles [t_lo, t_hi) of a segment, by all warps of the CTA in their roles.  Leaves the three block
// warpgroups' partials in slots slot0 .. slot0 + 2 of (s_m, s_l, part_o).  Buffer / stage parities follow the
// CTA-wide counts tc.gi / tc.gc: block number n uses the buffers of warpgroup n mod 3, chunk number m stage m mod kStages, and
// every completion of a barrier is either waited for or provably over before the barrier can complete again.
template <int BITS>
__device__ __forceinline__ void tc_body(const AttnParams &p, TcCtx &tc, const uint8_t *body, int t_lo, int t_hi,
                                        const float *s_stat, float sigma16, float *s_m, float *s_l, int slot0) {
  using F = RowFmt<BITS>;
  constexpr int TB = tile_bytes(BITS);
  constexpr int CHUNK = F::CHUNK_TILES;
  constexpr int ROW_BYTES = 16 * BITS;      // a token's K codes
  constexpr int CH_BYTES = 2 * BITS;        // a channel's V codes of one tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = warp & 3;
  const int tw = threadIdx.x & 127;         // token row of a block (K, scores) and channel (V, output)
  const int my_tile = tw >> 4, my_row = tw & 15;
  TcShared *sh = tc.sh;
  const uint32_t t_lane = (uint32_t)(quad * 32) << 16;
  const uint32_t tb = tc.tmem_base;
  const uint32_t g0 = tc.gi, c0g = tc.gc;
  {  // every thread advances the CTA-wide counts by this segment's blocks and chunks
    int nb = 0, nc = 0;
    for (int s = 0; s < kStreams; ++s) {
      const int j_lo = t_lo > s ? (t_lo - s + 7) >> 3 : 0, j_hi = t_hi > s ? (t_hi - s + 7) >> 3 : 0;
      const int r = j_hi - j_lo;
      nc += (r + CHUNK - 1) / CHUNK;
      nb += (r / CHUNK) * (CHUNK / 8) + ((r % CHUNK) + 7) / 8;
    }
    tc.gi += (uint32_t)nb;
    tc.gc += (uint32_t)nc;
  }
  constexpr uint32_t idesc_qk = tc05::idesc_f16(128, 16, 0), idesc_pv = tc05::idesc_f16(128, 16, 1);

  static_assert(CHUNK == 8, "a chunk is one MMA block: the stage belongs to the block's warpgroup alone");
  if (warp == kWarpCopy) {
    // ---- copies: one bulk copy per chunk into the ring, as far ahead as the ring has free stages ----
    int n_chunk = 0;
    for (int s = 0; s < kStreams; ++s) {
      const int j_lo = t_lo > s ? (t_lo - s + 7) >> 3 : 0, j_hi = t_hi > s ? (t_hi - s + 7) >> 3 : 0;
      for (int j = j_lo; j < j_hi; j += CHUNK, ++n_chunk) {
        const int tiles = min(CHUNK, j_hi - j);
        const uint32_t m = c0g + n_chunk, st = m % kStages;
        if (n_chunk >= kStages) tc_wait(tc, &sh->stage_free[st], m / kStages - 1, 8u);  // the stage's last chunk has been used up
        if (lane == 0) {
          const uint32_t bar = tc05::smem_u32(&sh->full[st]);
          tc05::mbar_arrive_expect_tx(bar, (uint32_t)(tiles * TB));
          tc05::bulk_g2s(tc05::smem_u32(tc.stages + (size_t)st * kStageBytes), body + (size_t)s * p.geom.stream_stride + (size_t)j * TB,
                         (uint32_t)(tiles * TB), bar);
        }
        __syncwarp();
      }
    }
  } else if (warp == kWarpMmaS) {
    // ---- score MMAs: S[token, head] = A_K . Q''^T once the block's K operand is in tensor memory.  The K
    //      operand and the score accumulators belong to the block's warpgroup, which has finished with both
    //      (its previous block's scores read, its softmax done) before it writes the next K operand. ----
    const uint64_t q_desc = tc05::smem_desc(tc05::smem_u32(tc.q_operand), 128, 2048);  // + 16 per k-step (256 bytes)
    tc_walk<CHUNK>(t_lo, t_hi, [&](int, int, int, int) {},
        [&](int i, int, int, int, int, int, bool) {
          const uint32_t n = g0 + i, wg = n % kTcGroups, use = n / kTcGroups;
          tc_wait(tc, &sh->ak_full[wg], use, 32u);
          __syncwarp();
          tc05::fence_after_sync();
          const uint32_t d_s = tb + kTmemDS + 16 * wg, a_k = tb + kTmemAK + 64 * wg;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) tc05::mma_f16_ts_elect(d_s, a_k + 8 * ks, q_desc + 16 * ks, idesc_qk, ks > 0 ? 1u : 0u);
          tc05::mma_commit_elect(tc05::smem_u32(&sh->bar_s[wg]));
        });
  } else if (warp >= kWarpMmaO) {
    // ---- output MMAs: O^T[channel, head] += A_V . w, one per live tile, into the accumulators of the block's
    //      warpgroup.  Two warps take alternate blocks: the blocks of different warpgroups do not depend on one
    //      another, and one warp issuing in block order holds every block behind the slowest softmax. ----
    const uint32_t w_base = tc05::smem_u32(tc.wbuf);
    const uint32_t mine = (uint32_t)(warp - kWarpMmaO);
    tc_walk<CHUNK>(t_lo, t_hi, [&](int, int, int, int) {},
        [&](int i, int, int, int, int, int nv, bool) {
          const uint32_t n = g0 + i, wg = n % kTcGroups, use = n / kTcGroups;
          if ((n & 1u) != mine) return;
          tc_wait(tc, &sh->av_full[wg], use, 64u);
          tc_wait(tc, &sh->w_full[wg], use, 128u);
          __syncwarp();
          tc05::fence_after_sync();
          const uint32_t fresh = *reinterpret_cast<volatile int *>(&sh->pv_fresh[wg]) != 0 ? 1u : 0u;
          const uint64_t w_desc = tc05::smem_desc(w_base + kWBufBytes * wg, 128, 2048);  // + 16 per tile (256 bytes) in the address field
          const uint32_t d_o = tb + kTmemDO + 16 * wg, a_v = tb + kTmemAV + 64 * wg;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (j < nv) tc05::mma_f16_ts_elect(d_o, a_v + 8 * j, w_desc + 16 * j, idesc_pv, (fresh && j == 0) ? 0u : 1u);
          tc05::mma_commit_elect(tc05::smem_u32(&sh->bar_o[wg]));
        });
  } else if (warp < kWarpCopy) {
    // ---- a block warpgroup: every third block, through all its steps.  Thread tw writes token row tw of A_K
    //      (the score MMAs start), then channel row tw of A_V, then turns the block's scores into weights. ----
    const uint32_t sw = (uint32_t)warp >> 2;   // this warpgroup: owns the blocks with n mod 3 == sw
    float2 mu2[4], sumq2[4], m2[4], l2[4], zs2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      mu2[j] = make_float2(ldexpf(1.0f, 24 - 14 + (int)s_stat[2 * j]), ldexpf(1.0f, 24 - 14 + (int)s_stat[2 * j + 1]));
      sumq2[j] = make_float2(s_stat[8 + 2 * j], s_stat[8 + 2 * j + 1]);
      m2[j] = make_float2(kNegBig, kNegBig);
      l2[j] = zs2[j] = make_float2(0.f, 0.f);
    }
    const float sigma_u = sigma16 * ldexpf(1.0f, F::SIGMA_LOG2);
    // the weight of this thread's token row in the output MMA carries the row's code position
    const float w_unit = ldexpf(1.0f, kEPV - F::pos(F::field(my_row))) / sigma_u;
    // The tensor core adds into its fp32 accumulators without rounding to nearest, and the sums of codes
    // times weights are all of one sign: left to grow over thousands of MMAs the loss shows in the output,
    // which is the small difference of that sum and the zero-point sum.  So every kEpochBlocks blocks the
    // accumulators of this thread's channel move into registers (ov) and the tensor-memory sums restart.
    constexpr int kEpochBlocks = 16;
    float ov[8];
#pragma unroll
    for (int h = 0; h < 8; ++h) ov[h] = 0.f;
    bool fresh = true;       // the tensor-memory accumulators hold nothing yet
    int since = 0;
    int mine_last = -1;      // last block (segment-local index) this warpgroup has handed to the output MMA
    int o_seen = -1;         // last such block whose output MMAs are known complete
    const uint32_t tDO = tb + kTmemDO + 16 * sw + t_lane, tDS = tb + kTmemDS + 16 * sw + t_lane;
    auto wait_o = [&](int blk) {  // output MMAs of this warpgroup's block blk (and its earlier ones) are complete
      if (blk >= 0 && o_seen < blk) {
        tc_wait(tc, &sh->bar_o[sw], (g0 + blk) / kTcGroups, 4u);
        tc05::fence_after_sync();
        o_seen = blk;
      }
    };
    tc_walk<CHUNK>(t_lo, t_hi, [&](int, int, int, int) {},
        [&](int i, int chunk, int s, int j0, int sb, int nv, bool) {
          const uint32_t n = g0 + i;
          if (n % kTcGroups != sw) return;
          const uint32_t b = sw, use = n / kTcGroups, st = (c0g + chunk) % kStages;
          tc_wait(tc, &sh->full[st], (c0g + chunk) / kStages, 1u);
          {  // ---- K: this thread's token row ----
            const uint8_t *kp = tc.stages + (size_t)st * kStageBytes + (sb + my_tile) * TB + my_row * ROW_BYTES;
            constexpr int HALF_CHUNKS = ROW_BYTES / 32;  // 16-byte chunks per half row
            uint4 raw[2 * HALF_CHUNKS];
#pragma unroll
            for (int c = 0; c < 2 * HALF_CHUNKS; ++c) raw[c] = *reinterpret_cast<const uint4 *>(kp + c * 16);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t r[32];
#pragma unroll
              for (int c = 0; c < HALF_CHUNKS; ++c) {
                const uint4 v = raw[half * HALF_CHUNKS + c];
                const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) F::extract(w4[e], r + (4 * c + e) * (32 / (4 * HALF_CHUNKS)));
              }
              tc05::tmem_st32(tb + kTmemAK + 64 * b + t_lane + 32 * half, r);
            }
            tc05::wait_st();
            tc05::fence_before_sync();
            warp_arrive(&sh->ak_full[b], lane);
          }
          wait_o(mine_last);  // the output MMAs of this warpgroup's last block have read its V operand and weights
          {  // ---- V: this thread's channel row ----
            const uint8_t *vp = tc.stages + (size_t)st * kStageBytes + sb * TB + v_part_offset(BITS) + tw * CH_BYTES;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t r[32];
#pragma unroll
              for (int t4 = 0; t4 < 4; ++t4) {
                const int t8 = 4 * half + t4;
                if constexpr (BITS == 2) {
                  F::extract(*reinterpret_cast<const uint32_t *>(vp + t8 * TB), r + 8 * t4);
                } else {
                  const uint2 v = *reinterpret_cast<const uint2 *>(vp + t8 * TB);
                  F::extract(v.x, r + 8 * t4);
                  F::extract(v.y, r + 8 * t4 + 4);
                }
              }
              tc05::tmem_st32(tb + kTmemAV + 64 * b + t_lane + 32 * half, r);
            }
            tc05::wait_st();
            tc05::fence_before_sync();
            warp_arrive(&sh->av_full[b], lane);
          }
          const uint8_t *blk = tc.stages + (size_t)st * kStageBytes + sb * TB;
          // token row (my_tile, my_row) of the block is token 16 (s + 8 (j0 + my_tile)) + my_row of the body
          const bool alive = my_tile < nv && ((s + 8 * (j0 + my_tile)) * 16 + my_row) < p.n_body;
          float4 meta = *reinterpret_cast<const float4 *>(blk + my_tile * TB + meta_offset(BITS) + my_row * 16);  // S_K Z_K S_V Z_V
          if (!alive) meta = make_float4(0.f, 0.f, 0.f, 0.f);  // a dead row holds arbitrary bytes
          warp_arrive(&sh->stage_free[st], lane);  // K, V and metadata of the block are in registers / tensor memory
          tc_wait(tc, &sh->bar_s[b], use, 2u);
          tc05::fence_after_sync();
          uint32_t sraw[16];
          tc05::tmem_ld16(tDS, sraw);
          tc05::wait_ld();
          tc05::fence_before_sync();
          float2 dot[4], a2[4], arg[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            dot[j] = __fadd2_rn(make_float2(__uint_as_float(sraw[2 * j]), __uint_as_float(sraw[2 * j + 1])),
                                make_float2(__uint_as_float(sraw[8 + 2 * j]), __uint_as_float(sraw[8 + 2 * j + 1])));
            a2[j] = __fmul2_rn(mu2[j], make_float2(meta.x, meta.x));
            const float2 bb = __ffma2_rn(make_float2(meta.y, meta.y), sumq2[j], make_float2(-m2[j].x, -m2[j].y));
            arg[j] = __ffma2_rn(a2[j], dot[j], bb);
            if (!alive) arg[j] = make_float2(-INFINITY, -INFINITY);
          }
          const float amax = fmaxf(fmaxf(fmaxf(arg[0].x, arg[0].y), fmaxf(arg[1].x, arg[1].y)),
                                   fmaxf(fmaxf(arg[2].x, arg[2].y), fmaxf(arg[3].x, arg[3].y)));
          if (swg_any(sw, amax > kTcMaxAhead)) {
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
              if (lane == 0) { sh->wmax[sw][quad][2 * j] = mx; sh->wmax[sw][quad][2 * j + 1] = my; }
            }
            swg_sync(sw);
            float f[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              float bx = kNegBig, by = kNegBig;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                bx = fmaxf(bx, sh->wmax[sw][q][2 * j]);
                by = fmaxf(by, sh->wmax[sw][q][2 * j + 1]);
              }
              const float nx = fmaxf(m2[j].x, bx + kTcHeadroom), ny = fmaxf(m2[j].y, by + kTcHeadroom);
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
            if (!fresh) {  // the output accumulators of channel row tw, once this warpgroup's output MMAs are complete
              wait_o(mine_last);
              uint32_t o[16];
              tc05::tmem_ld16(tDO, o);
              tc05::wait_ld();
#pragma unroll
              for (int h = 0; h < 8; ++h) {
                o[h] = __float_as_uint(__uint_as_float(o[h]) * f[h]);
                o[8 + h] = __float_as_uint(__uint_as_float(o[8 + h]) * f[h]);
              }
              tc05::tmem_st16(tDO, o);
              tc05::wait_st();
            }
            swg_sync(sw);  // wmax may be rewritten by the next move
          }
          if (since == kEpochBlocks) {  // move the accumulators into registers; the next output MMA starts afresh
            wait_o(mine_last);
            uint32_t o[16];
            tc05::tmem_ld16(tDO, o);
            tc05::wait_ld();
#pragma unroll
            for (int h = 0; h < 8; ++h) ov[h] += fmaf(__uint_as_float(o[8 + h]), 0x1p-11f, __uint_as_float(o[h]));
            fresh = true;
            since = 0;
          }

          // ---- probabilities and weights: w = p * S_V goes to the output MMA as fp16 hi + lo (22 bits), in
          //      columns h and 8 + h of the B operand; the sums take p itself ----
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
          wait_o(mine_last);  // the output MMAs that read this weight buffer are complete
          uint8_t *wbuf = tc.wbuf + kWBufBytes * b;
          *reinterpret_cast<uint4 *>(wbuf + tw * 16) = make_uint4(whi[0], whi[1], whi[2], whi[3]);
          *reinterpret_cast<uint4 *>(wbuf + 2048 + tw * 16) = make_uint4(wlo[0], wlo[1], wlo[2], wlo[3]);
          if (tw == 0) sh->pv_fresh[b] = fresh ? 1 : 0;
          tc05::fence_async_smem();
          tc05::fence_before_sync();
          warp_arrive(&sh->w_full[b], lane);
          mine_last = i;
          fresh = false;
          ++since;
        });
    // ---- this warpgroup's partial: (m, l, o[128]) per head ----
    if (mine_last >= 0) {
      wait_o(mine_last);
      uint32_t o[16];
      tc05::tmem_ld16(tDO, o);
      tc05::wait_ld();
#pragma unroll
      for (int h = 0; h < 8; ++h) ov[h] += fmaf(__uint_as_float(o[8 + h]), 0x1p-11f, __uint_as_float(o[h]));
    }
    const float f_out = ldexpf(sigma_u, 24 - kEPV);
    // sums over the 128 token rows
    float red[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      red[2 * j] = l2[j].x; red[2 * j + 1] = l2[j].y;
      red[8 + 2 * j] = zs2[j].x; red[8 + 2 * j + 1] = zs2[j].y;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) {
#pragma unroll
      for (int o = 16; o; o >>= 1) red[k] += __shfl_xor_sync(0xffffffffu, red[k], o);
    }
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < 16; ++k) sh->sums[sw][quad][k] = red[k];
    }
    tc05::fence_before_sync();
    swg_sync(sw);
    const int slot = slot0 + (int)sw;
    float (*po)[kHeadDim] = reinterpret_cast<float (*)[kHeadDim]>(tc.part_o + (size_t)slot * kMaxGroup * kHeadDim);
#pragma unroll
    for (int h = 0; h < 8; ++h) {
      const float zs = sh->sums[sw][0][8 + h] + sh->sums[sw][1][8 + h] + sh->sums[sw][2][8 + h] + sh->sums[sw][3][8 + h];
      po[h][tw] = fmaf(ov[h], f_out, zs);
    }
    if (tw == 0) {
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        s_m[slot * 8 + h] = (h & 1) ? m2[h >> 1].y : m2[h >> 1].x;
        s_l[slot * 8 + h] = sh->sums[sw][0][h] + sh->sums[sw][1][h] + sh->sums[sw][2][h] + sh->sums[sw][3][h];
      }
    }
  }
}

}  // namespace pmkvq

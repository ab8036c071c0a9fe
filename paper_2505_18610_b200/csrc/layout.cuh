// Tile layout of the packed KV cache in HBM.
//
// A tile holds 16 consecutive tokens of one (batch, kv_head) slice, K and V together:
//
//   [ K codes : 256*b bytes ][ V codes : 256*b bytes ][ metadata : 256 bytes ]      b = bit width
//
// so tile_bytes(b) = 512*b + 256 = 16 tokens * 2 * (16*b code bytes + 4 scale + 4 zero): the bytes
// the budget accounting of the progressive policy (Sec. 3.1) charges, nothing more.
//
// The arrangement of the codes inside a tile follows the unit that consumes them in the attention kernel.
// A cache is created for one of two attention paths: warp-level MMAs (every width uses lane-owned tiles) or
// tensor memory (the 4- and 2-bit body uses row tiles; 16 and 8 bit stay lane-owned).
//
// --- "lane-owned" tiles, read by warp-level MMAs from registers ---------------------------------------
// The 32 lanes of a warp own 16-byte chunks, chunk q of lane l at byte (q*32 + l)*16, so a warp reads a
// tile with fully coalesced 128-bit loads and every lane gets exactly the codes its fragments need, with
// no shuffle.  With lane = 4*g + tig:
//
//   K part: lane (g,tig) owns tokens {g, g+8} and channels {8*W + 2*tig + h : W=0..15, h=0,1}.
//           The two 16-bit halves of a 32-bit word are two channels (h) of ONE token: exactly the
//           k-pair of an m16n8k16 B fragment for S = Q K^T (k = channel, n = token).
//   V part: lane (g,tig) owns tokens {2*tig + 8*r + h : r=0,1, h=0,1} and channels {8*J + g : J=0..15}.
//           The two halves of a word are two consecutive tokens (h) of ONE channel: the k-pair of an
//           m16n8k16 A fragment for O^T = V^T P^T (m = channel, k = token).
//
// In both parts a 16-bit half-word holds n = 16/b codes of one token: index W (or J) = w*n + j sits
// in lane-word lw = r*b + w, at bits [j*b, j*b + b) of half h.
//
// Metadata: for tig = 0..3 a 64-byte record {S_K[4], Z_K[4], S_V[4], Z_V[4]} of the four tokens
// {2tig, 2tig+1, 8+2tig, 9+2tig} a lane needs for its score / probability fragments.
//
// --- "row" tiles (4 and 2 bit of a tensor-memory cache), read by tcgen05.mma through tensor memory ----
// The A operand of the MMAs lives in tensor memory, where a thread writes one lane (one matrix row):
// a token's row of K^T-side codes for the scores, a channel's row of V codes for the output.  So
//
//   K part: token row r takes 16*b contiguous bytes at r*16*b; its 32-bit word w holds the 32/b channels
//           (32/b)*w + 2*f + h at bits [16*h + b*f, +b): the two halves of a word are adjacent channels,
//           the k-pair of a 16-bit tensor-memory column.
//   V part: channel c takes 2*b contiguous bytes at c*2*b; its word w holds the tokens (32/b)*w + 2*f + h
//           of the tile at bits [16*h + b*f, +b).
//   Metadata: token row r has the record {S_K, Z_K, S_V, Z_V} at r*16.
//
// In both layouts, going from 2b to b bits merges two adjacent words into one (Eq. 3 applied per field).
//
// --- the body of a slice: eight interleaved streams ---------------------------------------------------
// Body tile i of a slice lives in stream i mod 8 at index i div 8: byte offset
// (i & 7) * stream_stride + (i >> 3) * tile_bytes(b).  Eight consecutive tiles (128 tokens, one MMA
// block) sit at the same index of the eight streams, and the in-place progressive reduce can compact
// every stream of every slice independently (outputs never run ahead of inputs inside a stream).
#pragma once
#include <cstddef>
#include <cstdint>

#if defined(__CUDACC__)
#define PMKVQ_HD __host__ __device__ __forceinline__
#else
#define PMKVQ_HD inline
#endif

namespace pmkvq {

constexpr int kHeadDim = 128;
constexpr int kTileTokens = 16;
constexpr int kStreams = 8;       // interleaved streams of a slice's body
constexpr int kBlockTiles = 8;    // tiles of one 128-token MMA block (one per stream)

PMKVQ_HD constexpr int code_part_bytes(int bits) { return 256 * bits; }
PMKVQ_HD constexpr int tile_bytes(int bits) { return 512 * bits + 256; }
PMKVQ_HD constexpr int v_part_offset(int bits) { return 256 * bits; }
PMKVQ_HD constexpr int meta_offset(int bits) { return 512 * bits; }
PMKVQ_HD constexpr bool row_layout(int bits, bool rows) { return rows && bits <= 4; }

// Byte offset of body tile i inside the body of a slice.
PMKVQ_HD size_t body_tile_offset(int i, int bits, size_t stream_stride) {
  return (size_t)(i & (kStreams - 1)) * stream_stride + (size_t)(i >> 3) * (size_t)tile_bytes(bits);
}

// Lane-owned tiles: byte offset (inside the K or V part) of the half-word that holds lane-element
// (lane, r, idx, h) and the bit position of the code inside that half-word.  idx is W (K part) or J (V part).
PMKVQ_HD void lane_slot(int bits, int lane, int r, int idx, int h, int &byte_off, int &bit_off) {
  const int n = 16 / bits;
  const int w = idx / n, j = idx % n;
  const int lw = r * bits + w;
  byte_off = ((lw >> 2) * 32 + lane) * 16 + (lw & 3) * 4 + h * 2;
  bit_off = j * bits;
}

// Row tiles: element `idx` (a channel of a token row, or a token of a channel row) of a row of
// `row_bytes` bytes: half-word byte offset inside the row and bit position inside the half-word.
PMKVQ_HD void row_slot(int bits, int idx, int &byte_off, int &bit_off) {
  const int per_word = 32 / bits;
  const int w = idx / per_word, i = idx % per_word;
  byte_off = 4 * w + 2 * (i & 1);
  bit_off = bits * (i >> 1);
}

// K code of (token row 0..15, channel 0..127): half-word byte offset inside the K part, bit offset
PMKVQ_HD void k_slot(int bits, bool rows, int row, int ch, int &byte_off, int &bit_off) {
  if (row_layout(bits, rows)) {
    row_slot(bits, ch, byte_off, bit_off);
    byte_off += row * 16 * bits;
    return;
  }
  const int g = row & 7, r = row >> 3;
  const int W = ch >> 3, tig = (ch & 7) >> 1, h = ch & 1;
  lane_slot(bits, g * 4 + tig, r, W, h, byte_off, bit_off);
}

// V code of (token row 0..15, channel 0..127)
PMKVQ_HD void v_slot(int bits, bool rows, int row, int ch, int &byte_off, int &bit_off) {
  if (row_layout(bits, rows)) {
    row_slot(bits, row, byte_off, bit_off);
    byte_off += ch * 2 * bits;
    return;
  }
  const int h = row & 1, tig = (row & 7) >> 1, r = row >> 3;
  const int g = ch & 7, J = ch >> 3;
  lane_slot(bits, g * 4 + tig, r, J, h, byte_off, bit_off);
}

// Byte offset inside the metadata block of kind (0 S_K, 1 Z_K, 2 S_V, 3 Z_V) of token row.
PMKVQ_HD int meta_slot(int bits, bool rows, int kind, int row) {
  if (row_layout(bits, rows)) return row * 16 + kind * 4;
  const int tig = (row & 7) >> 1;
  const int i = (row >> 3) * 2 + (row & 1);
  return tig * 64 + kind * 16 + i * 4;
}

// Eq. 3, one step 2b -> b on one code.  The product needs the full 32 unsigned bits at b = 8.
PMKVQ_HD uint32_t shift_step(uint32_t c, int b) {
  const uint32_t mult = (1u << (2 * b)) - (1u << b) + 1u;
  return (mult * (c + (1u << (b - 1)))) >> (3 * b);
}

// How a halving 2b -> b treats codes and metadata (Sec. 4.4.1 compares the three):
//   kShiftEquivalent  Eq. 3,          S_b = (2^b+1) S_2b, Z unchanged            (the method)
//   kShiftDirect      X_b = X_2b >> b, S_b = (2^b+1) S_2b, Z unchanged            (ablation 1)
//   kShiftModified    X_b = X_2b >> b, S_b = 2^b S_2b,     Z_b = Z_2b + (S_b - S_2b)/2  (ablation 2)
enum ShiftVariant { kShiftEquivalent = 0, kShiftDirect = 1, kShiftModified = 2 };

// 16-bit code -> `bits`-bit code through the chain 16 -> 8 -> 4 -> 2.
PMKVQ_HD uint32_t shift_chain(uint32_t c16, int bits, int variant = kShiftEquivalent) {
  if (variant != kShiftEquivalent) return c16 >> (16 - bits);  // b right shifts per halving add up
  uint32_t c = c16;
  for (int w = 8; w >= bits; w >>= 1) c = shift_step(c, w);
  return c;
}

}  // namespace pmkvq

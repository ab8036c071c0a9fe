// C ABI of the PM-KVQ decode hot path: host-side cache state machine (progressive policy of
// Sec. 3.1), arena layout, kernel launches, and the slice export used for bit-exact comparison.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <memory>
#include <new>
#include <vector>

#include "../../include/pmkvq.h"
#include "kernels_attn.cuh"
#include "kernels_cache.cuh"
#include "kernels_calib.cuh"
#include "layout.cuh"

using namespace pmkvq;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxCtas = 1024;      // upper bound on the attention grid (sizes the partials workspace)
// Fixed cost of one more segment (set-up, warp merge, publish, its share of the slice combine), in
// body tiles of each width: about 12 us at the measured per-SM tile rates.
inline int segment_cost_tiles(int bits) { return bits == 16 ? 48 : bits == 8 ? 96 : bits == 4 ? 176 : 160; }
constexpr int kMinUnitsPerCta = 32;  // do not cut the work finer than two tiles per warp

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool valid_bits(int b) { return b == 2 || b == 4 || b == 8 || b == 16; }

struct Layer {
  int fbit = 16;
  int cur_bits = 16;
  int n_tokens = 0;
  uint64_t budget = 0;
  size_t offset = 0;        // of the first slice inside the arena
  size_t slice_stride = 0;
  size_t stream_stride = 0; // bytes of each of the body's eight interleaved streams (capacity of a stream)
};

}  // namespace

struct pmkvq_cache {
  int layers, q_heads, kv_heads, batch, max_tokens, group, n_slices;
  int n_sink, window, evict_chunk, count_metadata, auto_reduce, shift_variant, rows;
  float sm_scale;
  uint8_t *arena;
  size_t arena_bytes;
  // arena sections
  size_t off_lambda, off_inv_lambda, off_vmax, off_tickets, off_partials, partial_bytes, off_geoms;  // scratch is per block
  size_t off_error;  // one word: bits set by a device-side wait that ran out
  int sink_tiles, ring_tiles, user_ctas;
  int resident_ctas[4];  // one wave of the attention kernel at body width 16, 8, 4, 2
  int resident_fused;    // one wave of the all-blocks attention kernel
  uint64_t launches = 0;  // kernels launched so far
  std::vector<Layer> L;

  // ---- policy arithmetic (Sec. 3.1) ----
  int tokbytes(int bits) const { return 16 * bits + (count_metadata ? 8 : 0); }
  int sink_at(int n) const { return std::min(n, n_sink); }
  int body_at(int n) const {
    const int excess = n - n_sink - window;
    return excess <= 0 ? 0 : excess / evict_chunk * evict_chunk;
  }
  uint64_t bytes_at(int n, int bits) const {
    const uint64_t nb = body_at(n), n16 = n - nb;
    return 2ull * n_slices * (n16 * tokbytes(16) + nb * tokbytes(bits));
  }
  uint64_t default_budget(int fbit) const {
    uint64_t best = 0;
    for (int n = std::max(0, max_tokens - evict_chunk + 1); n <= max_tokens; ++n) best = std::max(best, bytes_at(n, fbit));
    return best;
  }
  LayerGeom geom(const Layer &l) const {
    LayerGeom g;
    g.base = arena + l.offset;
    g.slice_stride = l.slice_stride;
    g.ring_off = (size_t)sink_tiles * tile_bytes(16);
    g.body_off = g.ring_off + (size_t)ring_tiles * tile_bytes(16);
    g.stream_stride = l.stream_stride;
    g.n_sink = n_sink;
    g.ring_tokens = ring_tiles * 16;
    g.shift_variant = shift_variant;
    g.rows = rows;
    return g;
  }
};

namespace {

bool check_config(const pmkvq_config *c) {
  if (!c) return false;
  if (c->layers <= 0 || c->q_heads <= 0 || c->kv_heads <= 0 || c->batch <= 0 || c->max_tokens <= 0) return false;
  if (c->head_dim != kHeadDim) return false;
  if (c->q_heads % c->kv_heads) return false;
  const int g = c->q_heads / c->kv_heads;
  if (g < 1 || g > kMaxGroup) return false;
  if (!c->fbit) return false;
  for (int i = 0; i < c->layers; ++i)
    if (!valid_bits(c->fbit[i])) return false;
  if (c->n_sink < 0 || c->window < 0 || c->evict_chunk < 1) return false;
  if (c->shift_variant < 0 || c->shift_variant > 2) return false;
  if (c->attention_path < 0 || c->attention_path > 1) return false;
  if ((int64_t)c->n_sink + c->window + c->evict_chunk > (1 << 24)) return false;
  if ((int64_t)c->batch * c->kv_heads > 65535) return false;
  if (c->lambda) {
    const size_t n = (size_t)c->layers * c->kv_heads * kHeadDim;
    for (size_t i = 0; i < n; ++i)
      if (!(c->lambda[i] > 0.0f) || !std::isfinite(c->lambda[i])) return false;
  }
  if (!(c->sm_scale >= 0.0f) || !std::isfinite(c->sm_scale)) return false;
  return true;
}

// Fills everything of the handle that depends only on the configuration; returns the arena size.
size_t plan(pmkvq_cache &k, const pmkvq_config *c) {
  k.layers = c->layers; k.q_heads = c->q_heads; k.kv_heads = c->kv_heads; k.batch = c->batch;
  k.max_tokens = c->max_tokens; k.group = c->q_heads / c->kv_heads; k.n_slices = c->batch * c->kv_heads;
  k.n_sink = c->n_sink; k.window = c->window; k.evict_chunk = c->evict_chunk;
  k.count_metadata = c->count_metadata ? 1 : 0; k.auto_reduce = c->auto_reduce ? 1 : 0;
  k.shift_variant = c->shift_variant;
  k.rows = c->attention_path == 1 ? 1 : 0;
  k.sm_scale = c->sm_scale > 0.0f ? c->sm_scale : 1.0f / std::sqrt((float)kHeadDim);
  k.sink_tiles = (k.n_sink + 15) / 16;
  k.ring_tiles = std::max(1, (k.window + k.evict_chunk - 1 + 15) / 16 + 1);
  k.user_ctas = 0;

  size_t off = 0;
  const size_t lam_bytes = (size_t)k.layers * k.kv_heads * kHeadDim * sizeof(float);
  k.off_lambda = off; off = align_up(off + lam_bytes, kAlign);
  k.off_inv_lambda = off; off = align_up(off + lam_bytes, kAlign);
  k.off_vmax = off; off = align_up(off + (size_t)k.layers * k.n_slices * sizeof(unsigned), kAlign);
  // tickets and split-K partials exist once per block: one launch computes the attention of all blocks
  k.off_tickets = off; off = align_up(off + (size_t)k.layers * k.n_slices * sizeof(unsigned), kAlign);
  k.partial_bytes = align_up(((size_t)kMaxCtas + (size_t)k.n_slices) * kMaxGroup * kPartialStride * sizeof(float), kAlign);
  k.off_partials = off; off = align_up(off + k.partial_bytes * k.layers, kAlign);
  k.off_geoms = off; off = align_up(off + (size_t)k.layers * sizeof(LayerGeom), kAlign);
  k.off_error = off; off = align_up(off + sizeof(unsigned), kAlign);

  k.L.assign(k.layers, Layer());
  for (int i = 0; i < k.layers; ++i) {
    Layer &l = k.L[i];
    l.fbit = c->fbit[i];
    l.budget = c->budget_bytes ? c->budget_bytes[i] : k.default_budget(l.fbit);
    // body capacity: the most tiles the policy can ever ask for at any width of the chain, dealt out
    // over the eight streams (tile i sits in stream i mod 8)
    size_t cap = 0;
    for (int b = 16; b >= l.fbit; b >>= 1) {
      int lo = 0, hi = k.max_tokens;  // largest n with bytes_at(n, b) <= budget (bytes_at is monotone enough
      while (lo < hi) {               // for a bisection on the chunk-aligned body count below)
        const int mid = (lo + hi + 1) / 2;
        // the worst window phase for a given body count is right before the next chunk leaves
        if (k.bytes_at(mid, b) <= l.budget) lo = mid; else hi = mid - 1;
      }
      int nb = 0;
      for (int n = std::max(0, lo - 2 * k.evict_chunk); n <= std::min(k.max_tokens, lo + 2 * k.evict_chunk); ++n)
        if (k.bytes_at(n, b) <= l.budget) nb = std::max(nb, k.body_at(n));
      const size_t tiles = (size_t)((nb + 15) / 16);
      cap = std::max(cap, (tiles + kStreams - 1) / kStreams * tile_bytes(b));
    }
    l.stream_stride = align_up(cap, kAlign);
    l.slice_stride = align_up((size_t)(k.sink_tiles + k.ring_tiles) * tile_bytes(16) + l.stream_stride * kStreams, kAlign);
    l.offset = off;
    off = align_up(off + l.slice_stride * k.n_slices, kAlign);
  }
  return off;
}

template <int B>
cudaError_t launch_reduce(const LayerGeom &g, int n_slices, int n_tiles, cudaStream_t st, uint64_t &launches) {
  // one CTA per (stream, slice): the streams compact in place independently of one another
  reduce_stream_kernel<B><<<dim3(kStreams, (unsigned)n_slices), reduce_warps<B>() * 32, 0, st>>>(g, n_tiles);
  ++launches;
  return cudaGetLastError();
}

template <int BITS, bool ROWS>
cudaError_t attention_setup_one(int &resident, int sms) {
  cudaError_t e = cudaFuncSetAttribute(decode_attn_splitk_kernel<BITS, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       attn_smem_bytes<BITS, ROWS>());
  int per_sm = 0;
  if (e == cudaSuccess)
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_attn_splitk_kernel<BITS, ROWS>, kAttnThreads,
                                                      attn_smem_bytes<BITS, ROWS>());
  resident = std::min(kMaxCtas, std::max(1, per_sm) * sms);
  return e;
}

template <bool ROWS>
cudaError_t attention_setup_path(pmkvq_cache *k, int sms) {
  cudaError_t e = attention_setup_one<16, ROWS>(k->resident_ctas[0], sms);
  if (e == cudaSuccess) e = attention_setup_one<8, ROWS>(k->resident_ctas[1], sms);
  if (e == cudaSuccess) e = attention_setup_one<4, ROWS>(k->resident_ctas[2], sms);
  if (e == cudaSuccess) e = attention_setup_one<2, ROWS>(k->resident_ctas[3], sms);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(decode_attn_fused_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             attn_fused_smem_bytes<ROWS>());
  int per_sm = 0;
  if (e == cudaSuccess)
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_attn_fused_kernel<ROWS>, kAttnThreads,
                                                      attn_fused_smem_bytes<ROWS>());
  k->resident_fused = std::min(kMaxCtas, std::max(1, per_sm) * sms);
  return e;
}

// Dynamic shared memory opt-in and the size of one wave of resident CTAs, per body width.
cudaError_t attention_setup(pmkvq_cache *k) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = k->rows ? attention_setup_path<true>(k, sms) : attention_setup_path<false>(k, sms);
  return e;
}

pmkvq_status do_reduce(pmkvq_cache *k, int layer, cudaStream_t st) {
  Layer &l = k->L[layer];
  const int b = l.cur_bits / 2;
  const int n_body = k->body_at(l.n_tokens);
  const int n_tiles = (n_body + 15) / 16;
  const LayerGeom g = k->geom(l);
  cudaError_t e = cudaSuccess;
  if (n_tiles > 0) {
    if (b == 8) e = launch_reduce<8>(g, k->n_slices, n_tiles, st, k->launches);
    else if (b == 4) e = launch_reduce<4>(g, k->n_slices, n_tiles, st, k->launches);
    else e = launch_reduce<2>(g, k->n_slices, n_tiles, st, k->launches);
  }
  if (e != cudaSuccess) return PMKVQ_ERR_CUDA;
  l.cur_bits = b;
  return PMKVQ_OK;
}

}  // namespace

// ---- scratch of pmkvq_decode_attention_static: lives in the library image, one copy per GPU ----
constexpr size_t kStaticTicketBytes = 16 * 1024;          // 4096 slice tickets
constexpr size_t kStaticScratchBytes = 4u * 1024 * 1024;  // tickets + split-K partials
constexpr size_t kStaticPartialSlots =
    (kStaticScratchBytes - kStaticTicketBytes) / (kMaxGroup * kPartialStride * sizeof(float));
constexpr int kMaxDevices = 64;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static void *g_static_scratch_addr[kMaxDevices];  // device address of the array on each GPU, looked up once

// Device address of g_static_scratch on the current GPU (in host code the array's name is only a
// handle for the runtime, not something a kernel can be given).
static cudaError_t static_scratch_address(unsigned char **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_static_scratch_addr[dev]) {
    void *ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    g_static_scratch_addr[dev] = ptr;
  }
  *out = static_cast<unsigned char *>(g_static_scratch_addr[dev]);
  return cudaSuccess;
}

extern "C" {

size_t pmkvq_arena_bytes_required(const pmkvq_config *cfg) {
  if (!check_config(cfg)) return 0;
  try {
    pmkvq_cache tmp{};
    return plan(tmp, cfg);
  } catch (...) {
    return 0;
  }
}

static pmkvq_status cache_create_impl(const pmkvq_config *cfg, pmkvq_cache **out) {
  if (!out || !check_config(cfg) || !cfg->d_arena) return PMKVQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cfg->d_arena) % kAlign) return PMKVQ_ERR_INVALID_ARG;
  std::unique_ptr<pmkvq_cache> owner(new (std::nothrow) pmkvq_cache{});  // released to the caller on success only
  pmkvq_cache *k = owner.get();
  if (!k) return PMKVQ_ERR_STATE;
  const size_t need = plan(*k, cfg);
  if (cfg->arena_bytes < need) return PMKVQ_ERR_ARENA_TOO_SMALL;
  k->arena = static_cast<uint8_t *>(cfg->d_arena);
  k->arena_bytes = cfg->arena_bytes;
  const size_t n_lam = (size_t)k->layers * k->kv_heads * kHeadDim;
  std::vector<float> lam(n_lam, 1.0f), inv(n_lam, 1.0f);
  if (cfg->lambda) {
    for (size_t i = 0; i < n_lam; ++i) {
      lam[i] = cfg->lambda[i];
      inv[i] = 1.0f / cfg->lambda[i];  // one IEEE fp32 division; Keys are multiplied by this (Eq. 9)
    }
  }
  cudaError_t e = cudaMemcpy(k->arena + k->off_lambda, lam.data(), n_lam * sizeof(float), cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(k->arena + k->off_inv_lambda, inv.data(), n_lam * sizeof(float), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(k->arena + k->off_vmax, 0, (size_t)k->layers * k->n_slices * sizeof(unsigned));
  if (e == cudaSuccess) e = cudaMemset(k->arena + k->off_tickets, 0, (size_t)k->layers * k->n_slices * sizeof(unsigned));
  if (e == cudaSuccess) e = cudaMemset(k->arena + k->off_error, 0, sizeof(unsigned));
  if (e == cudaSuccess) {
    std::vector<LayerGeom> geoms(k->layers);
    for (int i = 0; i < k->layers; ++i) geoms[i] = k->geom(k->L[i]);
    e = cudaMemcpy(k->arena + k->off_geoms, geoms.data(), geoms.size() * sizeof(LayerGeom), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = attention_setup(k);
  if (e != cudaSuccess) return PMKVQ_ERR_CUDA;
  *out = owner.release();
  return PMKVQ_OK;
}

pmkvq_status pmkvq_cache_create(const pmkvq_config *cfg, pmkvq_cache **out) {
  try {
    return cache_create_impl(cfg, out);
  } catch (...) {
    return PMKVQ_ERR_STATE;
  }
}

void pmkvq_cache_destroy(pmkvq_cache *cache) { delete cache; }

pmkvq_status pmkvq_progressive_reduce(pmkvq_cache *k, int32_t layer, void *stream) {
  if (!k || layer < 0 || layer >= k->layers) return PMKVQ_ERR_INVALID_ARG;
  if (k->L[layer].cur_bits <= k->L[layer].fbit) return PMKVQ_ERR_AT_FBIT;
  return do_reduce(k, layer, static_cast<cudaStream_t>(stream));
}

// Policy part of an append of n_new tokens to one block (Sec. 3.1), without side effects: capacity and
// budget tests; on PMKVQ_OK `n_reduce` is the number of halvings the budget asks for first.
static pmkvq_status append_check(const pmkvq_cache *k, int32_t layer, int32_t n_new, int &n_after_out, int &n_reduce_out) {
  const Layer &l = k->L[layer];
  const int64_t n_after64 = (int64_t)l.n_tokens + n_new;
  if (n_after64 > k->max_tokens) return PMKVQ_ERR_CAPACITY;
  const int n_after = (int)n_after64;
  int bits = l.cur_bits, n_reduce = 0;
  while (k->bytes_at(n_after, bits) > l.budget) {
    if (bits <= l.fbit) return PMKVQ_ERR_CAPACITY;
    bits >>= 1;
    ++n_reduce;
  }
  if (n_reduce && !k->auto_reduce) return PMKVQ_ERR_BUDGET_FULL;
  if ((size_t)(((k->body_at(n_after) + 15) / 16 + kStreams - 1) / kStreams) * tile_bytes(bits) > l.stream_stride)
    return PMKVQ_ERR_STATE;
  n_after_out = n_after;
  n_reduce_out = n_reduce;
  return PMKVQ_OK;
}

// The same, followed by the reduces.  On PMKVQ_OK the block can take the tokens.
static pmkvq_status append_prepare(pmkvq_cache *k, int32_t layer, int32_t n_new, cudaStream_t st, int &n_after_out) {
  int n_reduce = 0;
  const pmkvq_status c = append_check(k, layer, n_new, n_after_out, n_reduce);
  if (c != PMKVQ_OK) return c;
  for (int i = 0; i < n_reduce; ++i) {
    const pmkvq_status s = do_reduce(k, layer, st);
    if (s != PMKVQ_OK) return s;
  }
  return PMKVQ_OK;
}

pmkvq_status pmkvq_append(pmkvq_cache *k, int32_t layer, const void *d_K, const void *d_V, int32_t n_new,
                          void *stream) {
  if (!k || layer < 0 || layer >= k->layers || !d_K || !d_V || n_new <= 0) return PMKVQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_K) | reinterpret_cast<uintptr_t>(d_V)) & 7) return PMKVQ_ERR_INVALID_ARG;
  Layer &l = k->L[layer];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int n_after = 0;
  const pmkvq_status ps = append_prepare(k, layer, n_new, st, n_after);
  if (ps != PMKVQ_OK) return ps;
  const int new_body = k->body_at(n_after);
  const LayerGeom g = k->geom(l);
  const int n_old = l.n_tokens;
  const int old_win_start = k->sink_at(n_old) + k->body_at(n_old);
  const int new_win_start = k->sink_at(n_after) + new_body;
  // tokens already in the ring that now leave the window
  const int ev_first = std::max(old_win_start, k->n_sink);
  const int ev_last = std::min(new_win_start, n_old);
  const float *inv_lam = reinterpret_cast<const float *>(k->arena + k->off_inv_lambda) + (size_t)layer * k->kv_heads * kHeadDim;
  unsigned *vmax = reinterpret_cast<unsigned *>(k->arena + k->off_vmax) + (size_t)layer * k->n_slices;
  const int n_evict = std::max(0, ev_last - ev_first);
  // With window = 0 and chunked eviction the new token enters the body together with the chunk's other
  // tokens, possibly in one tile: they then go through separate launches (see append_decode_kernel).
  const bool shares_tile = k->window == 0 && k->evict_chunk > 1;
  if (n_new == 1 && !shares_tile) {
    // decode step: evictions and the new token in one launch (their ring slots cannot coincide)
    const long long warps = 2ll * (n_evict + 1) * k->n_slices;
    append_decode_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(
        static_cast<const uint16_t *>(d_K), static_cast<const uint16_t *>(d_V), inv_lam, vmax, g, k->n_slices, k->kv_heads,
        n_old, new_win_start, l.cur_bits, ev_first, n_evict);
    ++k->launches;
  } else {
    if (n_evict > 0) {
      const long long warps = 2ll * n_evict * k->n_slices;
      evict_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(g, k->n_slices, ev_first, n_evict, l.cur_bits);
      ++k->launches;
    }
    // new tokens that fill whole body tiles are written tile-wise, the rest (sink, ring, ragged ends) one by one
    const int j_lo = std::max(n_old, k->n_sink) - k->n_sink, j_hi = std::max(new_win_start, k->n_sink) - k->n_sink;
    const int tile_lo = (j_lo + 15) / 16, tile_hi = j_hi / 16;
    int skip_lo = n_old, skip_hi = n_old;  // absolute token range written tile-wise
    if (tile_hi > tile_lo) {
      skip_lo = k->n_sink + 16 * tile_lo;
      skip_hi = k->n_sink + 16 * tile_hi;
      const long long tw = 2ll * (tile_hi - tile_lo) * k->n_slices;
      append_tiles_kernel<<<(unsigned)((tw + 3) / 4), 128, 0, st>>>(static_cast<const uint16_t *>(d_K),
                                                                   static_cast<const uint16_t *>(d_V), inv_lam, vmax, g,
                                                                   k->n_slices, k->kv_heads, n_old, tile_lo,
                                                                   tile_hi - tile_lo, l.cur_bits);
      ++k->launches;
    }
    const int ranges[2][2] = {{n_old, skip_lo}, {skip_hi, n_after}};  // what is left, one token per warp
    for (int r = 0; r < 2; ++r) {
      const int cnt = ranges[r][1] - ranges[r][0];
      if (cnt <= 0) continue;
      const long long warps = 2ll * cnt * k->n_slices;
      append_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(static_cast<const uint16_t *>(d_K),
                                                                static_cast<const uint16_t *>(d_V), inv_lam, vmax, g, cnt,
                                                                k->n_slices, k->kv_heads, n_old, new_win_start, l.cur_bits,
                                                                ranges[r][0] - n_old);
      ++k->launches;
    }
  }
  if (cudaGetLastError() != cudaSuccess) return PMKVQ_ERR_CUDA;
  l.n_tokens = n_after;
  return PMKVQ_OK;
}

}  // extern "C"

// Everything of one attention launch except where its split-K scratch lives.
static pmkvq_status attn_params(pmkvq_cache *k, int32_t layer, const void *d_Q, float *d_out, AttnParams &p,
                                unsigned &n_ctas) {
  if (!k || layer < 0 || layer >= k->layers || !d_Q || !d_out) return PMKVQ_ERR_INVALID_ARG;
  const Layer &l = k->L[layer];
  if (l.n_tokens <= 0) return PMKVQ_ERR_INVALID_ARG;
  p.geom = k->geom(l);
  p.Q = static_cast<const uint16_t *>(d_Q);
  p.lambda = reinterpret_cast<const float *>(k->arena + k->off_lambda) + (size_t)layer * k->kv_heads * kHeadDim;
  p.vmax_bits = reinterpret_cast<const unsigned *>(k->arena + k->off_vmax) + (size_t)layer * k->n_slices;
  p.partials = nullptr;
  p.tickets = nullptr;
  p.out = d_out;
  p.kv_heads = k->kv_heads; p.group = k->group; p.q_heads = k->q_heads;
  p.n_tokens = l.n_tokens;
  p.n_sink_eff = k->sink_at(l.n_tokens);
  p.n_body = k->body_at(l.n_tokens);
  p.win_start = p.n_sink_eff + p.n_body;
  p.cur_bits = l.cur_bits;
  p.body_tiles = (p.n_body + 15) / 16;
  p.sink_tiles = k->sink_tiles;
  p.aux_tiles = k->sink_tiles + k->ring_tiles;
  p.n_slices = k->n_slices;
  // one line of work units over all slices: a body tile is one unit, an INT16 tile their byte ratio
  p.w16 = (tile_bytes(16) + tile_bytes(l.cur_bits) - 1) / tile_bytes(l.cur_bits);
  // every slice starts with empty units that stand for the fixed cost of a segment
  p.units_lead = segment_cost_tiles(l.cur_bits);
  p.units_aux = p.units_lead + (long long)p.aux_tiles * p.w16;
  p.units_slice = p.units_aux + p.body_tiles;
  p.units_total = p.units_slice * k->n_slices;
  const int width_idx = l.cur_bits == 16 ? 0 : l.cur_bits == 8 ? 1 : l.cur_bits == 4 ? 2 : 3;
  const int want = k->user_ctas > 0 ? k->user_ctas : k->resident_ctas[width_idx];
  const long long per = std::max<long long>((p.units_total + want - 1) / want, k->user_ctas > 0 ? 1 : kMinUnitsPerCta);
  p.units_per_cta = per;
  p.line_origin = 0;
  p.unit_weight = 1;
  p.cta_origin = 0;
  n_ctas = (unsigned)((p.units_total + per - 1) / per);
  p.qk_scale = k->sm_scale * 1.4426950408889634f;
  return PMKVQ_OK;
}

template <int BITS>
static cudaError_t attn_launch_width(const AttnParams &p, unsigned n_ctas, cudaStream_t st, unsigned *error_word) {
  if (p.geom.rows)
    decode_attn_splitk_kernel<BITS, true><<<n_ctas, kAttnThreads, attn_smem_bytes<BITS, true>(), st>>>(p, error_word);
  else
    decode_attn_splitk_kernel<BITS, false><<<n_ctas, kAttnThreads, attn_smem_bytes<BITS, false>(), st>>>(p, error_word);
  return cudaGetLastError();
}

static cudaError_t attn_launch(const AttnParams &p, unsigned n_ctas, cudaStream_t st, unsigned *error_word) {
  switch (p.cur_bits) {
    case 16: return attn_launch_width<16>(p, n_ctas, st, error_word);
    case 8: return attn_launch_width<8>(p, n_ctas, st, error_word);
    case 4: return attn_launch_width<4>(p, n_ctas, st, error_word);
    default: return attn_launch_width<2>(p, n_ctas, st, error_word);
  }
}

static pmkvq_status attention_on_arena(pmkvq_cache *k, int32_t layer, const void *d_Q, float *d_out, cudaStream_t st) {
  AttnParams p;
  unsigned n_ctas = 0;
  const pmkvq_status s = attn_params(k, layer, d_Q, d_out, p, n_ctas);
  if (s != PMKVQ_OK) return s;
  p.partials = reinterpret_cast<float *>(k->arena + k->off_partials + (size_t)layer * k->partial_bytes);
  p.tickets = reinterpret_cast<unsigned *>(k->arena + k->off_tickets) + (size_t)layer * k->n_slices;
  const cudaError_t e = attn_launch(p, n_ctas, st, reinterpret_cast<unsigned *>(k->arena + k->off_error));
  k->launches += 1;
  return e == cudaSuccess ? PMKVQ_OK : PMKVQ_ERR_CUDA;
}

// Time per 16-token tile at each width, in fiftieths of a 2-bit tile's (measured: 52.6 / 55.4 / 84.1 us per
// block of 130 560 tiles at 2 / 4 / 8 bit, about 160 us at 16 bit).
inline int tile_weight(int bits) { return bits == 16 ? 152 : bits == 8 ? 80 : bits == 4 ? 53 : 50; }

static pmkvq_status attention_all_blocks(pmkvq_cache *k, const void *d_Q, float *d_out, cudaStream_t st) {
  static_assert(kMaxFusedLayers >= kMaxStepLayers, "the step's argument tables share one size");
  FusedParams fp;
  fp.geoms = reinterpret_cast<const LayerGeom *>(k->arena + k->off_geoms);
  fp.Q = static_cast<const uint16_t *>(d_Q);
  fp.lambda = reinterpret_cast<const float *>(k->arena + k->off_lambda);
  fp.vmax_bits = reinterpret_cast<const unsigned *>(k->arena + k->off_vmax);
  fp.partials = reinterpret_cast<float *>(k->arena + k->off_partials);
  fp.out = d_out;
  fp.tickets = reinterpret_cast<unsigned *>(k->arena + k->off_tickets);
  fp.error_word = reinterpret_cast<unsigned *>(k->arena + k->off_error);
  fp.partial_stride = k->partial_bytes / sizeof(float);
  fp.layers = k->layers; fp.kv_heads = k->kv_heads; fp.group = k->group; fp.q_heads = k->q_heads;
  fp.n_slices = k->n_slices; fp.batch = k->batch;
  fp.n_sink = k->n_sink; fp.window = k->window; fp.evict_chunk = k->evict_chunk;
  fp.sink_tiles = k->sink_tiles; fp.ring_tiles = k->ring_tiles;
  fp.rows = k->rows;
  fp.qk_scale = k->sm_scale * 1.4426950408889634f;
  long long total = 0;
  for (int l = 0; l < k->layers; ++l) {
    const Layer &L = k->L[l];
    if (L.n_tokens <= 0) return PMKVQ_ERR_INVALID_ARG;
    const int bits = L.cur_bits;
    const int w16 = (tile_bytes(16) + tile_bytes(bits) - 1) / tile_bytes(bits);
    const long long body_tiles = (k->body_at(L.n_tokens) + 15) / 16;
    const long long units_slice = segment_cost_tiles(bits) + (long long)(k->sink_tiles + k->ring_tiles) * w16 + body_tiles;
    fp.start[l] = total;
    fp.n_tokens[l] = L.n_tokens;
    fp.bits[l] = (unsigned char)bits;
    fp.lead[l] = (unsigned char)segment_cost_tiles(bits);
    fp.weight[l] = (unsigned char)tile_weight(bits);
    total += units_slice * k->n_slices * tile_weight(bits);
  }
  fp.start[k->layers] = total;
  fp.total = total;
  const int want = k->user_ctas > 0 ? k->user_ctas : k->resident_fused;
  // A piece must never be shorter than the heaviest unit: then every CTA between the owners of a slice's
  // first and last unit holds the first fine unit of at least one unit of that slice and publishes a
  // partial, which is what the slice's ticket count expects.
  fp.per_cta = std::max<long long>((total + want - 1) / want,
                                   k->user_ctas > 0 ? (long long)tile_weight(16) : 50ll * kMinUnitsPerCta);
  const unsigned n_ctas = (unsigned)((total + fp.per_cta - 1) / fp.per_cta);
  if (k->rows) decode_attn_fused_kernel<true><<<n_ctas, kAttnThreads, attn_fused_smem_bytes<true>(), st>>>(fp);
  else decode_attn_fused_kernel<false><<<n_ctas, kAttnThreads, attn_fused_smem_bytes<false>(), st>>>(fp);
  k->launches += 1;
  return cudaGetLastError() == cudaSuccess ? PMKVQ_OK : PMKVQ_ERR_CUDA;
}

extern "C" {

pmkvq_status pmkvq_decode_attention(pmkvq_cache *k, int32_t layer, const void *d_Q, float *d_out, void *stream) {
  return attention_on_arena(k, layer, d_Q, d_out, static_cast<cudaStream_t>(stream));
}

pmkvq_status pmkvq_decode_attention_static(pmkvq_cache *k, int32_t layer, const void *d_Q, float *d_out, void *stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  AttnParams p;
  unsigned n_ctas = 0;
  const pmkvq_status s = attn_params(k, layer, d_Q, d_out, p, n_ctas);
  if (s != PMKVQ_OK) return s;
  // the fixed scratch holds one ticket per slice and one partial per (CTA, slice it touches)
  if ((size_t)k->n_slices * sizeof(unsigned) > kStaticTicketBytes ||
      (size_t)n_ctas + (size_t)k->n_slices > kStaticPartialSlots)
    return PMKVQ_ERR_SCRATCH_LIMIT;
  unsigned char *scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) return PMKVQ_ERR_CUDA;
  p.tickets = reinterpret_cast<unsigned *>(scratch);
  p.partials = reinterpret_cast<float *>(scratch + kStaticTicketBytes);
  // the array keeps whatever the previous call left: the tickets must start at zero
  if (cudaMemsetAsync(p.tickets, 0, (size_t)k->n_slices * sizeof(unsigned), st) != cudaSuccess) return PMKVQ_ERR_CUDA;
  const cudaError_t e = attn_launch(p, n_ctas, st, reinterpret_cast<unsigned *>(k->arena + k->off_error));
  k->launches += 1;
  return e == cudaSuccess ? PMKVQ_OK : PMKVQ_ERR_CUDA;
}

pmkvq_status pmkvq_decode_step(pmkvq_cache *k, const void *d_K, const void *d_V, const void *d_Q, float *d_out,
                               void *stream) {
  if (!k || !d_K || !d_V || !d_Q || !d_out) return PMKVQ_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_K) | reinterpret_cast<uintptr_t>(d_V)) & 7) return PMKVQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t kv_stride = (size_t)k->n_slices * kHeadDim * 2;            // bytes of one block's bf16 K (or V)
  const size_t q_stride = (size_t)k->batch * k->q_heads * kHeadDim * 2;   // bytes of one block's bf16 Q
  const size_t o_stride = (size_t)k->batch * k->q_heads * kHeadDim;       // floats of one block's output
  // 1. policy of every block, first without side effects: if any block cannot take its token (capacity, or a
  //    full budget without auto_reduce) the call fails here and no block has been reduced or appended to
  for (int layer = 0; layer < k->layers; ++layer) {
    int n_after = 0, n_reduce = 0;
    const pmkvq_status s = append_check(k, layer, 1, n_after, n_reduce);
    if (s != PMKVQ_OK) return s;
  }
  if (k->layers > kMaxStepLayers || (k->window == 0 && k->evict_chunk > 1)) {
    // too many blocks for one argument block, or appends that need two launches per block: block by block
    for (int layer = 0; layer < k->layers; ++layer) {
      pmkvq_status s = pmkvq_append(k, layer, static_cast<const uint8_t *>(d_K) + layer * kv_stride,
                                    static_cast<const uint8_t *>(d_V) + layer * kv_stride, 1, stream);
      if (s == PMKVQ_OK)
        s = pmkvq_decode_attention(k, layer, static_cast<const uint8_t *>(d_Q) + layer * q_stride,
                                   d_out + layer * o_stride, stream);
      if (s != PMKVQ_OK) return s;  // only a CUDA launch error can get here
    }
    return PMKVQ_OK;
  }
  //    then the reduces the budgets ask for; nothing is appended yet
  for (int layer = 0; layer < k->layers; ++layer) {
    int n_after = 0;
    const pmkvq_status s = append_prepare(k, layer, 1, st, n_after);
    if (s != PMKVQ_OK) return s;  // only a CUDA launch error can get here
  }
  // 2. quantize-on-append and evictions of all blocks in one launch
  StepParams sp;
  for (int layer = 0; layer < k->layers; ++layer) {
    sp.n_old[layer] = k->L[layer].n_tokens;
    sp.cur_bits[layer] = (unsigned char)k->L[layer].cur_bits;
  }
  const long long warps = 2ll * (k->evict_chunk + 1) * k->n_slices * k->layers;
  append_step_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(
      static_cast<const uint16_t *>(d_K), static_cast<const uint16_t *>(d_V),
      reinterpret_cast<const float *>(k->arena + k->off_inv_lambda), reinterpret_cast<unsigned *>(k->arena + k->off_vmax),
      reinterpret_cast<const LayerGeom *>(k->arena + k->off_geoms), sp, k->layers, k->n_slices, k->kv_heads, k->n_sink,
      k->window, k->evict_chunk);
  ++k->launches;
  if (cudaGetLastError() != cudaSuccess) return PMKVQ_ERR_CUDA;
  for (int layer = 0; layer < k->layers; ++layer) k->L[layer].n_tokens += 1;
  // 3. attention of all blocks in one launch: their tiles form one line of work cut into one piece per CTA
  return attention_all_blocks(k, d_Q, d_out, st);
}

pmkvq_status pmkvq_decode_attention_all(pmkvq_cache *k, const void *d_Q, float *d_out, void *stream) {
  if (!k || !d_Q || !d_out) return PMKVQ_ERR_INVALID_ARG;
  if (k->layers > kMaxFusedLayers) return PMKVQ_ERR_INVALID_ARG;
  return attention_all_blocks(k, d_Q, d_out, static_cast<cudaStream_t>(stream));
}

pmkvq_status pmkvq_device_status(pmkvq_cache *k, uint32_t *h_wait_bits) {
  if (!k) return PMKVQ_ERR_INVALID_ARG;
  unsigned word = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return PMKVQ_ERR_CUDA;
  if (cudaMemcpy(&word, k->arena + k->off_error, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return PMKVQ_ERR_CUDA;
  if (h_wait_bits) *h_wait_bits = word;
  return word ? PMKVQ_ERR_DEVICE_WAIT : PMKVQ_OK;
}

pmkvq_status pmkvq_selftest_bounded_wait(pmkvq_cache *k, void *stream, uint32_t *h_gave_up) {
  if (!k || !h_gave_up) return PMKVQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned *word = reinterpret_cast<unsigned *>(k->arena + k->off_error) + 1;  // beside the error word, never read by it
  if (cudaMemsetAsync(word, 0, sizeof(unsigned), st) != cudaSuccess) return PMKVQ_ERR_CUDA;
  bounded_wait_selftest_kernel<<<1, 1, 0, st>>>(word, 1u << 10);
  ++k->launches;
  unsigned got = 0;
  if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(&got, word, sizeof(got), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return PMKVQ_ERR_CUDA;
  *h_gave_up = got;
  return PMKVQ_OK;
}

pmkvq_status pmkvq_restore_layer_state(pmkvq_cache *k, int32_t layer, int32_t n_tokens, int32_t cur_bits) {
  if (!k || layer < 0 || layer >= k->layers || n_tokens < 0 || n_tokens > k->max_tokens || !valid_bits(cur_bits))
    return PMKVQ_ERR_INVALID_ARG;
  Layer &l = k->L[layer];
  if (cur_bits < l.fbit) return PMKVQ_ERR_INVALID_ARG;
  if (k->bytes_at(n_tokens, cur_bits) > l.budget) return PMKVQ_ERR_INVALID_ARG;
  if ((size_t)(((k->body_at(n_tokens) + 15) / 16 + kStreams - 1) / kStreams) * tile_bytes(cur_bits) > l.stream_stride)
    return PMKVQ_ERR_INVALID_ARG;
  l.n_tokens = n_tokens;
  l.cur_bits = cur_bits;
  return PMKVQ_OK;
}

pmkvq_status pmkvq_arena_layout(const pmkvq_cache *k, int32_t layer, uint64_t *h_out) {
  if (!k || !h_out || layer < 0 || layer >= k->layers) return PMKVQ_ERR_INVALID_ARG;
  const Layer &l = k->L[layer];
  const LayerGeom g = k->geom(l);
  h_out[0] = k->arena_bytes;
  h_out[1] = l.offset;
  h_out[2] = g.slice_stride;
  h_out[3] = g.ring_off;
  h_out[4] = g.body_off;
  h_out[5] = g.stream_stride;
  h_out[6] = (uint64_t)k->ring_tiles * kTileTokens;
  h_out[7] = k->off_partials + (uint64_t)layer * k->partial_bytes;
  h_out[8] = k->partial_bytes;
  h_out[9] = (uint64_t)kMaxGroup * kPartialStride * sizeof(float);
  return PMKVQ_OK;
}

pmkvq_status pmkvq_layer_state(const pmkvq_cache *k, int32_t layer, int32_t *n_tokens, int32_t *cur_bits,
                               uint64_t *bytes_used, uint64_t *budget_bytes) {
  if (!k || layer < 0 || layer >= k->layers) return PMKVQ_ERR_INVALID_ARG;
  const Layer &l = k->L[layer];
  if (n_tokens) *n_tokens = l.n_tokens;
  if (cur_bits) *cur_bits = l.cur_bits;
  if (bytes_used) *bytes_used = k->bytes_at(l.n_tokens, l.cur_bits);
  if (budget_bytes) *budget_bytes = l.budget;
  return PMKVQ_OK;
}

uint64_t pmkvq_launch_count(const pmkvq_cache *k) { return k ? k->launches : 0; }

uint64_t pmkvq_attention_bytes(const pmkvq_cache *k, int32_t layer) {
  if (!k || layer < 0 || layer >= k->layers) return 0;
  const Layer &l = k->L[layer];
  const uint64_t nb = k->body_at(l.n_tokens), n16 = l.n_tokens - nb;
  const uint64_t kv = 2ull * k->n_slices * (n16 * (16 * 16 + 8) + nb * (16 * l.cur_bits + 8));
  const uint64_t qo = (uint64_t)k->batch * k->q_heads * kHeadDim * (2 + 4);
  return kv + qo + (uint64_t)k->kv_heads * kHeadDim * 4;
}

static pmkvq_status export_slice_impl(pmkvq_cache *k, int32_t layer, int32_t batch_idx, int32_t kv_head, int32_t is_value,
                                      uint16_t *h_codes, float *h_scale, float *h_zero, uint8_t *h_bits, uint8_t *h_packed) {
  if (!k || layer < 0 || layer >= k->layers || batch_idx < 0 || batch_idx >= k->batch || kv_head < 0 ||
      kv_head >= k->kv_heads)
    return PMKVQ_ERR_INVALID_ARG;
  const Layer &l = k->L[layer];
  if (cudaDeviceSynchronize() != cudaSuccess) return PMKVQ_ERR_CUDA;
  const LayerGeom g = k->geom(l);
  const int n = l.n_tokens, n_sink_eff = k->sink_at(n), n_body = k->body_at(n), win_start = n_sink_eff + n_body;
  const size_t fixed = g.body_off;
  const size_t body_bytes = n_body > 0 ? g.stream_stride * kStreams : 0;
  std::vector<uint8_t> host(fixed + body_bytes);
  const uint8_t *src = g.base + (size_t)(batch_idx * k->kv_heads + kv_head) * g.slice_stride;
  if (cudaMemcpy(host.data(), src, host.size(), cudaMemcpyDeviceToHost) != cudaSuccess) return PMKVQ_ERR_CUDA;
  size_t packed_off = 0;
  for (int t = 0; t < n; ++t) {
    const uint8_t *tile;
    int row, bits;
    if (t < k->n_sink) {
      tile = host.data() + (size_t)(t >> 4) * tile_bytes(16); row = t & 15; bits = 16;
    } else if (t < win_start) {
      const int j = t - k->n_sink;
      tile = host.data() + g.body_off + body_tile_offset(j >> 4, l.cur_bits, g.stream_stride); row = j & 15; bits = l.cur_bits;
    } else {
      const int rp = (t - k->n_sink) % g.ring_tokens;
      tile = host.data() + g.ring_off + (size_t)(rp >> 4) * tile_bytes(16); row = rp & 15; bits = 16;
    }
    const uint8_t *part = tile + (is_value ? v_part_offset(bits) : 0);
    const uint32_t cmask = (1u << bits) - 1u;
    uint8_t packed[256];
    std::memset(packed, 0, sizeof(packed));
    for (int ch = 0; ch < kHeadDim; ++ch) {
      int bo, sh;
      if (is_value) v_slot(bits, k->rows != 0, row, ch, bo, sh); else k_slot(bits, k->rows != 0, row, ch, bo, sh);
      uint16_t hw;
      std::memcpy(&hw, part + bo, 2);
      const uint32_t c = (hw >> sh) & cmask;
      if (h_codes) h_codes[(size_t)t * kHeadDim + ch] = (uint16_t)c;
      if (bits == 16) { packed[2 * ch] = c & 0xFF; packed[2 * ch + 1] = c >> 8; }
      else packed[(ch * bits) >> 3] |= (uint8_t)(c << ((ch * bits) & 7));
    }
    float sc, ze;
    std::memcpy(&sc, tile + meta_offset(bits) + meta_slot(bits, k->rows != 0, is_value ? 2 : 0, row), 4);
    std::memcpy(&ze, tile + meta_offset(bits) + meta_slot(bits, k->rows != 0, is_value ? 3 : 1, row), 4);
    if (h_scale) h_scale[t] = sc;
    if (h_zero) h_zero[t] = ze;
    if (h_bits) h_bits[t] = (uint8_t)bits;
    if (h_packed) std::memcpy(h_packed + packed_off, packed, 16 * bits);
    packed_off += 16 * bits;
  }
  return PMKVQ_OK;
}

pmkvq_status pmkvq_export_slice(pmkvq_cache *k, int32_t layer, int32_t batch_idx, int32_t kv_head, int32_t is_value,
                                uint16_t *h_codes, float *h_scale, float *h_zero, uint8_t *h_bits, uint8_t *h_packed) {
  try {
    return export_slice_impl(k, layer, batch_idx, kv_head, is_value, h_codes, h_scale, h_zero, h_bits, h_packed);
  } catch (...) {
    return PMKVQ_ERR_STATE;
  }
}

pmkvq_status pmkvq_set_attention_ctas(pmkvq_cache *k, int32_t n_ctas) {
  if (!k || n_ctas < 0 || n_ctas > kMaxCtas) return PMKVQ_ERR_INVALID_ARG;
  k->user_ctas = n_ctas;
  return PMKVQ_OK;
}

pmkvq_status pmkvq_calibrate_lambda(const void *d_K, int32_t n_tokens, int32_t n_seq, int32_t kv_heads, double pos_scale,
                                    double theta, float alpha, float floor_value, float *d_lambda, void *stream) {
  if (!d_K || !d_lambda || n_tokens <= 0 || n_seq <= 0 || kv_heads <= 0 || !(pos_scale > 0.0) || !(theta > 1.0) ||
      !(floor_value > 0.f) || !std::isfinite(alpha))
    return PMKVQ_ERR_INVALID_ARG;
  if ((int64_t)n_seq * kv_heads > (1 << 20)) return PMKVQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n = kv_heads * kHeadDim;
  if (cudaMemsetAsync(d_lambda, 0, (size_t)n * sizeof(float), st) != cudaSuccess) return PMKVQ_ERR_CUDA;
  const int tokens_per_cta = std::max(1, (n_tokens + 148 * 8 - 1) / (148 * 8));
  const unsigned grid = (unsigned)((n_tokens + tokens_per_cta - 1) / tokens_per_cta);
  calib_absmax_kernel<<<grid, 128, 0, st>>>(static_cast<const uint16_t *>(d_K), reinterpret_cast<unsigned *>(d_lambda),
                                            n_tokens, n_seq * kv_heads, kv_heads, tokens_per_cta, pos_scale, theta);
  calib_finish_kernel<<<(n + 255) / 256, 256, 0, st>>>(d_lambda, n, floor_value, alpha);
  return cudaGetLastError() == cudaSuccess ? PMKVQ_OK : PMKVQ_ERR_CUDA;
}

static size_t grid_ws_round(size_t b) { return (b + 255) / 256 * 256; }

// workspace of the alpha grid search: abs-max, rotation table, loss sums, alphas, then fp32 copies of this
// pass's Keys, of the Values (as given and quantized) and the unquantized operator's output
struct GridWorkspace {
  size_t amax, table, loss, alphas, k_pass, v_raw, v_hat, o_ref, total;
};
static GridWorkspace grid_workspace(int64_t n_tokens, int64_t n_seq, int64_t kv_heads, int64_t group) {
  GridWorkspace w;
  size_t off = 0;
  const size_t kv = (size_t)(n_tokens * n_seq * kv_heads) * kHeadDim * sizeof(float);
  w.amax = off; off += grid_ws_round((size_t)kv_heads * kHeadDim * sizeof(float));
  w.table = off; off += grid_ws_round((size_t)n_tokens * 64 * sizeof(float2));
  w.loss = off; off += grid_ws_round(kMaxAlphas * sizeof(double));
  w.alphas = off; off += grid_ws_round(kMaxAlphas * sizeof(float));
  w.k_pass = off; off += grid_ws_round(kv);
  w.v_raw = off; off += grid_ws_round(kv);
  w.v_hat = off; off += grid_ws_round(kv);
  w.o_ref = off; off += grid_ws_round(kv * (size_t)group);
  w.total = off;
  return w;
}

uint64_t pmkvq_alpha_grid_workspace_bytes(int32_t n_tokens, int32_t n_seq, int32_t kv_heads, int32_t group) {
  if (n_tokens <= 0 || n_seq <= 0 || kv_heads <= 0 || group <= 0) return 0;
  return grid_workspace(n_tokens, n_seq, kv_heads, group).total;
}

pmkvq_status pmkvq_alpha_grid_search(const void *d_K, const void *d_Q, const void *d_V, int32_t n_tokens, int32_t n_seq,
                                     int32_t kv_heads, int32_t group, int32_t bits, const float *h_alphas,
                                     int32_t n_alphas, double pos_scale, double theta, float floor_value,
                                     void *d_workspace, double *h_losses, int32_t *h_best, void *stream) {
  if (!d_K || !d_Q || !d_V || !h_alphas || !d_workspace || !h_losses || n_tokens <= 0 || n_seq <= 0 || kv_heads <= 0 ||
      group <= 0 || n_alphas <= 0 || n_alphas > kMaxAlphas || !(pos_scale > 0.0) || !(theta > 1.0) || !(floor_value > 0.f))
    return PMKVQ_ERR_INVALID_ARG;
  if (bits != 2 && bits != 4 && bits != 8 && bits != 16) return PMKVQ_ERR_INVALID_ARG;
  if ((int64_t)n_seq * kv_heads > (1 << 20) || (int64_t)kv_heads * group > 65535 || n_seq > 65535 ||
      (reinterpret_cast<uintptr_t>(d_workspace) & 255))
    return PMKVQ_ERR_INVALID_ARG;
  for (int i = 0; i < n_alphas; ++i)
    if (!std::isfinite(h_alphas[i])) return PMKVQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const GridWorkspace w = grid_workspace(n_tokens, n_seq, kv_heads, group);
  uint8_t *ws = static_cast<uint8_t *>(d_workspace);
  float *d_amax = reinterpret_cast<float *>(ws + w.amax);
  float2 *d_table = reinterpret_cast<float2 *>(ws + w.table);
  double *d_loss = reinterpret_cast<double *>(ws + w.loss);
  float *d_alphas = reinterpret_cast<float *>(ws + w.alphas);
  float *d_k = reinterpret_cast<float *>(ws + w.k_pass), *d_v_raw = reinterpret_cast<float *>(ws + w.v_raw);
  float *d_v_hat = reinterpret_cast<float *>(ws + w.v_hat), *d_o_ref = reinterpret_cast<float *>(ws + w.o_ref);
  if (cudaMemsetAsync(d_amax, 0, (size_t)kv_heads * kHeadDim * sizeof(float), st) != cudaSuccess ||
      cudaMemsetAsync(d_loss, 0, kMaxAlphas * sizeof(double), st) != cudaSuccess ||
      cudaMemcpyAsync(d_alphas, h_alphas, (size_t)n_alphas * sizeof(float), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return PMKVQ_ERR_CUDA;
  const uint16_t *K = static_cast<const uint16_t *>(d_K), *Q = static_cast<const uint16_t *>(d_Q),
                 *V = static_cast<const uint16_t *>(d_V);
  const int tokens_per_cta = std::max(1, (n_tokens + 148 * 8 - 1) / (148 * 8));
  calib_absmax_kernel<<<(unsigned)((n_tokens + tokens_per_cta - 1) / tokens_per_cta), 128, 0, st>>>(
      K, reinterpret_cast<unsigned *>(d_amax), n_tokens, n_seq * kv_heads, kv_heads, tokens_per_cta, pos_scale, theta);
  rope_table_kernel<<<(unsigned)((n_tokens * 64 + 255) / 256), 256, 0, st>>>(d_table, n_tokens, pos_scale, theta);
  if (cudaFuncSetAttribute(alpha_grid_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGridSmemBytes) != cudaSuccess)
    return PMKVQ_ERR_CUDA;
  const long long n_vectors = (long long)n_tokens * n_seq * kv_heads;
  const unsigned prep_grid = (unsigned)((n_vectors + 3) / 4);
  const dim3 grid((unsigned)((n_tokens + kGridQueries - 1) / kGridQueries), (unsigned)(kv_heads * group), (unsigned)n_seq);
  // pass -1: the unquantized operator; passes 0 .. n_alphas - 1: Eq. 9 at each alpha
  for (int pass = -1; pass < n_alphas; ++pass) {
    float *v_out = pass == -1 ? d_v_raw : pass == 0 ? d_v_hat : nullptr;
    alpha_grid_prep_kernel<<<prep_grid, 128, 0, st>>>(K, V, d_amax, d_table, d_alphas, pass, n_vectors, n_seq * kv_heads,
                                                      kv_heads, bits, floor_value, d_k, v_out);
    alpha_grid_attn_kernel<<<grid, 128, kGridSmemBytes, st>>>(Q, d_k, pass == -1 ? d_v_raw : d_v_hat, d_amax, d_table,
                                                              d_alphas, pass, n_tokens, n_seq, kv_heads, group, floor_value,
                                                              d_o_ref, d_loss);
  }
  if (cudaGetLastError() != cudaSuccess) return PMKVQ_ERR_CUDA;
  double sums[kMaxAlphas];
  if (cudaMemcpyAsync(sums, d_loss, (size_t)n_alphas * sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return PMKVQ_ERR_CUDA;
  const double count = (double)n_tokens * n_seq * kv_heads * group * kHeadDim;
  int best = 0;
  for (int i = 0; i < n_alphas; ++i) {
    h_losses[i] = sums[i] / count;
    if (h_losses[i] < h_losses[best]) best = i;  // the first one on ties
  }
  if (h_best) *h_best = best;
  return PMKVQ_OK;
}

static pmkvq_status allocate_bits_impl(int32_t layers, int32_t n_choices, const uint8_t *h_widths, const double *h_sens,
                                       const uint64_t *h_mem, uint64_t budget, uint8_t *h_fbit_out, double *h_cost_out) {
  if (layers <= 0 || n_choices <= 0 || n_choices > 8 || !h_widths || !h_sens || !h_mem || !h_fbit_out)
    return PMKVQ_ERR_INVALID_ARG;
  for (int i = 0; i < layers * n_choices; ++i)
    if (!std::isfinite(h_sens[i])) return PMKVQ_ERR_INVALID_ARG;
  // memory above each block's smallest choice, in units of the gcd of those differences
  std::vector<uint64_t> base(layers), extra((size_t)layers * n_choices);
  uint64_t floor_sum = 0, g = 0;
  for (int i = 0; i < layers; ++i) {
    base[i] = *std::min_element(h_mem + (size_t)i * n_choices, h_mem + (size_t)(i + 1) * n_choices);
    floor_sum += base[i];
    for (int c = 0; c < n_choices; ++c) {
      uint64_t d = h_mem[(size_t)i * n_choices + c] - base[i], a = g;
      extra[(size_t)i * n_choices + c] = d;
      while (d) { const uint64_t t = a % d; a = d; d = t; }
      g = a;
    }
  }
  if (floor_sum > budget) return PMKVQ_ERR_CAPACITY;
  if (g == 0) g = 1;  // all choices of every block cost the same
  uint64_t max_extra = 0;
  for (int i = 0; i < layers; ++i) {
    uint64_t m = 0;
    for (int c = 0; c < n_choices; ++c) m = std::max(m, extra[(size_t)i * n_choices + c] / g);
    max_extra += m;
  }
  const uint64_t cap = std::min((budget - floor_sum) / g, max_extra);
  if (cap >= (1ull << 26) / (uint64_t)layers) return PMKVQ_ERR_INVALID_ARG;  // table of (cap + 1) * layers cells
  const size_t W = (size_t)cap + 1;
  const double inf = std::numeric_limits<double>::infinity();
  // best[i][w]: minimal sensitivity of blocks 0..i-1 using exactly w units; pick[i][w]: choice of block i-1
  std::vector<double> prev(W, inf), cur(W);
  std::vector<int8_t> pick((size_t)layers * W, -1);
  prev[0] = 0.0;
  for (int i = 0; i < layers; ++i) {
    std::fill(cur.begin(), cur.end(), inf);
    for (int c = 0; c < n_choices; ++c) {
      const uint64_t wc = extra[(size_t)i * n_choices + c] / g;
      const double sc = h_sens[(size_t)i * n_choices + c];
      for (size_t w = wc; w < W; ++w) {
        const double v = prev[w - wc] + sc;
        if (v < cur[w]) { cur[w] = v; pick[(size_t)i * W + w] = (int8_t)c; }  // strict: the lower index wins ties
      }
    }
    prev.swap(cur);
  }
  size_t best_w = 0;
  for (size_t w = 1; w < W; ++w)
    if (prev[w] < prev[best_w]) best_w = w;  // strict: less memory wins ties
  if (!(prev[best_w] < inf)) return PMKVQ_ERR_STATE;
  if (h_cost_out) *h_cost_out = prev[best_w];
  size_t w = best_w;
  for (int i = layers - 1; i >= 0; --i) {
    const int c = pick[(size_t)i * W + w];
    if (c < 0) return PMKVQ_ERR_STATE;
    h_fbit_out[i] = h_widths[c];
    w -= (size_t)(extra[(size_t)i * n_choices + c] / g);
  }
  return PMKVQ_OK;
}

// host allocations (std::vector) must not throw across the C boundary
pmkvq_status pmkvq_allocate_bits(int32_t layers, int32_t n_choices, const uint8_t *h_widths, const double *h_sens,
                                 const uint64_t *h_mem, uint64_t budget, uint8_t *h_fbit_out, double *h_cost_out) {
  try {
    return allocate_bits_impl(layers, n_choices, h_widths, h_sens, h_mem, budget, h_fbit_out, h_cost_out);
  } catch (...) {
    return PMKVQ_ERR_STATE;
  }
}

const char *pmkvq_status_string(pmkvq_status s) {
  switch (s) {
    case PMKVQ_OK: return "ok";
    case PMKVQ_ERR_INVALID_ARG: return "invalid argument";
    case PMKVQ_ERR_ARENA_TOO_SMALL: return "arena too small";
    case PMKVQ_ERR_BUDGET_FULL: return "budget full: reduce the block first";
    case PMKVQ_ERR_AT_FBIT: return "block is already at its final bit width";
    case PMKVQ_ERR_CAPACITY: return "capacity exceeded";
    case PMKVQ_ERR_CUDA: return "CUDA error";
    case PMKVQ_ERR_STATE: return "internal state error";
    case PMKVQ_ERR_SCRATCH_LIMIT: return "problem too large for the built-in scratch: use pmkvq_decode_attention";
    case PMKVQ_ERR_DEVICE_WAIT: return "a device-side wait ran out: the results of the affected launch are invalid";
  }
  return "unknown status";
}

}  // extern "C"

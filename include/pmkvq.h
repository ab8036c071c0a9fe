/*
 * pmkvq.h - C ABI of the B200-native PM-KVQ decode hot path.
 *
 * PM-KVQ (Progressive Mixed-precision KV cache Quantization) stores a transformer block's
 * KV cache as integer codes with a per-token fp32 scale and zero-point, starts at 16 bit and
 * halves the width of the existing cache (16 -> 8 -> 4 -> 2) each time the block's memory
 * budget fills, down to the block's final width "Fbit" (Sec. 3.1).  Keys are channel-equalized
 * before quantization and the scale is migrated into the Query (Eq. 9, Sec. 3.3).
 *
 * Conventions
 *  - Pointers named d_* are DEVICE pointers owned by the caller; h_* are HOST pointers.
 *    The library never frees caller memory and never allocates device memory: the whole
 *    cache (codes, scales, zero-points, split-K partials) lives in one caller-supplied arena.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Kernel launches are
 *    asynchronous on that stream; an asynchronous CUDA error surfaces as PMKVQ_ERR_CUDA from a
 *    later call.
 *  - Every call returns a status; nothing throws, aborts or traps.  Argument errors are
 *    detected on the host before any launch and leave the cache state unchanged.
 *  - All sequences of the batch share one length.  head_dim is 128 (one quantization group =
 *    one token x one KV head x 128 channels, group size 128, Sec. 4.1.3).
 *  - A cache handle is not thread-safe.
 */
#ifndef PMKVQ_H_
#define PMKVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pmkvq_cache pmkvq_cache; /* opaque; host heap; created / destroyed by the library */

typedef enum {
  PMKVQ_OK = 0,
  PMKVQ_ERR_INVALID_ARG = 1,     /* bad pointer, size, layer index, bit width ... */
  PMKVQ_ERR_ARENA_TOO_SMALL = 2, /* arena_bytes < pmkvq_arena_bytes_required()   */
  PMKVQ_ERR_BUDGET_FULL = 3,     /* append would exceed the block budget and cur_bits > Fbit:
                                    call pmkvq_progressive_reduce and retry (or set auto_reduce) */
  PMKVQ_ERR_AT_FBIT = 4,         /* progressive_reduce on a block already at its Fbit */
  PMKVQ_ERR_CAPACITY = 5,        /* over budget at Fbit, or past max_tokens */
  PMKVQ_ERR_CUDA = 6,            /* a CUDA runtime call or launch failed */
  PMKVQ_ERR_STATE = 7,           /* internal invariant violated */
  PMKVQ_ERR_SCRATCH_LIMIT = 8,   /* pmkvq_decode_attention_static: more slices / CTAs than its fixed scratch holds */
  PMKVQ_ERR_DEVICE_WAIT = 9      /* pmkvq_device_status: a bounded wait inside a kernel ran out */
} pmkvq_status;

typedef struct {
  int32_t layers;       /* number of transformer blocks */
  int32_t q_heads;      /* query heads; q_heads / kv_heads (the GQA group) must be 1..8 */
  int32_t kv_heads;
  int32_t head_dim;     /* must be 128 */
  int32_t batch;
  int32_t max_tokens;   /* maximum context length the budget is derived from (Sec. 3.1) */
  const uint8_t *fbit;           /* HOST [layers], each in {2,4,8,16}: per-block bit schedule (Sec. 3.2) */
  const uint64_t *budget_bytes;  /* HOST [layers], bytes per block for the whole batch (K+V, codes +
                                    fp32 scale + fp32 zero); NULL => size of max_tokens tokens with the
                                    body at Fbit (Sec. 3.1) */
  const float *lambda;           /* HOST [layers][kv_heads][128], > 0 and finite: Eq. 9's Lambda;
                                    NULL => all ones */
  int32_t n_sink;         /* leading tokens kept INT16 (Sec. 2.2: the first token); default 1 */
  int32_t window;         /* most recent tokens kept INT16 (Sec. 4.1.2: 128) */
  int32_t evict_chunk;    /* tokens leave the window in groups of this many (>= 1) */
  int32_t count_metadata; /* 1: budget accounting counts scale + zero bytes; 0: code bytes only */
  int32_t auto_reduce;    /* 1: pmkvq_append reduces by itself when the budget is full */
  float sm_scale;         /* softmax scale; 0 => 1/sqrt(head_dim) */
  void *d_arena;          /* DEVICE, 256-byte aligned, caller-owned, must outlive the cache */
  size_t arena_bytes;
  int32_t shift_variant;  /* how a halving 2b -> b is done (Sec. 4.4.1): 0 Equivalent Right Shift, Eq. 3 (the
                             method); 1 Direct Right Shift (X >> b, S_b = (2^b+1) S_2b, Z kept); 2 Modified
                             Right Shift (X >> b, S_b = 2^b S_2b, Z_b = Z_2b + (S_b - S_2b)/2) */
  int32_t attention_path; /* which contraction the 4- and 2-bit body is laid out for (chosen once, when the cache is
                             created, because it fixes the order of the codes inside a tile): 0 warp-level MMAs
                             (mma.sync, register operands; the faster one as measured), 1 tensor memory
                             (tcgen05.mma with the code operands unpacked into tensor memory) */
} pmkvq_config;

/* Bytes of device arena a cache with this configuration needs (d_arena / arena_bytes are
 * ignored).  Returns 0 for an invalid configuration. */
size_t pmkvq_arena_bytes_required(const pmkvq_config *cfg);

/* Problem statement of Sec. 3.1 / 3.4: create the (empty) cache of `layers` blocks, each with its
 * Fbit and budget.  Copies lambda / fbit / budgets; zero-initialises its bookkeeping in the arena
 * (synchronous).  *out is set only on PMKVQ_OK. */
pmkvq_status pmkvq_cache_create(const pmkvq_config *cfg, pmkvq_cache **out);
void pmkvq_cache_destroy(pmkvq_cache *cache);

/* Quantize-on-append (Eq. 1-2 at 16 bit; Keys multiplied by Lambda^-1 first, Eq. 9) of n_new
 * tokens, then window eviction: tokens leaving the INT16 window are shifted (Eq. 3, repeatedly)
 * to the block's current width.
 *   d_K_bf16, d_V_bf16: DEVICE bf16 [n_new][batch][kv_heads][128], read only.
 * Returns BUDGET_FULL (state unchanged) if the block must be reduced first and auto_reduce is 0,
 * INVALID_ARG for n_new < 1 (an empty append is refused, nothing is launched), CAPACITY beyond max_tokens. */
pmkvq_status pmkvq_append(pmkvq_cache *cache, int32_t layer, const void *d_K_bf16, const void *d_V_bf16,
                          int32_t n_new, void *stream);

/* One step of the progressive strategy (Sec. 3.1): shift every body token of the block from
 * 2b to b bits with Eq. 3, S_b = (2^b+1) S_2b, Z unchanged; sink and window tokens stay INT16. */
pmkvq_status pmkvq_progressive_reduce(pmkvq_cache *cache, int32_t layer, void *stream);

/* Decode-step attention of one block over all cached tokens (the one just appended included):
 * out = softmax(sm_scale * (Q Lambda) dequant(K Lambda^-1)^T) dequant(V)  (Eq. 9 with GQA).
 *   d_Q_bf16: DEVICE bf16 [batch][q_heads][128]; d_out: DEVICE fp32 [batch][q_heads][128].
 * A block without any cached token has no softmax to take: INVALID_ARG, nothing is launched. */
pmkvq_status pmkvq_decode_attention(pmkvq_cache *cache, int32_t layer, const void *d_Q_bf16, float *d_out,
                                    void *stream);

/* The same computation and the same kernel as pmkvq_decode_attention, for callers that are not
 * allowed to allocate device memory at the point of the call and have no arena workspace to offer:
 * code running inside a serving engine's pre-sized memory pool, a plugin called after the host
 * process has frozen its allocations, a real-time loop in which cudaMalloc's implicit device
 * synchronisation is not acceptable.  (The paper has no counterpart of this call; it exists for
 * such hosts.)  The split-K workspace (one ticket per slice, one partial result per CTA and slice)
 * is a 4 MiB array that is part of the library image: every GPU that loads the library holds it
 * until the process exits, and the call itself allocates and frees nothing.
 *   - Limits: batch * kv_heads <= 4096 and (attention CTAs + batch * kv_heads) <= 989; beyond them the
 *     call returns PMKVQ_ERR_SCRATCH_LIMIT and launches nothing (use pmkvq_decode_attention).
 *   - The first call on each GPU looks up the array's device address (one runtime query, with that
 *     GPU current); make that first call outside any stream capture.
 *   - All calls on a GPU share the one array, whatever cache or stream they use: two such calls that
 *     overlap on the GPU race and give wrong results.  Keep them on one stream or order them with
 *     events.  The tickets are cleared on `stream` before every launch; the partials are fully
 *     rewritten before they are read.
 * Arguments and results are those of pmkvq_decode_attention. */
pmkvq_status pmkvq_decode_attention_static(pmkvq_cache *cache, int32_t layer, const void *d_Q_bf16, float *d_out,
                                           void *stream);

/* One decode step of the whole model's attention path (Sec. 3.4, inference stage): for every block in
 * order, pmkvq_append of one new token followed by pmkvq_decode_attention; everything is enqueued on
 * `stream` without a host synchronisation.
 *   d_K_bf16, d_V_bf16: DEVICE bf16 [layers][batch][kv_heads][128]
 *   d_Q_bf16:           DEVICE bf16 [layers][batch][q_heads][128]
 *   d_out:              DEVICE fp32 [layers][batch][q_heads][128]
 * The budget of every block is tested first, without touching anything: if a block fails
 * (PMKVQ_ERR_BUDGET_FULL with auto_reduce = 0, PMKVQ_ERR_CAPACITY) its status is returned and the whole
 * cache is as it was: no block has been reduced and no block has received its token.  Only then are
 * the reduces run that the budgets ask for (auto_reduce = 1), one launch appends to all blocks and one
 * launch computes the attention of all blocks (up to 128 blocks; beyond that the call falls back to
 * one append and one attention launch per block). */
pmkvq_status pmkvq_decode_step(pmkvq_cache *cache, const void *d_K_bf16, const void *d_V_bf16, const void *d_Q_bf16,
                               float *d_out, void *stream);

/* The attention half of pmkvq_decode_step alone: decode attention of every block over its cached tokens
 * in one launch (Eq. 9 with GQA, Sec. 3.4), nothing appended.  Up to 128 blocks, every block non-empty.
 *   d_Q_bf16: DEVICE bf16 [layers][batch][q_heads][128]; d_out: DEVICE fp32 [layers][batch][q_heads][128]. */
pmkvq_status pmkvq_decode_attention_all(pmkvq_cache *cache, const void *d_Q_bf16, float *d_out, void *stream);

/* The attention kernels wait on hardware barriers (copies into shared memory, tensor-core completion); every
 * such wait has an iteration limit instead of spinning for ever.  A wait that runs out makes its CTA
 * skip the rest of its waits and return, and sets a bit in a word of the arena (1: tile copy, 2: score
 * MMAs, 4: output MMAs).  This call synchronises the device and returns PMKVQ_ERR_DEVICE_WAIT if any bit is
 * set (the outputs of the affected launch are then meaningless), PMKVQ_OK otherwise; *h_wait_bits (may be
 * NULL) receives the word.  The word is never cleared: create a new cache after a failure. */
pmkvq_status pmkvq_device_status(pmkvq_cache *cache, uint32_t *h_wait_bits);

/* Self-test of the bounded waits: launches one thread that waits on a barrier nothing will ever complete, with a
 * limit of 1024 polls.  The wait must give up, set *h_gave_up to 1 and let the kernel end normally; the CUDA
 * context stays usable (the attention kernels use the same wait with a limit of 2^20 polls and report through
 * pmkvq_device_status).  Synchronises `stream`. */
pmkvq_status pmkvq_selftest_bounded_wait(pmkvq_cache *cache, void *stream, uint32_t *h_gave_up);

/* Checkpoint / restore of a block's host-side state.  The device-side state of a cache is the arena; a
 * caller that saved a copy of the arena together with pmkvq_layer_state()'s (n_tokens, cur_bits) of every
 * block puts the bytes back and then calls this for every block.  INVALID_ARG if the pair cannot be a state
 * of this block (width below Fbit, over budget, beyond capacity); nothing on the device is touched. */
pmkvq_status pmkvq_restore_layer_state(pmkvq_cache *cache, int32_t layer, int32_t n_tokens, int32_t cur_bits);

/* Where a block's bytes sit inside the arena, for callers that checkpoint parts of it and for tests that watch
 * the bytes the kernels must not touch.  h_out receives ten values: [0] the arena bytes the cache uses
 * (= pmkvq_arena_bytes_required), [1] offset of the block's first (batch, kv_head) slice, [2] bytes between
 * slices, and inside a slice [3] offset of the INT16 window ring (the sink tiles sit at 0), [4] offset of the
 * body, [5] bytes between the body's eight streams (body tile i lives in stream i mod 8 at index i div 8,
 * tile_bytes(b) = 512 b + 256 apart), [6] ring capacity in tokens; [7] offset and [8] size of the block's
 * split-K workspace, [9] bytes of one partial slot in it. */
pmkvq_status pmkvq_arena_layout(const pmkvq_cache *cache, int32_t layer, uint64_t *h_out);

/* Split-K tuning of pmkvq_decode_attention (flash-decoding partition over the sequence): the tiles
 * of all (batch, kv_head) slices are cut into `n_ctas` equal contiguous pieces, one per CTA
 * (1..1024); 0 restores the default, one wave of resident CTAs on the GPU's SMs. */
pmkvq_status pmkvq_set_attention_ctas(pmkvq_cache *cache, int32_t n_ctas);

/* Host-side state of a block; any out pointer may be NULL. */
pmkvq_status pmkvq_layer_state(const pmkvq_cache *cache, int32_t layer, int32_t *n_tokens, int32_t *cur_bits,
                               uint64_t *bytes_used, uint64_t *budget_bytes);

/* Number of CUDA kernels this cache has launched since it was created (all calls). */
uint64_t pmkvq_launch_count(const pmkvq_cache *cache);

/* Algorithmic bytes one pmkvq_decode_attention call on this block moves in its current state:
 * codes + fp32 scale + fp32 zero of every cached token of K and V, Q in, out, lambda. */
uint64_t pmkvq_attention_bytes(const pmkvq_cache *cache, int32_t layer);

/* Copy one (batch, kv_head) slice of K (is_value = 0) or V (1) to the host in token order, for
 * bit-exact comparison.  Synchronises the device.  Any of the outputs may be NULL.
 *   h_codes  [n_tokens][128] uint16, each < 2^bits of its token
 *   h_scale, h_zero [n_tokens] fp32;  h_bits [n_tokens]
 *   h_packed canonical packed bytes, token after token: token t takes 16*bits_t bytes, element i in
 *            byte floor(i*bits/8) at bit (i*bits) mod 8 (16-bit codes little-endian). */
pmkvq_status pmkvq_export_slice(pmkvq_cache *cache, int32_t layer, int32_t batch_idx, int32_t kv_head,
                                int32_t is_value, uint16_t *h_codes, float *h_scale, float *h_zero,
                                uint8_t *h_bits, uint8_t *h_packed);

/* Calibration of the equalization vector with positional interpolation (Sec. 3.3, Eq. 10-12), on the
 * device: pre-RoPE Keys are rotated with RoPE whose position index is multiplied by pos_scale (Eq. 12;
 * 1.0 = plain RoPE, Eq. 11; pairs (i, i + 64), theta_i = theta^(-2i/128)), and
 *     lambda[h][i] = max( max over tokens and sequences |K_rot[.., h, i]| , floor )^alpha      (Eq. 10).
 *   d_K_pre_bf16  DEVICE bf16 [n_tokens][n_seq][kv_heads][128], token t sits at position t
 *   d_lambda      DEVICE fp32 [kv_heads][128], written (it also serves as the kernel's only workspace)
 * The rotation is computed in fp32 from fp64 angles; the result feeds pmkvq_config.lambda after a copy to
 * the host.  alpha is an argument; pmkvq_alpha_grid_search below picks it as Sec. 4.1.1 does. */
pmkvq_status pmkvq_calibrate_lambda(const void *d_K_pre_bf16, int32_t n_tokens, int32_t n_seq, int32_t kv_heads,
                                    double pos_scale, double theta, float alpha, float floor_value, float *d_lambda,
                                    void *stream);

/* alpha of Eq. 10 by grid search (Sec. 4.1.1: the alpha that minimises the reconstruction loss of the
 * self-attention operator), on the device, for one transformer block's calibration tensors.
 * For every alpha of the grid: lambda = max(amax, floor)^alpha from the Keys rotated per Eq. 12; the
 * quantized operator is Eq. 9, (Q Lambda) . Q_b(K Lambda^-1)^T, with K Lambda^-1 quantized at 16 bit
 * (Eq. 1-2, per token and KV head) and taken down the Eq. 3 chain to `bits`, Values quantized the same
 * way; loss[alpha] = mean squared difference between the causal self-attention output (softmax of
 * Q K^T / sqrt(128), query head h reads KV head h / group, token t attends to tokens 0..t) of the
 * unquantized rotated tensors and of the quantized ones, over tokens, sequences, heads and channels.
 * Arithmetic: rotation, equalization and quantizer decisions in fp32 (as in pmkvq_append); the attention
 * contractions run on the tensor cores with every operand carried as the sum of two fp16 numbers (22
 * significant bits) and fp32 accumulation; softmax in fp32; sums of squared errors in fp64.
 * 2 + 2 (n_alphas + 1) launches: abs-max, rotation table, then per pass one launch that writes the pass's
 * Keys (and once the Values) into the workspace and one attention launch.
 *   d_K_pre_bf16, d_V_bf16  DEVICE bf16 [n_tokens][n_seq][kv_heads][128]; Keys before RoPE, token t at position t
 *   d_Q_pre_bf16            DEVICE bf16 [n_tokens][n_seq][kv_heads * group][128], before RoPE
 *   bits                    2, 4, 8 or 16: the width whose loss is minimised (the block's Fbit)
 *   h_alphas                HOST [n_alphas], 1 <= n_alphas <= 64 (the section's grid: j / 20, j = 0..19)
 *   d_workspace             DEVICE, 256-byte aligned, pmkvq_alpha_grid_workspace_bytes(...) bytes of the same sizes
 *                           (each pass's Keys and Values at 4 bytes per element, the unquantized output in fp32)
 *   h_losses                HOST [n_alphas], written
 *   h_best                  HOST, may be NULL: index of the smallest loss (the first one on ties)
 * The call synchronises `stream` before it returns (its results are host values).  The paper states
 * the criterion only; causal masking, the quantization of the Values and the mean-squared form are
 * this library's reading of it. */
uint64_t pmkvq_alpha_grid_workspace_bytes(int32_t n_tokens, int32_t n_seq, int32_t kv_heads, int32_t group);
pmkvq_status pmkvq_alpha_grid_search(const void *d_K_pre_bf16, const void *d_Q_pre_bf16, const void *d_V_bf16,
                                     int32_t n_tokens, int32_t n_seq, int32_t kv_heads, int32_t group, int32_t bits,
                                     const float *h_alphas, int32_t n_alphas, double pos_scale, double theta,
                                     float floor_value, void *d_workspace, double *h_losses, int32_t *h_best,
                                     void *stream);

/* Block-wise bit allocation (Sec. 3.2, Eq. 6-8), host only: choose one bit width per block so that the
 * summed sensitivity is minimal and the summed memory stays within the budget,
 *     min  sum_i s[i][c_i]   s.t.  sum_i mem[i][c_i] <= budget,   c_i in {0 .. n_choices-1}.
 * Solved exactly as a multiple-choice knapsack by dynamic programming over memory in units of the
 * greatest common divisor of the memory differences (blocks of one model share their shapes, so the
 * table is tiny); ties are broken towards less memory, then towards the lower choice index in the
 * earlier block.
 *   h_widths       HOST [n_choices]           the candidate widths, e.g. {2, 4} (B of Eq. 8)
 *   h_sensitivity  HOST [layers][n_choices]   s_{i,b} of Eq. 5 (finite, any sign)
 *   h_mem_bytes    HOST [layers][n_choices]   Mem of block i at width b
 *   h_fbit_out     HOST [layers]              chosen width per block (a pmkvq_config.fbit array)
 *   h_cost_out     HOST, may be NULL          the minimal summed sensitivity
 * Returns PMKVQ_ERR_CAPACITY if even the smallest choice of every block exceeds the budget and
 * PMKVQ_ERR_INVALID_ARG for bad arguments or a table beyond 2^26 cells. */
pmkvq_status pmkvq_allocate_bits(int32_t layers, int32_t n_choices, const uint8_t *h_widths,
                                 const double *h_sensitivity, const uint64_t *h_mem_bytes, uint64_t budget_bytes,
                                 uint8_t *h_fbit_out, double *h_cost_out);

const char *pmkvq_status_string(pmkvq_status s);

#ifdef __cplusplus
}
#endif
#endif /* PMKVQ_H_ */

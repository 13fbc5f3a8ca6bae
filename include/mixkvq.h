/*
 * mixkvq.h — C ABI of the MixKVQ decode hot path for NVIDIA B200 (sm_100a).
 *
 * MixKVQ (arxiv 2512.19206) keeps the KV cache of a decoder in three stores per (layer, batch element,
 * KV head) "stream" (Appendix D, "Storage Layout"): bit-packed low-precision codes, the critical key
 * channels in BF16, and a full-precision residual window of the newest <= R tokens.  This library
 * implements the three data-parallel steps of one decode step on that cache:
 *
 *   mixkvq_select_channels   query-aware key-channel scoring and three-tier assignment (Section 4.2)
 *   mixkvq_quantize_append   append to the residual window and, every R tokens, quantize and pack
 *                            (Section 4.2 workflow, Eq. 2; Appendix D.1 lazy update, D.2 accumulator)
 *   mixkvq_decode_attention  softmax(q K~^T * scale) V~ over the mixed-precision cache (Eq. 1, Eq. 3)
 *
 * Conventions
 *   - Every pointer named *_dev is DEVICE memory, owned by the caller, 16-byte aligned.  The library
 *     allocates no device memory and frees none.  `mixkvq_cache*` is a small HOST object.
 *   - bf16 tensors are passed as `const void*` (raw 16-bit bfloat16, row-major, innermost dim = head_dim).
 *   - `stream` is a `cudaStream_t` passed as `void*` (NULL = default stream).  All work is enqueued on
 *     it; only mixkvq_query_status synchronizes.
 *   - Every function returns MIXKVQ_OK (0) or a negative MIXKVQ_E_* code.  Nothing aborts, traps or
 *     throws.  Conditions discovered on the device (extras arena full, a staged copy that never arrived)
 *     set a sticky device status word that mixkvq_query_status returns.
 *   - All sequences of the batch have the same length (the library tracks it per layer on the host).
 *   - head_dim must be 128.
 */
#ifndef MIXKVQ_H_
#define MIXKVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MIXKVQ_OK = 0,
  MIXKVQ_E_INVALID_ARG = -1,          /* null pointer, bad dimension, layer out of range            */
  MIXKVQ_E_UNSUPPORTED = -2,          /* head_dim != 128, v_bits not 2 or 4, unsupported R, G or layout */
  MIXKVQ_E_ALIGNMENT = -3,            /* a device pointer is not 16-byte aligned                     */
  MIXKVQ_E_BUFFER_TOO_SMALL = -4,     /* cache memory or attention workspace smaller than required   */
  MIXKVQ_E_CAPACITY = -5,             /* append would exceed max_tokens                              */
  MIXKVQ_E_CUDA = -6,                 /* a CUDA runtime call or kernel launch reported an error: an
                                         append may then have advanced part of the way (the handle
                                         counts what was enqueued before the failing launch), so the
                                         layer's contents are undefined until mixkvq_cache_reset      */
  MIXKVQ_E_EMPTY = -7,                /* attention or selection requested on a layer with no tokens  */
  MIXKVQ_E_BUILTIN_SCRATCH = -8       /* mixkvq_decode_attention_noalloc: batch * n_kv_heads exceeds
                                         MIXKVQ_NOALLOC_MAX_STREAMS                                  */
};

/* bits of the sticky device status word */
enum {
  MIXKVQ_DEV_EXTRAS_FULL = 1,         /* a block's promoted channels did not fit the stream's extras arena.  The
                                         block's base part is written as usual, but nothing goes to the arena and the
                                         block's table entry records no promoted channel (n16 = n4 = 0): its BF16-tier
                                         channels then read as 0 and its UINT4 channels lose their high plane, so the
                                         layer's attention is wrong from that block on, until the cache is reset
                                         (with a larger extras_budget_bytes).  Earlier blocks are unaffected            */
  MIXKVQ_DEV_COPY_TIMEOUT = 2         /* a bounded wait (for a staged bulk copy, or for the partner warp of a pair) ran out:
                                         the warps concerned contributed nothing to that call's output, which is
                                         therefore wrong (0 where no warp contributed); later calls are unaffected    */
};

typedef struct mixkvq_config {
  int32_t n_layers;
  int32_t batch;                      /* B                                                           */
  int32_t n_q_heads;                  /* Hq, a multiple of n_kv_heads, Hq/Hkv <= 8                   */
  int32_t n_kv_heads;                 /* Hkv                                                         */
  int32_t head_dim;                   /* D, must be 128                                              */
  int32_t max_tokens;                 /* capacity per sequence                                       */
  int32_t residual_len;               /* R (Section 5.1: 128): multiple of 32, <= 256, multiple of G */
  int32_t group_size;                 /* G (Section 5.1: 32): 32, 64 or 128                          */
  int32_t v_bits;                     /* value bit-width: 2 (Section 4.2), or 4 (fragment layout only; stored as
                                         two 2-bit planes, the value scale must then stay below 2^7)  */
  int32_t score_bits;                 /* B of the sensitivity score S_d (Section 4.2), 2 or 4        */
  float tau_bf16;                     /* A_d >  tau_bf16            -> BF16                          */
  float tau_u4;                       /* tau_u4 < A_d <= tau_bf16   -> UINT4, else UINT2             */
  int32_t importance_mode;            /* 0: |q| accumulated within the current window (Section 4.2);
                                         1: cumulative over the whole history (Appendix D.2);
                                         2: error-only ablation (Appendix E): I_d = 1, A_d = S_d     */
  int32_t block_layout;               /* 0: fragment layout (any R; mma.sync attention kernel), the default;
                                         1: tile layout (R must be 128; tcgen05 attention kernel)        */
  uint64_t extras_budget_bytes;       /* per stream, for promoted channels; 0 = library default
                                         (1/8 of the bf16 size of max_tokens keys)                   */
  int32_t budget_bf16;                /* fixed-budget form of the tier rule of Section 4.2: when budget_bf16 +     */
  int32_t budget_u4;                  /* budget_u4 > 0 the thresholds are ignored; the budget_bf16 channels of highest
                                         salience A_d of a window go to BF16, the next budget_u4 to UINT4, the rest to
                                         UINT2 (equal saliences: lower channel first).  Every block then has the same
                                         tier counts.  Sum <= 128                                       */
  int32_t sink_len;                   /* sink tokens (the "sink length" of the settings in Appendix E): the first sink_len
                                         tokens of every sequence stay in bf16 for good, outside the residual window, the
                                         importance accumulator and the quantized blocks.  0, or a multiple of 32 <= 256 */
  int32_t reserved;                   /* must be 0                                                    */
} mixkvq_config;

typedef struct mixkvq_cache mixkvq_cache;

/* Byte offsets (from the start of the cache memory) and strides of one layer's arrays, for tools
 * and tests that inspect the cache.  The element formats are part of the library's documentation. */
typedef struct mixkvq_layout_desc {
  uint64_t state_off, state_stride;       /* per stream: acc fp64[128], cnt u32, extras_used16 u32   */
  uint64_t table_off, table_stride;       /* per stream: max_blocks entries of 8 bytes               */
  uint64_t resk_off, resk_stride;         /* per stream: [R][128] bf16                               */
  uint64_t resv_off, resv_stride;         /* per stream: [R][128] bf16                               */
  uint64_t base_off, base_stride;         /* per stream: max_blocks blocks of base_bytes             */
  uint64_t extras_off, extras_stride;     /* per stream: extras arena                                */
  uint64_t base_bytes;                    /* size of one block's fixed part                          */
  uint32_t max_blocks, n_streams;
  uint32_t n_blocks, residual_tokens;     /* current fill of sequence 0 (mixkvq_sequence_fill: any)  */
  uint64_t sink_off, sink_stride;         /* per stream: [sink_len][128] bf16 keys, then the same for values */
  uint32_t sink_tokens, sink_len;         /* sink rows filled so far, and their capacity              */
} mixkvq_layout_desc;

/* Sizes the caller must provide: the cache memory for all layers and the workspace of one
 * mixkvq_decode_attention call (split partials).  Host-only, no CUDA call. */
int mixkvq_cache_bytes(const mixkvq_config* cfg, size_t* cache_bytes, size_t* attn_workspace_bytes);

/* Creates the host handle over caller-owned device memory and enqueues the zeroing of the per-stream
 * state on `stream`.  cache_dev must hold at least the size reported by mixkvq_cache_bytes. */
int mixkvq_cache_init(const mixkvq_config* cfg, void* cache_dev, size_t bytes, void* stream, mixkvq_cache** out);

/* Frees the host handle only. */
int mixkvq_cache_destroy(mixkvq_cache* cache);

/* Empties one layer (layer >= 0) or all layers (layer < 0): lengths to zero, state re-zeroed on `stream`. */
int mixkvq_cache_reset(mixkvq_cache* cache, int layer, void* stream);

/* (1) Section 4.2: I_d (mean |q| over the window and the GQA group), S_d (key range over the window
 * divided by 2^score_bits - 1), A_d = I_d * S_d, and the tier of every key channel for the CURRENT
 * residual window of `layer`; a pure function of the cache state.
 *   tiers_dev    [B, Hkv, 128] uint8: 0 = UINT2, 1 = UINT4, 2 = BF16
 *   salience_dev [B, Hkv, 128] double A_d, or NULL */
int mixkvq_select_channels(mixkvq_cache* cache, int layer, uint8_t* tiers_dev, double* salience_dev, void* stream);

/* Stateless form of (1) on explicit windows: q_dev [B, Hq, Lq, 128] bf16, k_dev [B, Hkv, Lk, 128] bf16. */
int mixkvq_select_channels_raw(const void* q_dev, const void* k_dev, int batch, int n_q_heads, int n_kv_heads,
                               int lq, int lk, int score_bits, float tau_bf16, float tau_u4,
                               uint8_t* tiers_dev, double* salience_dev, void* stream);

/* (2) Appends n_tokens (1 = decode step, > 1 = prefill / bulk) post-RoPE tokens to `layer`, in token order:
 * for each token, if the residual window already holds R tokens it is first scored, quantized (keys per
 * channel at the tier's bit-width, values per token at 2 bits, groups of G, Eq. 2) and packed; then the
 * token is stored in the window and |q| is added to the importance accumulator.
 * Complete windows of a long append are quantized straight from the tensors (the prefill path); the result is byte for
 * byte that of n_tokens single appends.
 *   k_dev, v_dev [B, Hkv, n_tokens, 128] bf16;  q_dev [B, Hq, n_tokens, 128] bf16 */
int mixkvq_quantize_append(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                           int n_tokens, void* stream);

/* (3) Eq. 1 for one decode step of `layer` over [packed blocks, residual window], keys and values
 * dequantized on the fly (Eq. 3).
 *   q_dev [B, Hq, 128] bf16  ->  out_dev [B, Hq, 128] float
 *   workspace_dev: at least attn_workspace_bytes (mixkvq_cache_bytes); contents are scratch
 * Numeric range: the tensor-core operands are fp16, so |q| must stay below 4094, a stored key scale below 2^11 and a
 * stored value scale below 2^9 (value ranges up to about 1500); beyond that the output overflows to inf or NaN.
 * The kernels are launched with programmatic stream serialization and wait on the device for all earlier work of
 * the stream before they read q_dev or write anything, so stream order holds as for any other launch.  One access comes
 * before that wait: the first packed blocks of the layer are requested early unless the call this library enqueued last
 * on this handle wrote packed blocks of this layer (a flush; initialisation and reset count for all layers).  Cache
 * memory is written through this library only; a caller that writes it by other means (restoring saved cache bytes with
 * a kernel of its own, say) calls mixkvq_cache_written_externally before the next attention call.
 * No wait inside the kernels is unbounded: a staged copy or a hand-over between two warps that has not arrived after
 * 2^21 polls (each poll suspends the thread for up to about a microsecond: two seconds at most, milliseconds if the
 * polls return at once) sets MIXKVQ_DEV_COPY_TIMEOUT and the call returns. */
int mixkvq_decode_attention(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev, float softmax_scale,
                            void* workspace_dev, size_t workspace_bytes, void* stream);

/* (2) + (3) fused for one decode step of `layer`: appends the step's token (k_dev, v_dev [B, Hkv, 1, 128],
 * q_dev [B, Hq, 1, 128] bf16, flushing the residual window first if it is full) and attends with the same q_dev.
 * The cache state and out_dev are exactly those of mixkvq_quantize_append(n_tokens = 1) followed by
 * mixkvq_decode_attention; the attention kernel stores the token and updates the importance accumulator itself
 * (Appendix D.1, D.2), which saves a kernel launch per layer. */
int mixkvq_decode_step(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                       float* out_dev, float softmax_scale, void* workspace_dev, size_t workspace_bytes, void* stream);

/* (2) for a batch whose sequences differ in length (the serving setting of the efficiency experiment: requests of
 * unequal length share a batch).  Sequence b takes the first n_tokens_host[b] tokens (0 <= n_tokens_host[b] <=
 * n_tokens_max; 0 = the sequence takes no token in this call) of its rows of the tensors:
 *   k_dev, v_dev [B, Hkv, n_tokens_max, 128], q_dev [B, Hq, n_tokens_max, 128] bf16; n_tokens_host: HOST array [B].
 * Every sequence keeps its own number of packed blocks, residual tokens and sink rows; each is flushed when ITS window
 * is full, exactly as if it were alone in the batch (the bytes of its streams equal those of a batch-1 cache fed the
 * same tokens).  Neighbouring sequences with the same fill and the same count go through the kernels together, so a
 * batch of equal lengths costs what mixkvq_quantize_append costs (which is this call with equal counts).
 * The capacity check covers every sequence before anything is enqueued.
 * After sequences have diverged, mixkvq_decode_attention, mixkvq_decode_step and mixkvq_select_channels work per
 * sequence: the attention kernel reads every sequence's fill from a table in device memory (written on the stream as
 * kernel arguments, no copy) and splits the positions of all streams evenly over its CTAs; a sequence without tokens
 * gets an all-zero output.  Restrictions of a diverged batch: fragment layout, the default or the split-only
 * attention kernel, B <= 128 (MIXKVQ_E_UNSUPPORTED otherwise). */
int mixkvq_quantize_append_ragged(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev,
                                  int n_tokens_max, const int32_t* n_tokens_host, void* stream);

/* Fill of sequence b of a layer (any pointer may be NULL). */
int mixkvq_sequence_fill(const mixkvq_cache* cache, int layer, int b, uint32_t* n_blocks, uint32_t* residual_tokens,
                         uint32_t* sink_tokens);

/* Decode attention for a context whose tokens are spread over several caches (one per GPU: a sequence split for
 * contexts beyond one GPU's memory).  Eq. 1 over this cache's tokens alone, in the form the merge needs:
 *   out_dev [B, Hq, 128] float: softmax-weighted values over this cache's tokens (normalised by this cache's own
 *   denominator);  lse_dev [B, Hq] float: natural logarithm of that denominator sum_j exp(scale q.k_j).
 * A sequence (or a whole cache) without tokens gives zeros and lse = -inf.  Same kernels, workspace and queue
 * behaviour as mixkvq_decode_attention; fragment layout and the default kernel only (MIXKVQ_E_UNSUPPORTED otherwise). */
int mixkvq_decode_attention_partial(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev, float* lse_dev,
                                    float softmax_scale, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Eq. 1 over the union of disjoint token sets from the per-set results of mixkvq_decode_attention_partial (the
 * log-sum-exp identity): out = sum_r w_r o_r / sum_r w_r, w_r = exp(lse_r - max_r lse_r).  Stateless.
 *   o_parts_dev [n_parts, rows, 128] float, lse_parts_dev [n_parts, rows] float (rows = B * Hq; the layout an
 *   all-gather of the ranks' results produces)  ->  out_dev [rows, 128] float.  Parts with lse = -inf weigh 0;
 *   rows whose parts are all empty come out as zeros.  1 <= n_parts <= 1024. */
int mixkvq_merge_partials(const float* o_parts_dev, const float* lse_parts_dev, int n_parts, int rows, float* out_dev,
                          void* stream);

/* The prefill phase of Section 4.2 for one layer: causal attention of the prompt over itself in full precision (Eq. 1,
 * position i sees positions 0..i), then the prompt's keys and values go into the cache exactly as
 * mixkvq_quantize_append(n_tokens) would put them (complete windows quantized, the last 1..R tokens in the residual
 * window).  The layer must be empty (MIXKVQ_E_UNSUPPORTED otherwise: a later chunk would have to attend to a
 * dequantized cache).
 *   k_dev, v_dev [B, Hkv, n_tokens, 128], q_dev [B, Hq, n_tokens, 128] bf16 (post-RoPE)  ->  out_dev [B, Hq, n_tokens, 128] float
 *   scratch_dev: device memory of at least mixkvq_prefill_scratch_bytes(cfg, n_tokens) bytes, 16-byte aligned, owned by
 *   the caller and free for reuse once the work enqueued by this call has run (it holds K and V of the prompt
 *   rearranged into the tensor core's tile layout); too small -> MIXKVQ_E_CAPACITY.
 * The attention runs on the tcgen05 tensor cores (bf16 products for the logits, fp16 probabilities and values for the
 * output, fp32 accumulation in tensor memory); values must stay inside the fp16 range.  softmax_scale > 0.  A barrier
 * wait that runs out sets MIXKVQ_DEV_COPY_TIMEOUT in the status word and leaves the affected output rows unwritten.
 * Nothing is allocated and nothing synchronises with the host. */
size_t mixkvq_prefill_scratch_bytes(const mixkvq_config* cfg, int n_tokens);
int mixkvq_prefill(mixkvq_cache* cache, int layer, const void* k_dev, const void* v_dev, const void* q_dev, int n_tokens,
                   float* out_dev, float softmax_scale, void* scratch_dev, size_t scratch_bytes, void* stream);

/* Appendix D ("saliency evaluation is performed post-transformation"): for models with rotary position embeddings the
 * scores, the stored keys and the attention all use rotated queries and keys.  These two calls rotate before they
 * append.  k_dev [B, Hkv, n_tokens, 128] and q_dev [B, Hq, n_tokens, 128] (bf16) are rotated IN PLACE: afterwards q_dev
 * holds the rotated queries that mixkvq_decode_attention takes, k_dev the keys that were stored.  v_dev is not touched.
 *   cos_dev, sin_dev: float tables [n_positions, 64] of the caller's angles (row p = position p, entry i the angle of
 *   channel pair (i, i + 64): the "rotate-half" pairing); token j of the call uses row pos0 + j.  The caller owns them.
 *   Arithmetic: y[i] = x[i] c - x[i+64] s, y[i+64] = x[i+64] c + x[i] s, every product and the sum one fp32 operation
 *   rounded to nearest, the result rounded to bf16 (ties to even).  The cache then equals, byte for byte, that of
 *   mixkvq_quantize_append on tensors rotated in this way.
 * Errors as for mixkvq_quantize_append / mixkvq_decode_step; on MIXKVQ_E_CAPACITY nothing was rotated. */
int mixkvq_rope_append(mixkvq_cache* cache, int layer, void* k_dev, const void* v_dev, void* q_dev, const float* cos_dev,
                       const float* sin_dev, int pos0, int n_tokens, void* stream);
/* The same for one decode step: rotates the step's k_dev [B, Hkv, 1, 128] and q_dev [B, Hq, 1, 128] with table row `pos`,
 * then does what mixkvq_decode_step does. */
int mixkvq_rope_decode_step(mixkvq_cache* cache, int layer, void* k_dev, const void* v_dev, void* q_dev,
                            const float* cos_dev, const float* sin_dev, int pos, float* out_dev, float softmax_scale,
                            void* workspace_dev, size_t workspace_bytes, void* stream);

/* (The paper has no counterpart of this entry point; it exists for integration reasons only.)
 * Same computation and same results as mixkvq_decode_attention, for callers that have no way to hand
 * over a workspace: code that runs inside a serving engine's pre-sized memory pool, a plugin that may
 * not call cudaMalloc (or any allocating library routine) once the engine has started, or a host
 * program written in a language binding that exposes no device allocator.  The split partials go to a
 * scratch array that is compiled into the library (static device storage of
 * (1184 + 2 * MIXKVQ_NOALLOC_MAX_STREAMS) * 4160 bytes, about 6.7 MiB, which every GPU that loads the
 * library holds until the process exits).  The call allocates and frees nothing.
 *   - batch * n_kv_heads of the cache must be <= MIXKVQ_NOALLOC_MAX_STREAMS, else
 *     MIXKVQ_E_BUILTIN_SCRATCH is returned and nothing is launched.
 *   - The first call on each device looks up the device address of the scratch array (with that device
 *     current, which must be the device that owns the cache memory: MIXKVQ_E_INVALID_ARG otherwise).  Make
 *     that first call before any stream capture begins, and from one thread: the look-up is not guarded
 *     against concurrent first calls.  The address is kept for the life of the process; it does not
 *     survive a cudaDeviceReset.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (every partial a
 *     call reads was written by that same call), so stale contents of earlier calls are harmless; but
 *     two calls whose kernels overlap on the GPU (different streams, no ordering between them) race on
 *     it and both results are undefined.  Calls on one stream are ordered and safe. */
#define MIXKVQ_NOALLOC_MAX_STREAMS 256
int mixkvq_decode_attention_noalloc(mixkvq_cache* cache, int layer, const void* q_dev, float* out_dev,
                                    float softmax_scale, void* stream);

/* Tells the library that cache memory was written by other means than its own calls since the last call on this
 * handle: the next decode attention of every layer then waits for all earlier work of the stream before its first read. */
int mixkvq_cache_written_externally(mixkvq_cache* cache);

/* Test hook for the give-up path of the decode-attention kernel (fragment layout) and of the prefill attention.  While
 * extra_bytes > 0 (a multiple of 16), the barrier of the first staged copy of every warp pair (decode) or of every
 * CTA's first key tile (prefill) is armed for extra_bytes more than the copy delivers, so it never completes, and every
 * wait gives up after max_polls polls (0: the default): the call returns, the device status word carries
 * MIXKVQ_DEV_COPY_TIMEOUT, the decode output rows are zero and the prefill output is left unwritten.  Nothing faults or
 * hangs: the copies themselves are the normal ones.  (0, 0) restores normal operation. */
int mixkvq_test_arm_copy_timeout(mixkvq_cache* cache, uint32_t extra_bytes, uint32_t max_polls);

/* Selects the decode-attention kernel: 0 = tensor-core kernel (default), 1 = plain-ALU kernel
 * (kept for comparison; same results within tolerance, much slower), 2 = the tensor-core split kernel
 * alone: the split partials stay in the workspace and out_dev is NOT written (for timing that kernel). */
int mixkvq_set_attention_kernel(mixkvq_cache* cache, int kind);

/* Synchronizes `stream`, then returns the sticky device status word (MIXKVQ_DEV_* bits). */
int mixkvq_query_status(mixkvq_cache* cache, int* device_status, void* stream);

/* Where one layer's arrays live inside the cache memory, and how full the layer is. */
int mixkvq_cache_describe(const mixkvq_cache* cache, int layer, mixkvq_layout_desc* out);

/* Number of kernels launched by this handle since it was created (diagnostic). */
uint64_t mixkvq_launch_count(const mixkvq_cache* cache);

const char* mixkvq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MIXKVQ_H_ */

/*
 * kvq.h -- C ABI of the B200 (sm_100a) adaptive mixed-precision KV cache.
 *
 * The library implements the data-parallel hot path of "Don't Waste Bits!"
 * adaptive KV-cache quantization:
 *
 *   features --(controller MLP, Eq. 19-23)--> bit-width per token in {2,4,8,16}
 *   K,V rows --(Q_b of Eq. 24, append of Eq. 4)--> packed mixed-precision cache
 *   query    --(decode attention, Eq. 5)--> output, reading that cache
 *
 * Quantizer (the paper names Q_b in Eq. 24 without defining it; this is the
 * reading the library implements): per token and per KV head, asymmetric
 * min-max over the 64 head channels; scale = (max-min)/(2^b-1) computed in
 * fp32 and stored as fp16; zero-point = row minimum (fp16, -0 stored as +0);
 * code_i = clamp(rint((x_i-min) * (1/scale_fp16)), 0, 2^b-1), ties to even;
 * dequantized value = code*scale + zero-point.  16 "bits" keeps the fp16 row.
 * One bit-width per token is used for its K row and its V row, in every KV
 * head.  Class index <-> bit-width: 0,1,2,3 <-> 2,4,8,16 (Algorithm 1).
 *
 * Store: one pool per precision; the rows of one (layer, sequence, KV head,
 * precision) stream are kept in slot order in 64 KB blocks of a common arena
 * that are taken when an append first reaches them; slot = number of earlier
 * tokens of that (layer, sequence) with the same precision.  A per-token index
 * word (pool << 30 | slot) is kept per (layer, sequence, position).
 *
 * Conventions
 *   - Every function returns 0 (KVQ_OK) or a negative KVQ_ERR_* code, except
 *     kvq_strerror.  Nothing throws, aborts or traps the device.
 *   - "dev" pointers are device memory owned by the caller (for instance a
 *     torch tensor's data_ptr()) on the device that was current at
 *     kvq_create; they must stay valid until the work queued on `stream` has
 *     finished.  "host" pointers are ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls that take a stream only enqueue work; they do not synchronize.
 *     Calls without a stream argument synchronize the device.
 *   - All sequences of the batch advance together: every append adds the same
 *     number of tokens to each of the `batch` sequences of that layer.
 *   - fp16 tensors are IEEE binary16, row-major, innermost dimension last.
 *   - The handle is not thread-safe; use one handle from one thread at a time, and queue its calls on one
 *     stream (or order the streams yourself): the calls share scratch buffers of the handle (class bytes,
 *     histograms and arrival counters of the append, partial records of the attention, the lengths ring).
 */
#ifndef KVQ_H
#define KVQ_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVQ_OK                 0
#define KVQ_ERR_ARG           -1   /* NULL pointer, value out of range, unsupported shape   */
#define KVQ_ERR_CAPACITY      -2   /* append would exceed max_ctx                           */
#define KVQ_ERR_NO_CONTROLLER -3   /* controller weights were never set                     */
#define KVQ_ERR_CUDA          -4   /* a CUDA call failed; see kvq_last_cuda_error           */
#define KVQ_ERR_EMPTY         -5   /* decode attention on a layer that holds no token       */
#define KVQ_ERR_DEVICE_FLAG   -6   /* a kernel recorded a problem (e.g. a bit-width not in
                                      {2,4,8,16}); see kvq_device_status                     */
#define KVQ_ERR_NOMEM         -7   /* host or device allocation failed                      */
#define KVQ_ERR_TOO_LARGE     -8   /* problem exceeds the fixed scratch of kvq_decode_attn_static */

typedef struct kvq_ctx kvq_ctx;    /* opaque; owned by the library */

/* Row size of the canonical export format, bytes per (token, KV head, tensor). */
#define KVQ_EXPORT_ROW_BYTES 128

/*
 * Create a cache for `layers` layers, `batch` sequences, `q_heads` query heads
 * sharing `kv_heads` KV heads (q_heads % kv_heads == 0; query head h reads KV
 * head h / (q_heads/kv_heads)), head_dim == 64, up to `max_ctx` tokens per
 * sequence (Eq. 4: the cache that decode steps append to).  Allocates the
 * arena of packed rows at its worst-case size on the current device (about 504
 * bytes per token, KV head and layer: every token could take any precision)
 * plus block tables, index, counters and split-attention scratch, and zeroes
 * them.  *out receives the handle.  KVQ_ERR_ARG for unsupported shapes,
 * KVQ_ERR_NOMEM / KVQ_ERR_CUDA if allocation fails (nothing is leaked).
 */
int kvq_create(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim,
               int max_ctx, int batch);

/*
 * The same with a chosen budget for the packed rows.  The rows live in an arena of 64 KB
 * blocks; a block serves one (layer, sequence, KV head, precision) stream and is taken from
 * the arena when an append first reaches it, so the memory in use is the sum of the stored row
 * bytes (40 / 72 / 136 / 256 per token and KV head, against 256 for an fp16 cache) plus at most
 * one partly filled block per stream -- the footprint reduction the paper's abstract claims,
 * measurable with kvq_arena_usage.  arena_bytes is rounded down to whole blocks; 0 means the
 * worst case (what kvq_create takes).  An append that finds the arena exhausted stores nothing
 * for the tokens that did not fit, sets the device flag KVQ_FLAG_ARENA_FULL (see
 * kvq_device_status) and leaves the cache unusable until kvq_reset.
 */
int kvq_create_arena(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim,
                     int max_ctx, int batch, uint64_t arena_bytes);

/*
 * The same with a chosen granularity of the min-max quantizer (Eq. 24 only names Q_b and leaves its
 * granularity open; the related work of Section 2 uses finer-grained scales).  scale_groups = 1: one {scale,
 * zero-point} pair per (token, KV head) row of 64 channels, what kvq_create and
 * kvq_create_arena build.  scale_groups = 2: one pair per group of 32 consecutive channels
 * (channels 0..31 and 32..63), each group quantized by the row quantizer on its own values; the
 * codes keep their place, a stored row grows by 8 bytes (48 / 80 / 144 / 256 bytes per token and
 * KV head) and a 64 KB block holds 80 / 50 / 28 / 16 tiles.  Every other entry point behaves the
 * same; the export calls return 2 * scale_groups meta words per (token, KV head, tensor).  Any
 * other scale_groups is KVQ_ERR_ARG.
 */
int kvq_create_grouped(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim,
                       int max_ctx, int batch, uint64_t arena_bytes, int scale_groups);

/*
 * The same with PER-CHANNEL KEYS, the granularity of the key quantizers in the related work the paper cites in
 * Section 2 (Eq. 24 only names Q_b).  Tokens still go to the pool of their bit-width and take slots in position
 * order; the slots of a (sequence, KV head, precision) stream are cut into windows of 16.  In a complete window
 * every key CHANNEL is quantized by the row quantizer over its 16 values (one per token): one {scale,
 * zero-point} pair per channel and window, codes as before.  The keys of the stream's last, incomplete window
 * wait as fp16 rows and are packed when the window fills; the decode calls read them as they are.  Values keep
 * one pair per token.  A stored row takes 52 / 84 / 148 / 256 bytes per token and KV head, plus 6 KB per stream
 * for the waiting rows.  kvq_export_range returns, in k_codes, packed codes for keys in complete windows and the
 * fp16 row otherwise, and {0,0} in k_meta; kvq_export_k_channels returns a window's pairs.  kvq_attend_last takes
 * n_queries == 1 only and kvq_workspace_bytes / kvq_create_in do not offer this layout; everything else behaves
 * as with kvq_create_arena.
 */
int kvq_create_perchannel(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim,
                          int max_ctx, int batch, uint64_t arena_bytes);

/*
 * Per-channel keys: the 64 {scale, zero-point} pairs (fp16 bit patterns, host uint16 [64][2]) of window
 * `window` (slots 16 window .. 16 window + 15) of the stream (layer, sequence b, kv_head, bits in {2,4,8}).
 * KVQ_ERR_ARG if the window is not complete or the cache has another layout.  Synchronizes.
 */
int kvq_export_k_channels(kvq_ctx* ctx, int layer, int b, int kv_head, int bits, int window, uint16_t* host_meta);

/*
 * The same cache inside device memory that the caller owns (for instance one torch tensor), so that
 * the library itself allocates no device memory for it.  kvq_workspace_bytes gives the size the other
 * arguments need (host uint64; it reads the current device's properties, allocates nothing).
 * kvq_create_in takes `workspace`, a dev pointer aligned to 256 bytes with at least that many bytes,
 * carves every buffer of the handle out of it and zeroes what kvq_create zeroes.  The memory must stay
 * valid until kvq_destroy, which leaves it alone.  KVQ_ERR_NOMEM if workspace_bytes is too small,
 * KVQ_ERR_ARG for a NULL or misaligned workspace; otherwise as kvq_create_grouped.
 */
int kvq_workspace_bytes(int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                        uint64_t arena_bytes, int scale_groups, uint64_t* bytes_out);
int kvq_create_in(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim,
                  int max_ctx, int batch, uint64_t arena_bytes, int scale_groups,
                  void* workspace, uint64_t workspace_bytes);

/*
 * Arena fill: blocks handed out so far, blocks available, bytes per block (host uint64, any
 * may be NULL).  Synchronizes.
 */
int kvq_arena_usage(kvq_ctx* ctx, uint64_t* blocks_in_use, uint64_t* blocks_total, uint64_t* block_bytes);

/* Free everything the handle owns.  NULL is a no-op.  Synchronizes the device. */
int kvq_destroy(kvq_ctx* ctx);

/*
 * Install the controller of Eq. 19-21: a 4 -> hidden -> hidden -> 4 MLP with
 * ReLU after the first two layers.  Host pointers, fp32, row-major [out][in]:
 * W1 [hidden][4], b1 [hidden], W2 [hidden][hidden], b2 [hidden], W3 [4][hidden],
 * b3 [4].  The values are copied to the device; 1 <= hidden <= 128 (the paper's
 * width; the whole parameter block is kept in shared memory).
 */
int kvq_set_controller(kvq_ctx* ctx, int hidden,
                       const float* W1, const float* b1,
                       const float* W2, const float* b2,
                       const float* W3, const float* b3);

/*
 * Controller decision (Eq. 19-23) for n tokens.  feats: dev fp32 [n][4].
 * bits: dev uint8 [n], receives 2, 4, 8 or 16.  logits_opt: dev fp32 [n][4] or
 * NULL.  Arithmetic: fp32, each product rounded, then each sum rounded, inputs
 * in ascending order starting from the bias; argmax takes the lowest class on
 * ties; a NaN logit selects 16.  n == 0 is a no-op.
 */
int kvq_select_bits(kvq_ctx* ctx, const float* feats, int n, uint8_t* bits,
                    float* logits_opt, void* stream);

/*
 * Quantize-append (Eq. 24, then Eq. 4) of n_new tokens per sequence to `layer`.
 * K, V: dev fp16 [batch][n_new][kv_heads][64].  bits: dev uint8 [batch][n_new]
 * with values in {2,4,8,16}; any other value stores the token as fp16 and sets
 * the device flag KVQ_FLAG_BAD_BITS.  KVQ_ERR_CAPACITY (nothing is queued) if
 * the layer would exceed max_ctx.  n_new == 0 is a no-op.
 */
int kvq_append(kvq_ctx* ctx, int layer, const void* K, const void* V,
               const uint8_t* bits, int n_new, void* stream);

/*
 * Same as kvq_select_bits followed by kvq_append, with the controller (Eq. 19-23)
 * evaluated inside the kernels that quantize and pack (Eq. 24): feats is dev fp32
 * [batch][n_new][4].  bits_out_opt (dev uint8 [batch][n_new] or NULL) receives
 * the decisions.  Launches: one kernel for up to 256 new tokens per sequence (a
 * decode step included); a longer prefill runs two: the controller, which also
 * counts the classes per chunk of tokens and reserves the arena blocks, and the
 * quantize-and-pack kernel, which reads the classes (one byte per token) back
 * from a scratch array because slots are handed out in position order across
 * chunks.
 */
int kvq_append_fused(kvq_ctx* ctx, int layer, const void* K, const void* V,
                     const float* feats, int n_new, uint8_t* bits_out_opt, void* stream);

/*
 * Ragged batches: the same append with a different number of new tokens per sequence.  K, V
 * (and bits, or feats) keep n_max rows per sequence; sequence b appends its first
 * host_lens[b] rows (host int [batch], 0 <= host_lens[b] <= n_max), the rest is ignored.
 * Exactly one of bits (dev uint8 [batch][n_max]) and feats (dev fp32 [batch][n_max][4], the
 * controller decides; bits_out_opt as in kvq_append_fused) is given, the other is NULL.
 * Afterwards the sequences of the layer differ in length: kvq_seq_lens reports them,
 * kvq_seq_len the longest, kvq_decode_attn attends for every sequence over what it holds
 * (a sequence that holds nothing gets a zero row), kvq_export_range and kvq_attend_last are
 * limited by the shortest.  Does not synchronize: host_lens is copied before the call returns (the caller may
 * reuse it at once) and travels to the device behind the work already queued on `stream`.
 */
int kvq_append_ragged(kvq_ctx* ctx, int layer, const void* K, const void* V, const uint8_t* bits,
                      const float* feats, int n_max, const int* host_lens, uint8_t* bits_out_opt,
                      void* stream);

/* Tokens cached per sequence in `layer` (host int [batch]; host-side mirror, no device access). */
int kvq_seq_lens(kvq_ctx* ctx, int layer, int* host_lens_out);

/*
 * Decode-step attention (Eq. 5) of one query row per (sequence, query head)
 * over every token cached in `layer`, dequantizing on the fly:
 * O = Softmax(q K^T / 8) V.  Q, O: dev fp16 [batch][q_heads][64].  fp32
 * accumulation, online softmax; the work is split over warps (see kvq_set_splits); the warp
 * that delivers the last partial result of a (sequence, query head) merges them, all in one
 * kernel.
 * KVQ_ERR_EMPTY if the layer holds no token.
 */
int kvq_decode_attn(kvq_ctx* ctx, int layer, const void* Q, void* O, void* stream);

/*
 * kvq_decode_attn that also returns the attention-variance feature of Eq. 16 for the step's
 * tokens: var_out (dev fp32 [batch]) receives V = (1/h) sum over the query heads of the variance
 * of that head's attention weights over the cached tokens of the sequence.  (The paper takes
 * the last transformer layer; which layer to ask is the caller's choice.)  One extra
 * multiply-add per cached token and a small second kernel.
 */
int kvq_decode_attn_var(kvq_ctx* ctx, int layer, const void* Q, void* O, float* var_out, void* stream);

/*
 * The controller's input vector of Eq. 17 for n tokens, s_t = [H_t, R_t, V_t, C_t], computed on
 * the device.  No handle is needed.
 *   logits      dev [n][vocab], fp16 (logits_are_fp32 == 0) or fp32: the pre-softmax scores z_t
 *   H_t         entropy of Softmax(z_t), natural logarithm (Eq. 14)
 *   C_t         confidence; the paper names it without a definition: max_v Softmax(z_t)_v
 *   token_ids   dev int32 [n], counts dev uint32 [vocab], total_count = N, observed_tokens =
 *               |V_obs|: R_t = -log((counts[token] + 1) / (N + |V_obs| + 1)) (Eq. 15); a token id outside
 *               [0, vocab) is taken as never seen (count 0)
 *   attn_var_opt dev fp32 [n] or NULL (then V_t = 0): the attention variance of Eq. 16, e.g. from
 *               kvq_decode_attn_var
 *   feats       dev fp32 [n][4] in the order H, R, V, C of Eq. 17 (16-byte aligned)
 * The logits are read once; rows are read with 16-byte loads when vocab % 8 == 0 and the base
 * is 32-byte aligned.  Masked entries (-inf) count as probability zero (p log p = 0); a row must
 * keep at least one finite entry (a row that is masked throughout has no distribution: its H and C
 * are unspecified).  fp32 logits below -1e28 are treated as masked.  The library treats the controller's inputs as four opaque numbers, so a
 * controller must have been trained on this order to be fed from here.
 */
int kvq_token_features(const void* logits, int logits_are_fp32, int n, int vocab,
                       const int32_t* token_ids, const uint32_t* counts, uint64_t total_count,
                       uint32_t observed_tokens, const float* attn_var_opt, float* feats, void* stream);

/*
 * Causal attention of several query rows over the cache (Eq. 5 applied at each of the last
 * n_queries cached positions): query row i belongs to the token at position len - n_queries + i
 * and attends over positions <= its own, the rows after it stay invisible.  This is what a
 * speculative or chunked decode step needs after appending n_queries tokens at once.
 * Q, O: dev fp16 [batch][n_queries][q_heads][64].  1 <= n_queries <= cached length
 * (KVQ_ERR_ARG otherwise); n_queries == 1 is kvq_decode_attn.  Rows are served eight per
 * launch; every row reads the cache on its own (no sharing between rows).
 */
int kvq_attend_last(kvq_ctx* ctx, int layer, const void* Q, void* O, int n_queries, void* stream);

/*
 * kvq_decode_attn without any buffer that had to be allocated for it.  (No counterpart in
 * the paper: this is a packaging variant of the call above, same arithmetic, same result.)
 *
 * Who it is for: code that must not touch the CUDA allocator when it runs -- a serving loop
 * under a "no allocation after start-up" rule, a plug-in inside a process whose device
 * memory is entirely owned by another allocator, a caller that cannot tolerate the implicit
 * device synchronisation of cudaMalloc/cudaFree.  Such a caller cannot ask a library to
 * reserve per-call or per-handle scratch on its behalf.  Here the split-attention partials
 * and their arrival counters (the only scratch the decode step needs) live in a fixed array
 * that is part of the library image: KVQ_STATIC_MAX_PARTIALS records of 66 floats plus the
 * counters, about 2.2 MB, which every
 * GPU that loads the library holds until the process exits.  The call performs no
 * cudaMalloc, no cudaFree and calls no allocating routine; the handle's store is read as
 * input, Q is read and O is written exactly as in kvq_decode_attn, and none of the
 * handle's own scratch is used.
 *
 * Limit: batch * q_heads * (parts + 1) <= KVQ_STATIC_MAX_PARTIALS, where parts is the number of
 * pieces a (sequence, query head) unit is cut into.  A value given to kvq_set_splits is taken as
 * it is, and KVQ_ERR_TOO_LARGE is returned (nothing is queued) if it does not fit.  In automatic
 * mode the planner picks the best split that fits the array, which may be coarser than what
 * kvq_decode_attn would pick; KVQ_ERR_TOO_LARGE only if 2 * batch * q_heads records do not fit.
 *
 * Set-up: the first call on each device looks up the device address of the array (once
 * per device, with that device current).  Make that first call outside any stream capture.
 *
 * Sharing: every call on a device uses the same array, whatever the handle or stream.
 * Two calls whose kernels overlap on the GPU (different streams, or different threads)
 * race on it; serialise them.  The array keeps the previous call's partials, which is
 * harmless: every record a merge reads is written first by the same call.  Only the arrival
 * counters must be zero when a call starts; they are zero when the library is loaded and
 * each call puts back to zero every counter it used.
 */
#define KVQ_STATIC_MAX_PARTIALS 8192
int kvq_decode_attn_static(kvq_ctx* ctx, int layer, const void* Q, void* O, void* stream);

/*
 * One decode step on device buffers: the controller's decision for the step's `batch` tokens
 * (Eq. 19-23), quantize-append of their K/V rows to `layer` (Eq. 24, Eq. 4), then attention of
 * Q over everything cached in the layer, the new token included (Eq. 5).  Same result as
 * kvq_append_fused with n_new = 1 followed by kvq_decode_attn.  feats dev fp32 [batch][4];
 * K, V dev fp16 [batch][1][kv_heads][64]; Q, O dev fp16 [batch][q_heads][64]; bits_out_opt
 * dev uint8 [batch] or NULL.  Launches: ONE kernel when the keys are quantized per token (one
 * or two scale groups), whatever the lengths and the controller's width: some CTAs of the
 * launch store the token while the others attend over the cache as it was and add the token
 * from its fp16 rows, quantized in registers exactly as it is stored, so the attention does
 * not wait for the store.  (A controller of hidden width 32 is evaluated by every warp that
 * needs the decision; a wider one by the storing CTAs, which publish the class for the
 * attending warps of the same launch: those pick it up at the end of their work through a
 * bounded wait, see KVQ_FLAG_WAIT_TIMEOUT.)  With per-channel keys the two kernels of the two
 * calls, whose launches overlap.  Errors as for the two calls (an empty layer is fine: the step's token is
 * then all there is).
 */
int kvq_decode_step(kvq_ctx* ctx, int layer, const float* feats, const void* K, const void* V,
                    const void* Q, void* O, uint8_t* bits_out_opt, void* stream);

/*
 * One decode step from HOST buffers, copies included (kvq_decode_step on host
 * memory, then a stream synchronization): controller decision for
 * the step's `batch` tokens, quantize-append of their K/V rows to `layer`,
 * attention of Q over the layer, result copied back.  feats host fp32
 * [batch][4]; K, V host fp16 [batch][1][kv_heads][64]; Q host fp16
 * [batch][q_heads][64]; O host fp16 [batch][q_heads][64] (written);
 * bits_out_opt host uint8 [batch] or NULL.  Returns after the stream has been
 * synchronized.  When feats, K, V, Q and O are all page-locked (cudaHostAlloc,
 * cudaHostRegister, a pinned torch tensor) and 16-byte aligned, the kernels read
 * and write them across the bus directly; otherwise the call copies through
 * staging buffers owned by the handle.  Either way every byte of the step's
 * inputs and of its result crosses the bus inside the call.
 */
int kvq_decode_step_host(kvq_ctx* ctx, int layer, const float* feats, const void* K,
                         const void* V, const void* Q, void* O, uint8_t* bits_out_opt,
                         void* stream);

/* Forget all cached tokens of every layer (counters go to 0, every arena block is free again). */
int kvq_reset(kvq_ctx* ctx, void* stream);

/* Tokens cached by the longest sequence of `layer` (host-side mirror; no device access). */
int kvq_seq_len(kvq_ctx* ctx, int layer, int* host_len_out);

/*
 * How kvq_decode_attn cuts the work: 0 = automatic (default): one launch of as many warps as
 * stay resident on the device, each taking an equal share of all (sequence, query head)
 * units; 1..64 = every unit is cut into exactly that many equal parts, one warp each.
 */
int kvq_set_splits(kvq_ctx* ctx, int splits);

/*
 * How a prefill append (more than 256 new tokens per sequence) cuts the new tokens into chunks
 * for slot assignment and packing: 0 = automatic (default: 512-token chunks when that still
 * leaves many CTAs, else 256), 256 or 512 = always that size.  The stored result does not depend
 * on it; the setting exists for tuning and for tests.  Other values: KVQ_ERR_ARG.
 */
int kvq_set_append_chunk(kvq_ctx* ctx, int chunk_tokens);

/*
 * Canonical copy of tokens [pos0, pos0+n) of every sequence of `layer`, for
 * comparison with other implementations.  All outputs are dev pointers:
 *   bits      uint8  [batch][n]                 2,4,8,16
 *   pool_slot uint32 [batch][n]                 pool << 30 | slot
 *   k_codes, v_codes uint8 [batch][n][kv_heads][128]: packed codes, element i in
 *             bits [(i*b)%8, +b) of byte floor(i*b/8); for b == 16 the fp16 row,
 *             little-endian; bytes past 64*b/8 are zero
 *   k_meta, v_meta  uint16 [batch][n][kv_heads][2]: fp16 bit patterns of
 *             {scale, zero-point}; {0,0} for b == 16.  A cache made with scale_groups = 2
 *             returns [batch][n][kv_heads][2][2]: the pair of channels 0..31, then of 32..63
 * Any output pointer may be NULL to skip it.
 */
int kvq_export_range(kvq_ctx* ctx, int layer, int pos0, int n,
                     uint8_t* bits, uint32_t* pool_slot,
                     void* k_codes, void* v_codes, uint16_t* k_meta, uint16_t* v_meta,
                     void* stream);

/* The same for one token of one sequence, into HOST buffers ([kv_heads][128] and
 * [kv_heads][2 * scale_groups]); synchronizes. */
int kvq_export_token(kvq_ctx* ctx, int layer, int b, int pos,
                     uint8_t* bits, uint32_t* pool_slot,
                     void* k_codes, void* v_codes, uint16_t* k_meta, uint16_t* v_meta);

/*
 * Snapshot of the cache (every layer): the packed rows in use, block tables, per-token index, pool
 * fills and sequence lengths, as one host blob that kvq_load_state puts back, into this handle or into
 * another one created with the same shape arguments and scale_groups (its arena may have a different
 * budget as long as the snapshot's blocks fit).  The controller weights are not part of it.
 * kvq_state_bytes: size of a snapshot taken now (host uint64).  kvq_save_state: host_buf (host memory,
 * host_bytes >= that size) receives it.  kvq_load_state: replaces the handle's contents; KVQ_ERR_ARG
 * if the blob is truncated, was not written by kvq_save_state or belongs to another shape.  All three
 * synchronize the device.
 */
int kvq_state_bytes(kvq_ctx* ctx, uint64_t* bytes_out);
int kvq_save_state(kvq_ctx* ctx, void* host_buf, uint64_t host_bytes);
int kvq_load_state(kvq_ctx* ctx, const void* host_buf, uint64_t host_bytes);

/*
 * Pool fill of `layer`: host_counts (host uint32 [batch][4], may be NULL)
 * receives tokens per precision class; resident_bytes (host, may be NULL) the
 * bytes of packed rows in use, sum over tokens of kv_heads * {40,72,136,256};
 * expected_bits (host, may be NULL) the mean bit-width sum_c count_c*b_c / tokens
 * (the paper's E[b], Eq. 11).  Synchronizes.
 */
int kvq_stats(kvq_ctx* ctx, int layer, uint32_t* host_counts, uint64_t* resident_bytes,
              double* expected_bits);

/*
 * Timing hooks for benchmarks.  While profiling is on, kvq_decode_attn records CUDA events on its
 * stream before and after its kernel (up to 1024 calls are kept; later calls are not recorded).
 * kvq_profile_read synchronizes, adds up the elapsed times of the recorded calls into
 * attn_ms_total (host double, may be NULL), stores their number in calls (host int, may be NULL)
 * and forgets them.
 */
int kvq_set_profiling(kvq_ctx* ctx, int on);
int kvq_profile_read(kvq_ctx* ctx, double* attn_ms_total, int* calls);

/* Device flags recorded by kernels since the last call (host uint32, cleared on read). */
#define KVQ_FLAG_BAD_BITS 1u      /* a bit-width outside {2,4,8,16} was appended (stored as fp16) */
#define KVQ_FLAG_ARENA_FULL 4u    /* an append ran out of arena blocks; the tokens that did not fit are lost */
#define KVQ_FLAG_WAIT_TIMEOUT 2u  /* a bounded wait expired in a decode call (on an async copy, or in
                                     kvq_decode_step on the class that the storing CTAs publish); that
                                     call's output is invalid.  The warp that gave up still hands in an
                                     (empty) partial for the rest of its share, so every arrival counter
                                     the call used is back at zero when it ends and later calls on the
                                     handle are unaffected; kvq_device_status also runs kvq_recover when
                                     it reports this flag. */
int kvq_device_status(kvq_ctx* ctx, uint32_t* host_flags_out);

/*
 * Put the split-attention bookkeeping of the handle back into its start-up state: the arrival counters of
 * the handle's scratch, those of the fixed array of kvq_decode_attn_static on the handle's device (if that
 * call was ever used there) and the device flag word are set to zero.  Cached tokens are untouched.  For use
 * after a decode call was cut short from outside (the process aborted a stream, a debugger killed a
 * kernel); a call that ended by itself, even with KVQ_FLAG_WAIT_TIMEOUT, needs none.  Synchronizes.
 */
int kvq_recover(kvq_ctx* ctx);

/* Bytes of device memory the handle holds (pools + index + scratch). */
int kvq_device_bytes(kvq_ctx* ctx, uint64_t* host_bytes_out);

/* Kernels this handle has launched since creation (for launch accounting). */
int kvq_launch_count(kvq_ctx* ctx, uint64_t* host_count_out);

/* cudaError_t value of the last failing CUDA call of this handle (0 if none). */
int kvq_last_cuda_error(kvq_ctx* ctx);

/* Static, human-readable text for a return code. */
const char* kvq_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* KVQ_H */

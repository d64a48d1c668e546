/*
 * mixattn.h -- C ABI of the MixAttention inference attention library (sm_100a).
 *
 * The library implements the attention + KV-cache path of "Inference-Friendly
 * Models With MixAttention" (arXiv 2409.15012): every layer is either a
 * standard attention layer or a sliding-window layer with window s, and either
 * computes its own KV cache or reuses the cache of an earlier layer
 * (Section 3).  Grouped-query attention maps query head h to KV head
 * h / (n_q_heads / n_kv_heads) (Section 3, last paragraph).
 *
 * Conventions for every call
 *   - returns MIXATTN_OK (0) or a negative MIXATTN_ERR_* code; nothing throws,
 *     aborts or traps.  All validation happens on the host before any launch,
 *     and a call that fails it changes no state.  The one exception is
 *     MIXATTN_ERR_CUDA from a launch or copy the CUDA runtime refused in the
 *     middle of a call: the cache bookkeeping may already have moved, so the
 *     context turns unusable (every later call that would touch the device
 *     returns MIXATTN_ERR_CUDA); destroy it.
 *   - "host" pointers are read (or written) before the call returns.
 *     "device" pointers are borrowed until `stream` has executed the work the
 *     call enqueued.  `stream` is a cudaStream_t passed as void* (NULL = the
 *     legacy default stream).  Calls are asynchronous on that stream.
 *   - a context is not thread-safe; use one stream at a time per context.
 *   - tensors are dense, row-major, in the context's dtype (float or bf16).
 */
#ifndef MIXATTN_H_
#define MIXATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mixattn_ctx mixattn_ctx; /* opaque; owned by the library */

enum { MIXATTN_FULL = 0, MIXATTN_SLIDING = 1 };
enum { MIXATTN_F32 = 0, MIXATTN_BF16 = 1 };
/* How cached keys and values are stored (mixattn_config.kv_format). */
enum {
  MIXATTN_KV_NATIVE = 0,   /* in the context's dtype                                               */
  MIXATTN_KV_FP8_E4M3 = 1  /* quantised: see "Quantised KV storage" below                          */
};

enum {
  MIXATTN_OK = 0,
  MIXATTN_ERR_INVALID_ARG = -1,    /* null pointer, size out of range, duplicate sequence id        */
  MIXATTN_ERR_INVALID_LAYOUT = -2, /* layer layout breaks the rules listed at mixattn_create        */
  MIXATTN_ERR_NOT_OWNER = -3,      /* K/V offered to a layer that reuses another layer's cache      */
  MIXATTN_ERR_OUT_OF_PAGES = -4,   /* the paged pool has too few free pages for the call            */
  MIXATTN_ERR_EMPTY_CONTEXT = -5,  /* decode on a sequence whose cache holds no token               */
  MIXATTN_ERR_BAD_SEQ = -6,        /* sequence id outside 0 .. max_seqs-1                           */
  MIXATTN_ERR_UNSUPPORTED = -7,    /* valid request this library does not implement                 */
  MIXATTN_ERR_CUDA = -8,           /* a CUDA call failed, or the context is host-only               */
  MIXATTN_ERR_TOO_LARGE = -9       /* mixattn_decode_static_scratch: request exceeds the static array */
};

/* One layer of the layout (Section 3: a mix of sliding-window layers, standard
 * layers and layers that reuse a KV cache).  `window` is the paper's s and is
 * ignored for MIXATTN_FULL.  `kv_owner_layer` is the layer whose cache this
 * layer reads: itself, or an earlier layer. */
typedef struct {
  int32_t kind;
  int32_t window;
  int32_t kv_owner_layer;
} mixattn_layer_desc;

typedef struct {
  int32_t n_layers;
  const mixattn_layer_desc* layers; /* host, n_layers entries, copied by create                    */
  int32_t n_q_heads, n_kv_heads;    /* n_q_heads % n_kv_heads == 0                                  */
  int32_t head_dim;                 /* 64 or 128                                                    */
  int32_t dtype;                    /* MIXATTN_F32 or MIXATTN_BF16: type of Q, K, V, out and cache  */
  int32_t max_seqs;                 /* sequence slots 0 .. max_seqs-1                               */
  int32_t page_size;                /* tokens per page of the full-attention cache; must be 16      */
  int32_t n_pages;                  /* physical pages per full-attention owner                      */
  int32_t max_seq_len;              /* longest sequence; 0 = n_pages * page_size                    */
  const int32_t* free_order;        /* host, optional permutation of 0..n_pages-1: initial FIFO
                                       order of the free pages; NULL = 0,1,2,...                    */
  float softmax_scale;              /* 0 = 1/sqrt(head_dim)                                         */
  int32_t device;                   /* CUDA device ordinal; -1 = host-only context that keeps the
                                       cache bookkeeping but launches nothing (append_kv then
                                       ignores k/v; decode and prefill return MIXATTN_ERR_CUDA)     */
  void* arena;                      /* device memory allocated by the caller, 256-byte aligned      */
  size_t arena_bytes;               /* >= mixattn_arena_bytes(); the library never frees it         */
  int32_t chunk_scratch_tokens;     /* K/V rows of scratch kept in the arena for
                                       mixattn_attend_chunk; 0 = that call is unavailable           */
  int32_t kv_format;                /* MIXATTN_KV_NATIVE or MIXATTN_KV_FP8_E4M3                     */
} mixattn_config;

/* Quantised KV storage (kv_format = MIXATTN_KV_FP8_E4M3).
 *
 * Section 2 of the paper ("KV Quantization") names storing the cached keys and
 * values at reduced precision as a technique that combines with MixAttention:
 * it shrinks the cache and the bytes a decode step moves, which Section 1
 * gives as the cost of long-context inference.  The paper fixes no format;
 * this library stores every head vector (one token, one KV head; K and V
 * apart) as head_dim FP8 E4M3 elements (OCP 8-bit float: 1 sign, 4 exponent
 * bits with bias 7, 3 mantissa bits, largest value 448, no infinity) plus one
 * byte holding a shared power-of-two exponent X (stored as X + 127):
 *     X       = floor(log2(max |x|)) - 8, clamped to [-127, 127]; -127 for a zero vector
 *     element = x / 2^X rounded to the nearest E4M3 value, ties to even,
 *               saturating at +-448
 * and a reader sees element * 2^X, which is again a bf16 number.  Cached
 * bytes per token and KV head: 2 * (head_dim + 1) instead of 4 * head_dim.
 * Requirements: dtype MIXATTN_BF16 and head_dim 128 (else
 * MIXATTN_ERR_UNSUPPORTED from create).  Q, K, V and out of every call stay
 * bf16: mixattn_append_kv (and _rope, and the store of mixattn_prefill)
 * quantise on the way in; mixattn_decode reads the quantised cache, widening
 * elements exactly to fp16 for the tensor-core products with Q and P converted
 * to fp16 as well (so |q| must stay below 65504 and max |v| of a row below
 * 2^23); mixattn_attend_chunk reads the cached part dequantised and the
 * chunk's own K/V as given.  mixattn_prefill attends over the K/V it is given,
 * unquantised. */

/* Bytes of device memory a context with this config carves out of `arena`:
 * K/V storage (see mixattn_cache_bytes), the device copy of the block tables
 * and the split-KV workspace.  Writes *out_bytes.  Errors: INVALID_ARG,
 * INVALID_LAYOUT. */
int mixattn_arena_bytes(const mixattn_config* cfg, size_t* out_bytes);

/* Bytes of K/V storage alone: one paged pool of n_pages pages per
 * full-attention owner and one ring of `window` tokens (rounded up to whole
 * 16-token pages) per sequence slot per sliding-window owner (Section 3: a
 * window-s layer only stores the past s tokens).  Layers that reuse a cache
 * add nothing (Section 3: l layers sharing one cache shrink it by 1/l). */
int mixattn_cache_bytes(const mixattn_config* cfg, size_t* out_bytes);

/* Builds a context.  Layout rules (Section 3: a layer may reuse the cache
 * computed by an EARLIER layer), each violation -> MIXATTN_ERR_INVALID_LAYOUT:
 *   0 <= kv_owner_layer <= layer index;  the owner owns itself (no chains);
 *   a reader has its owner's kind and, if sliding, its owner's window >= 1.
 * Other bad fields -> INVALID_ARG.  With device >= 0 the arena is cleared on
 * that device's legacy default stream and create returns after it finished.
 * *out receives the context; the caller releases it with mixattn_destroy. */
int mixattn_create(const mixattn_config* cfg, mixattn_ctx** out);

/* Releases the context's host memory and CUDA events.  The arena is the
 * caller's.  The caller makes sure no work of the context is still running. */
int mixattn_destroy(mixattn_ctx* ctx);

/* Empties sequence slot `seq` in every cache: lengths become 0 and its pages
 * return to the tail of the free FIFO in logical-block order. */
int mixattn_seq_reset(mixattn_ctx* ctx, int32_t seq);

/* Appends new tokens' K/V to the cache OWNED by `layer` (Section 1: keys and
 * values of earlier tokens are cached; Section 3: a sliding-window cache keeps
 * the past s tokens).
 *   seq_ids  host, n_seqs distinct sequence ids
 *   n_new    host, tokens per sequence (>= 0), or NULL for one token each
 *   k, v     device, [sum n_new, n_kv_heads, head_dim], sequences in call order
 * Full-attention owner: token t of a sequence goes to page
 * block_table[t / 16], offset t % 16; a free page is taken from the FIFO head
 * when a sequence first reaches a logical block (sequences in call order,
 * tokens in position order).  All full-attention owners share one block table
 * per sequence.  Sliding owner: token t overwrites ring slot t % window.
 * Errors: NOT_OWNER if the layer reuses another layer's cache, BAD_SEQ,
 * OUT_OF_PAGES (nothing appended), INVALID_ARG (null, duplicates, length
 * beyond max_seq_len). */
int mixattn_append_kv(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                      const int32_t* n_new, const void* k, const void* v, void* stream);

/* mixattn_append_kv with the rotary position embedding fused into the copy
 * (Section 3: the models use RoPE, with a base theta that grows with the
 * context length; the embedding is RoFormer's): before a key row is stored,
 * its channel pairs (2i, 2i+1) are rotated by the angle t * theta^(-2i/d),
 * t the token's position in the sequence and d = head_dim.  Values are stored
 * unchanged.  Angles are reduced in double precision, the rotation runs in
 * fp32 and bf16 rows are rounded once.  (Queries are the caller's: they are
 * never stored.)  rope_theta must be finite and > 1, else INVALID_ARG; all
 * else as mixattn_append_kv. */
int mixattn_append_kv_rope(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                           const int32_t* n_new, const void* k, const void* v, float rope_theta,
                           void* stream);

/* One decode step of `layer` for n_seqs sequences (Section 3).  With n the
 * number of tokens in the cache the layer reads (its owner's, after this
 * step's append) the query sits at position n-1 and attends to keys
 * [0, n) for a standard layer and to the last min(n, window) keys for a
 * sliding-window layer:  out = softmax(scale * q K^T) V  per query head.
 *   q, out   device, [n_seqs, n_q_heads, head_dim]
 * Split-KV flash decoding: partial results go to the context's workspace and a
 * combine pass writes `out`.  Errors: EMPTY_CONTEXT if a sequence has n == 0
 * (nothing is written), BAD_SEQ, INVALID_ARG, CUDA. */
int mixattn_decode(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                   const void* q, void* out, void* stream);

/* One decode step over the layers layer_begin .. layer_end - 1, in order (Section 3, layer by
 * layer as a forward pass visits them; the generation loop of Section 5.4's workload): for each
 * layer, mixattn_append_kv of one new token per sequence if the layer owns its cache, then
 * mixattn_decode.  One call instead of one or two per layer: at small batches issuing the calls
 * is what a step costs.
 *   q, out   host arrays indexed by layer (n_layers entries; only the range is read) of device
 *            pointers, [n_seqs, n_q_heads, head_dim] each
 *   k, v     the same for the new token's K/V, [n_seqs, n_kv_heads, head_dim]; entries of
 *            layers that reuse a cache are ignored and may be NULL
 * The effect is that of the individual calls made one after the other, and the call stops at
 * the first of them that fails, returning its status: layers before it stand (their caches
 * have moved).  *layers_done, if not NULL, receives the number of layers completed.
 * Errors: INVALID_ARG for a bad range or null arrays, else those of the two calls. */
int mixattn_decode_layers(mixattn_ctx* ctx, int32_t layer_begin, int32_t layer_end, int32_t n_seqs,
                          const int32_t* seq_ids, const void* const* q, const void* const* k,
                          const void* const* v, void* const* out, void* stream, int32_t* layers_done);

/* Prompt attention of `layer` for n_seqs sequences that start at position 0
 * (Section 3; causal as in Section 1).  Query i attends to keys j <= i
 * (standard) or i - window < j <= i (sliding window); key tiles wholly outside
 * that band are skipped.
 *   seq_lens host, prompt length S_b of each sequence (>= 1)
 *   q, out   device, [sum S_b, n_q_heads, head_dim], sequences back to back
 *   k, v     device, [sum S_b, n_kv_heads, head_dim]: the K/V computed by the
 *            layer's owner (a reader is handed its owner's tensors)
 * If `layer` owns its cache the call also stores K/V as mixattn_append_kv
 * would (a ring ends up holding the last min(S_b, window) tokens); the
 * owner's cache for these sequences must be empty, else UNSUPPORTED.  A
 * reader stores nothing.  Errors: as append_kv and decode.
 * Performance note: bf16 (head_dim 128 or 64) with 16-byte aligned tensors
 * runs on the tensor cores; fp32 contexts and unaligned tensors take an exact
 * CUDA-core kernel that is about two orders of magnitude slower (the same
 * holds for mixattn_attend_chunk). */
int mixattn_prefill(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                    const int32_t* seq_lens, const void* q, const void* k, const void* v,
                    void* out, void* stream);

/* Attention of a chunk of new tokens behind what the caches already hold
 * (Section 3's definition with the queries at positions n .. n+S-1; Section 5
 * serves prompts of tens of thousands of tokens, which arrive in chunks, and a
 * chunk of a few tokens is a multi-token decode step).  For each sequence, with
 * n = tokens in the cache `layer` reads, query r of the chunk sits at position
 * n + r and attends to the cached keys and to the chunk's own keys up to its
 * position: all of them (standard layer) or the last `window` (sliding window).
 *   seq_lens host, chunk length S_b of each sequence (>= 1)
 *   q, out   device, [sum S_b, n_q_heads, head_dim], sequences back to back
 *   k, v     device, [sum S_b, n_kv_heads, head_dim]: the chunk's K/V as the
 *            layer's owner computed them (16-byte aligned)
 * The call STORES NOTHING: once every layer that reads a cache has run on the
 * chunk, the caller appends the chunk to that cache's owner with
 * mixattn_append_kv (a ring shared by several layers must still hold the
 * window of the chunk's first token when the last of them runs).
 * The cached keys the chunk needs (all of a paged cache, the last window-1
 * tokens of a ring) and the chunk's are first copied into plain tensors in the
 * context's chunk scratch, sequences in groups that fit it.  Exception: a ring
 * whose window is a multiple of 128 tokens (bf16, native storage)
 * is read in place, see mixattn_set_chunk_ring_direct; the size rules below
 * are the same either way.
 * Errors: UNSUPPORTED if the context was created with chunk_scratch_tokens = 0,
 * TOO_LARGE if one sequence's keys alone exceed the scratch, BAD_SEQ,
 * INVALID_ARG (null, duplicates, S_b < 1, n + S_b beyond max_seq_len), CUDA. */
int mixattn_attend_chunk(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                         const int32_t* seq_lens, const void* q, const void* k, const void* v,
                         void* out, void* stream);

/* One copy for all the layers that share a cache (Section 3: such layers read
 * the same cached keys, and a layer that reuses a cache is handed its owner's
 * K/V for the chunk, so consecutive mixattn_attend_chunk calls of these layers
 * would copy identical rows into the chunk scratch).  With reuse enabled, a
 * chunk call skips the copy when the previous chunk call on this context read
 * the same owner's cache for the same seq_ids and seq_lens with the same k and
 * v pointers on the same stream, fitted the scratch in one piece, and no call
 * since has changed a cache (append, prefill of an owner, seq_reset).  By
 * enabling it the caller promises that the contents behind k and v do not
 * change between such calls.  Off by default; enable = 0 switches it off again
 * and forgets what the scratch holds.  Results are identical either way.
 * Errors: INVALID_ARG for a null context. */
int mixattn_set_chunk_gather_reuse(mixattn_ctx* ctx, int32_t enable);

/* Chunk calls on sliding-window layers without the copy (Section 3: such a
 * layer keeps the last `window` tokens; the chunk's queries need at most the
 * last window-1 of them).  Token p of a ring lives in slot p mod window, so
 * when window is a multiple of the 128-key tile of the tensor-core kernel, a
 * tile of cached keys is eight whole pages of the sequence's ring, stored in
 * the layout the tensor cores read; the kernel then fetches those tiles from
 * the ring itself and the chunk's own K/V from the caller's tensors.  Applies
 * to bf16 contexts with native KV storage; every other chunk
 * call copies as described above.  On by default; enable = 0 makes every chunk
 * call copy.  Both ways attend to the same keys; the results differ by
 * rounding only (the keys are cut into tiles at different places).
 * Errors: INVALID_ARG for a null context. */
int mixattn_set_chunk_ring_direct(mixattn_ctx* ctx, int32_t enable);

/* Size of the static device array behind mixattn_decode_static_scratch. */
#define MIXATTN_STATIC_SCRATCH_BYTES (8u << 20)

/* The same decode step as mixattn_decode, for callers that hand the library an
 * arena holding the caches only.  (The paper has no counterpart: this is a
 * packaging variant of the decode call, not a different computation.)
 *
 * mixattn_decode keeps the partial results of its split pass in a workspace at
 * the end of the caller's arena.  Some integrations cannot provide that room,
 * nor any other device allocation, when they call: a plugin inside a serving
 * engine that has already handed out all device memory, a caller whose buffer
 * was sized for the caches alone (mixattn_cache_bytes) by a party it does not
 * control, or a runtime whose allocator must not be re-entered from inside the
 * attention call.  For them this entry point keeps those partial results in an
 * array that is part of the library image: MIXATTN_STATIC_SCRATCH_BYTES (8 MiB)
 * of device memory, held by every GPU context that loads the library until the
 * process exits.  The call itself never allocates or frees device memory,
 * neither directly nor through a library.
 *
 * Arguments, results and errors are those of mixattn_decode, plus:
 *   - n_seqs > 128, or more scratch needed than the array holds
 *     (splits * n_q_heads * (head_dim + 2) * 4 bytes, where a sequence of n
 *     attended keys makes about n / 4096 splits) -> MIXATTN_ERR_TOO_LARGE,
 *     nothing launched;
 *   - the first call on a device looks up the array's device address (a CUDA
 *     runtime query with that device current); make that first call outside
 *     any stream capture.  The address is kept for the life of the process;
 *     after a cudaDeviceReset of that device it is stale and this entry point
 *     must not be used any more;
 *   - all calls, from every context and stream of the process, share the one
 *     array per device.  Its contents are left over from the previous call;
 *     nothing in it needs to start at zero, since each call overwrites every
 *     slot before it reads it.  Two calls whose kernels overlap on the GPU
 *     (different streams) race on it: keep such calls on one stream, or order
 *     them with events. */
int mixattn_decode_static_scratch(mixattn_ctx* ctx, int32_t layer, int32_t n_seqs,
                                  const int32_t* seq_ids, const void* q, void* out, void* stream);

/* ---- introspection: the surface on which cache indexing is compared bit for bit ---- */

/* Tokens appended so far to the cache `layer` reads, for sequence `seq`. */
int mixattn_get_len(mixattn_ctx* ctx, int32_t layer, int32_t seq, int32_t* len);

/* Copies the sequence's block table (page id per logical block) to out[0..cap)
 * (host) and writes the number of blocks in use to *n_blocks (even if > cap). */
int mixattn_get_block_table(mixattn_ctx* ctx, int32_t seq, int32_t* out, int32_t cap,
                            int32_t* n_blocks);

/* Number of pages on the free FIFO. */
int mixattn_get_n_free_pages(mixattn_ctx* ctx, int32_t* n_free);

/* Ring of a sliding-window layer: slot the next token will take (len % window)
 * and number of valid slots (min(len, window)).  INVALID_ARG for a full layer. */
int mixattn_get_ring_state(mixattn_ctx* ctx, int32_t layer, int32_t seq, int32_t* next_slot,
                           int32_t* n_valid);

/* Where token `pos` of `seq` lives in the cache `layer` reads: page id and
 * offset within the page for a full layer; -1 and ring slot for a sliding
 * layer.  INVALID_ARG if the token is not stored (any more). */
int mixattn_locate(mixattn_ctx* ctx, int32_t layer, int32_t seq, int32_t pos, int32_t* page,
                   int32_t* slot);

/* Copies K and V of token `pos` ([n_kv_heads, head_dim] each, context dtype)
 * from the device cache to host buffers.  Waits for the whole device first.
 * The page is looked up in the DEVICE copy of the block table, so the call
 * also checks that copy.  For tests. */
int mixattn_debug_read_kv(mixattn_ctx* ctx, int32_t layer, int32_t seq, int32_t pos, void* k_host,
                          void* v_host);

/* Quantised storage only: the stored bytes of token `pos`: head_dim E4M3 codes per KV head
 * ([n_kv_heads, head_dim] bytes each for K and V) and the shared exponents X
 * ([n_kv_heads] int32 each).  UNSUPPORTED on a context with native storage;
 * all else as mixattn_debug_read_kv, which on a quantised cache returns the
 * dequantised bf16 values. */
int mixattn_debug_read_kv_fp8(mixattn_ctx* ctx, int32_t layer, int32_t seq, int32_t pos,
                              uint8_t* k_codes, int32_t* k_exp, uint8_t* v_codes, int32_t* v_exp);

/* Waits for the device, then reports the status word the kernels share:
 * 0 = fine, 1 = a bounded wait inside a kernel ran out (results invalid). */
int mixattn_get_device_status(mixattn_ctx* ctx, int32_t* status);

/* ---- tuning and measurement ---- */

/* Target number of keys per split of the split-KV decode; 0 = automatic.
 * Results do not depend on it beyond fp32 summation order. */
int mixattn_set_split_tokens(mixattn_ctx* ctx, int32_t tokens);

/* Kernel classes for mixattn_profile_read. */
enum {
  MIXATTN_K_APPEND = 0,
  MIXATTN_K_DECODE_FULL = 1,    /* split pass of a standard layer        */
  MIXATTN_K_DECODE_SLIDING = 2, /* split pass of a sliding-window layer  */
  MIXATTN_K_COMBINE = 3,
  MIXATTN_K_PREFILL_FULL = 4,
  MIXATTN_K_PREFILL_SLIDING = 5,
  MIXATTN_K_GATHER = 6,         /* copy of cached + chunk keys ahead of a chunk's attention */
  MIXATTN_K_COUNT = 7
};

/* enable != 0: from now on every kernel launch is bracketed by CUDA events on
 * its stream (costs a little; leave off when timing whole steps) and earlier
 * records are dropped.  enable == 0: stop recording. */
int mixattn_profile_enable(mixattn_ctx* ctx, int32_t enable);

/* Waits for the recorded events, then reports launches and summed device
 * milliseconds of one kernel class since the last enable. */
int mixattn_profile_read(mixattn_ctx* ctx, int32_t kernel_class, int32_t* launches, float* ms);

/* Kernel launches enqueued by this context since create. */
int mixattn_get_launch_count(mixattn_ctx* ctx, int64_t* launches);

/* Text for a status code; never NULL. */
const char* mixattn_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MIXATTN_H_ */

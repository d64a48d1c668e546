// Shared declarations of the library's translation units (host + device).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mixattn.h"

namespace mixattn {

constexpr int kPage = 16;          // tokens per page (paged pools and rings alike)
constexpr int kMaxCallSeqs = 128;  // sequences per kernel launch (metadata travels in kernel params)
constexpr int kMaxGroupRows = 8;   // query heads of one KV head handled by one work item
constexpr int kWsExtraChunks = 1024;                        // splits beyond one per sequence
constexpr int kWsWaveChunks = 256;                          // splits added to fill a single wave of SMs
constexpr int kWsChunks = kMaxCallSeqs + kWsExtraChunks + kWsWaveChunks;  // split slots in the workspace

// ---------------------------------------------------------------------------
// K/V storage format.
//
// Paged pools and rings use the same 16-token page.  A page holds, for every KV
// head g, one contiguous block  [K: 16 tokens x D][V: 16 tokens x D]  so that the
// decode kernel stages (page, g) with a single bulk copy.  In bf16 mode the 16-byte
// chunks of a token row are stored XOR-swizzled by (token & 7): the block in HBM is
// already the bank-conflict-free shared-memory image that ldmatrix wants, and the
// copy engine needs no tensor map.  fp32 rows are stored unswizzled.
// Quantised storage (FP8 E4M3 elements, one shared exponent byte per head vector):
//   [K: 16 tokens x D bytes][V^T: D channels x 16 tokens][X_K: 16 B][X_V: 16 B].
// K rows are swizzled by fp8_k_swizzle(token); V is stored TRANSPOSED (one 16-byte row per
// channel) because both tensor-core products of the decode kernel want their 8-bit operand
// with the contraction index contiguous: channels for K, tokens for V.
// ---------------------------------------------------------------------------
struct KvGeom {
  int32_t n_kv_heads;
  int32_t head_dim;
  int32_t elem_bytes;     // of Q / K / V / out as the caller passes them: 2 or 4
  int32_t row_bytes;      // head_dim * elem_bytes: one head vector in the caller's tensors
  int32_t st_row_bytes;   // one stored head vector: row_bytes, or head_dim for quantised storage
  int32_t fp8;            // 1: quantised storage
  int32_t blk_bytes;      // K and V (and exponents) of one (page, head)
  int32_t swizzle;        // 1 unless fp32
  int64_t page_bytes;     // n_kv_heads * blk_bytes
};

__host__ __device__ inline KvGeom make_geom(int n_kv_heads, int head_dim, int dtype, int kv_format) {
  KvGeom g;
  g.n_kv_heads = n_kv_heads;
  g.head_dim = head_dim;
  g.elem_bytes = dtype == MIXATTN_BF16 ? 2 : 4;
  g.row_bytes = head_dim * g.elem_bytes;
  g.fp8 = kv_format == MIXATTN_KV_FP8_E4M3 ? 1 : 0;
  g.st_row_bytes = g.fp8 ? head_dim : g.row_bytes;
  g.blk_bytes = 2 * kPage * g.st_row_bytes + (g.fp8 ? 2 * kPage : 0);
  g.swizzle = dtype == MIXATTN_BF16 ? 1 : 0;
  g.page_bytes = (int64_t)n_kv_heads * g.blk_bytes;
  return g;
}

// Chunk permutation of a quantised K row.  The decode kernel reads the 16 tokens of a page in the
// order 0 1 4 5 8 9 12 13 | 2 3 6 7 10 11 14 15 (see decode_bf16.cu): each half must hit eight
// different 16-byte columns.
__host__ __device__ inline int fp8_k_swizzle(int tok) { return (tok & 1) | ((tok >> 2) << 1); }

// Byte offset, inside a pool, of 16-byte chunk `chunk` of the stored row of token slot `tok`
// (0..15) of page `page`, KV head `g`, which = 0 (K) or 1 (V; native storage only).
__host__ __device__ inline int64_t kv_chunk_offset(const KvGeom& ge, int64_t page, int g, int which,
                                                   int tok, int chunk) {
  int c = !ge.swizzle ? chunk : ge.fp8 ? (chunk ^ fp8_k_swizzle(tok)) : (chunk ^ (tok & 7));
  return page * ge.page_bytes + (int64_t)g * ge.blk_bytes + (int64_t)which * kPage * ge.st_row_bytes +
         (int64_t)tok * ge.st_row_bytes + (int64_t)c * 16;
}

// Quantised storage: byte offset of V element (channel, tok) of that page and head.
__host__ __device__ inline int64_t kv_fp8_v_offset(const KvGeom& ge, int64_t page, int g, int channel, int tok) {
  return page * ge.page_bytes + (int64_t)g * ge.blk_bytes + (int64_t)kPage * ge.st_row_bytes +
         (int64_t)channel * kPage + tok;
}

// Quantised storage: byte offset of the shared-exponent byte of that row.
__host__ __device__ inline int64_t kv_exp_offset(const KvGeom& ge, int64_t page, int g, int which, int tok) {
  return page * ge.page_bytes + (int64_t)g * ge.blk_bytes + 2 * kPage * ge.st_row_bytes + which * kPage + tok;
}

// ---------------------------------------------------------------------------
// kernel parameter blocks (passed by value: no per-call metadata copy)
// ---------------------------------------------------------------------------
struct AppendEntry {
  int32_t seq;        // sequence slot
  int32_t start_pos;  // position of the first new token
  int32_t n_new;      // tokens appended
  int32_t src_row0;   // row of the first new token in k / v
  int32_t page_hint;  // n_new == 1 on a paged pool: page id resolved by the host; else -1
  int32_t tbl_idx;    // >= 0: device block-table entry this call must set to page_hint
};

struct AppendParams {
  const void* k;
  const void* v;
  char* pool;            // paged pool or ring storage of the owner
  int32_t* table;        // device block tables [max_seqs][table_stride]
  int32_t table_stride;
  int32_t is_ring;
  int32_t window;
  int32_t ring_pages;    // pages per sequence in a ring
  KvGeom geom;
  double rope_log2_theta;  // > 0: K rows are rotated (rotary embedding, base theta) at their positions
  int32_t n_entries;
  AppendEntry e[kMaxCallSeqs];
};

struct DecodeParams {
  const void* q;          // [n_seqs, Hq, D]
  void* out;              // [n_seqs, Hq, D]
  const char* pool;       // storage of the cache the layer reads
  const int32_t* table;   // device block tables, or nullptr for a ring
  int32_t table_stride;
  int32_t ring_pages;
  KvGeom geom;
  int32_t n_q_heads;
  int32_t group;          // query heads per KV head
  int32_t head_chunks;    // ceil(group / 8)
  float scale_log2e;      // softmax scale * log2(e)
  uint32_t l2_keep_bytes; // leading bytes of `pool` whose lines are cached normally (a ring that later
  uint32_t l2_pool_bytes; // layers re-read); the rest of the pool's l2_pool_bytes, and everything when
                          // l2_keep_bytes is 0, is marked evict-first (read once)
  float* part_o;          // [chunks, Hq, D] unnormalised partial outputs
  float2* part_ml;        // [chunks, Hq] running max (log2 units) and sum
  int32_t* status;        // device error word (0 = fine)
  int32_t n_seqs;
  int32_t total_items;    // chunks * Hkv * head_chunks
  int32_t seq_id[kMaxCallSeqs];
  int32_t n_eff[kMaxCallSeqs];           // keys attended: min(len, window) or len
  int32_t chunk_len[kMaxCallSeqs];       // keys per split of this sequence (multiple of 16)
  int32_t chunk_base[kMaxCallSeqs + 1];  // first split index of each sequence
};

struct PrefillParams {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t window;        // 0 = standard layer
  float scale_log2e;
  int32_t n_seqs;
  int32_t* status;
  int32_t row0[kMaxCallSeqs + 1];   // first row of each sequence in q / out (packed)
  int32_t krow0[kMaxCallSeqs];      // first row of each sequence in k / v
  int32_t prefix[kMaxCallSeqs];     // keys of the sequence that precede its first query
  // The first cached[b] of those keys are not in k / v but in a ring cache, read in place by the
  // tensor-core kernel (k / v then hold prefix[b] - cached[b] + (row0[b + 1] - row0[b]) rows for
  // sequence b); 0 everywhere = every key comes from k / v.  Keys are then numbered by their
  // position in the sequence, so that key tiles fall on whole ring pages.
  int32_t cached[kMaxCallSeqs];
  int32_t ring_page0[kMaxCallSeqs]; // first page of the sequence's ring in ring_pool
  const void* ring_pool = nullptr;  // storage of the ring (nullptr = no sequence has cached keys)
  int32_t ring_pages;               // pages per sequence in the ring (a multiple of 8)
  int64_t ring_total_pages;         // pages in ring_pool
  KvGeom geom;
};

// Copies the cached keys a chunk of queries needs, followed by the chunk's own keys, into
// plain [rows, Hkv, D] tensors (the layout the prompt kernels read).
struct GatherEntry {
  int32_t seq;        // sequence slot
  int32_t pos0;       // position of the first cached token copied
  int32_t n_prefix;   // cached tokens copied (positions pos0 .. pos0 + n_prefix - 1)
  int32_t n_chunk;    // tokens taken from the chunk tensors after them
  int32_t src_row0;   // first row of the chunk in k_chunk / v_chunk
  int32_t dst_row0;   // first row written in k_out / v_out
};

struct GatherParams {
  const void* k_chunk;
  const void* v_chunk;
  void* k_out;
  void* v_out;
  const char* pool;
  const int32_t* table;
  int32_t table_stride;
  int32_t is_ring;
  int32_t window;
  int32_t ring_pages;
  KvGeom geom;
  int32_t n_entries;
  GatherEntry e[kMaxCallSeqs];
};

// Block-table entries a bulk append sets on the device before its copy kernel reads them.
constexpr int kTableSetMax = 1024;
struct TableSetParams {
  int32_t* table;
  int32_t n;
  int32_t idx[kTableSetMax];    // entry index: seq * table_stride + logical block
  int32_t page[kTableSetMax];
};

// device status codes written to the status word
enum { kDevOk = 0, kDevWaitTimeout = 1 };

// launchers (each returns the cudaError_t of its launch)
cudaError_t launch_append(const AppendParams& p, int max_n_new, cudaStream_t st);
cudaError_t launch_table_set(const TableSetParams& p, cudaStream_t st);
cudaError_t launch_gather(const GatherParams& p, int max_rows, cudaStream_t st);
cudaError_t prepare_decode_bf16();
cudaError_t launch_decode_split_bf16(const DecodeParams& p, int sm_count, cudaStream_t st);   // native or quantised cache
cudaError_t launch_decode_split_f32(const DecodeParams& p, cudaStream_t st);
cudaError_t launch_decode_combine(const DecodeParams& p, int dtype, cudaStream_t st);
cudaError_t launch_prefill_simple(const PrefillParams& p, int dtype, int max_len, cudaStream_t st);
bool prefill_tc_supported(int dtype, int head_dim, const void* q, const void* k, const void* v);
bool prefill_tc_ring_direct_supported(const KvGeom& ge, int window);   // cached keys read in place from a ring
cudaError_t prepare_prefill_tc();
cudaError_t launch_prefill_tc(const PrefillParams& p, int max_len, int sm_count, cudaStream_t st);

}  // namespace mixattn

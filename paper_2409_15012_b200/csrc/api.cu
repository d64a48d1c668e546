// The C ABI (include/mixattn.h): argument validation, host bookkeeping, arena carving and
// kernel launches.  Everything that can fail is checked on the host before any launch.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <new>
#include <vector>

#include "cache_manager.hpp"
#include "internal.h"

using namespace mixattn;

namespace {

constexpr size_t kAlign = 256;
constexpr int kSplitTokens = 4096;    // automatic split length of long caches (keys)
constexpr int kMinSplitTokens = 1024; // single-wave splitting never makes splits shorter than this
constexpr double kL2FitsShare = 0.55;  // a re-read ring up to this share of the L2 is cached whole
constexpr double kL2KeepShare = 0.45;  // of a larger one, this share of the L2 is kept

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct ArenaPlan {
  std::vector<size_t> owner_off;  // per owner slot
  std::vector<size_t> owner_bytes;
  size_t table_off = 0, table_bytes = 0;
  size_t part_o_off = 0, part_ml_off = 0, status_off = 0;
  size_t chunk_k_off = 0, chunk_v_off = 0;   // [chunk_scratch_tokens, Hkv, D] each
  size_t cache_bytes = 0, total = 0;
};

int ring_pages_of(int window) { return (window + kPage - 1) / kPage; }

ArenaPlan plan_arena(const CacheManager& cm, const mixattn_config& cfg) {
  ArenaPlan pl;
  KvGeom ge = make_geom(cfg.n_kv_heads, cfg.head_dim, cfg.dtype, cfg.kv_format);
  size_t off = 0;
  for (int o : cm.owners()) {
    const LayerInfo& li = cm.layer(o);
    size_t bytes = li.kind == MIXATTN_FULL
                       ? (size_t)cfg.n_pages * ge.page_bytes
                       : (size_t)cfg.max_seqs * ring_pages_of(li.window) * ge.page_bytes;
    pl.owner_off.push_back(off);
    pl.owner_bytes.push_back(bytes);
    pl.cache_bytes += bytes;
    off += align_up(bytes);
  }
  pl.table_off = off;
  pl.table_bytes = (size_t)cm.max_seqs() * cm.max_blocks() * sizeof(int32_t);
  off += align_up(pl.table_bytes);
  pl.part_o_off = off;
  off += align_up((size_t)kWsChunks * cfg.n_q_heads * cfg.head_dim * sizeof(float));
  pl.part_ml_off = off;
  off += align_up((size_t)kWsChunks * cfg.n_q_heads * sizeof(float2));
  pl.status_off = off;
  off += kAlign;
  if (cfg.chunk_scratch_tokens > 0) {
    const size_t bytes = align_up((size_t)cfg.chunk_scratch_tokens * ge.n_kv_heads * ge.row_bytes);
    pl.chunk_k_off = off;
    off += bytes;
    pl.chunk_v_off = off;
    off += bytes;
  }
  pl.total = off;
  return pl;
}

struct ProfileRecord {
  int cls;
  cudaEvent_t start, stop;
};

}  // namespace

struct mixattn_ctx {
  CacheManager cm;
  mixattn_config cfg;  // layers / free_order pointers are not kept
  KvGeom geom;
  ArenaPlan plan;
  char* arena = nullptr;
  bool host_only = true;
  int device = -1;
  int sm_count = 148;
  int64_t l2_bytes = 0;
  float scale = 0.f;
  int32_t split_tokens = 0;
  int64_t launches = 0;
  bool profiling = false;
  std::vector<ProfileRecord> records;
  std::vector<cudaEvent_t> event_pool;
  bool sticky_cuda_error = false;
  // Chunk calls of layers that share a cache gather the same rows: what the scratch holds is
  // remembered so that, when the caller has enabled it, the copy runs once per run of such calls.
  bool chunk_reuse = false;
  // Chunk calls of sliding-window layers whose window is a whole number of key tiles read the
  // cached keys in place from the ring (no copy); off = every chunk call copies.
  bool chunk_ring_direct = true;
  uint64_t cache_epoch = 0;   // bumped by every call that changes a cache
  struct GatherKey {
    bool valid = false;
    int owner = -1;
    uint64_t epoch = 0;
    const void* k = nullptr;
    const void* v = nullptr;
    cudaStream_t st = nullptr;
    std::vector<int32_t> ids, lens;
  } scratch_holds;

  char* owner_storage(int layer) const { return arena + plan.owner_off[cm.layer(layer).owner_slot]; }
  int32_t* dev_table() const { return reinterpret_cast<int32_t*>(arena + plan.table_off); }
  int32_t* dev_status() const { return reinterpret_cast<int32_t*>(arena + plan.status_off); }
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    target = dev;
  }
  ~DeviceGuard() {
    if (ok && prev >= 0 && prev != target) cudaSetDevice(prev);
  }
  int target = -1;
};

cudaEvent_t take_event(mixattn_ctx* c) {
  if (!c->event_pool.empty()) {
    cudaEvent_t e = c->event_pool.back();
    c->event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// Brackets one launch with events when profiling is on.
template <typename F>
cudaError_t launch_recorded(mixattn_ctx* c, int cls, cudaStream_t st, F&& f) {
  ProfileRecord rec{cls, nullptr, nullptr};
  if (c->profiling) {
    rec.start = take_event(c);
    rec.stop = take_event(c);
    if (rec.start) cudaEventRecord(rec.start, st);
  }
  cudaError_t e = f();
  if (c->profiling) {
    if (rec.stop) cudaEventRecord(rec.stop, st);
    c->records.push_back(rec);
  }
  if (e == cudaSuccess) ++c->launches;
  else c->sticky_cuda_error = true;
  return e;
}

int validate_config(const mixattn_config* cfg, CacheManager* cm, bool allocate = true) {
  if (cfg == nullptr) return MIXATTN_ERR_INVALID_ARG;
  int rc = cm->init(*cfg, allocate);
  if (rc != MIXATTN_OK) return rc;
  if (cfg->softmax_scale < 0.f || !isfinite(cfg->softmax_scale)) return MIXATTN_ERR_INVALID_ARG;
  if (cm->n_full_owners() > 0 && cfg->n_pages < 1) return MIXATTN_ERR_INVALID_ARG;
  if (cfg->chunk_scratch_tokens < 0) return MIXATTN_ERR_INVALID_ARG;
  if (cfg->kv_format != MIXATTN_KV_NATIVE && cfg->kv_format != MIXATTN_KV_FP8_E4M3) return MIXATTN_ERR_INVALID_ARG;
  if (cfg->kv_format == MIXATTN_KV_FP8_E4M3 && (cfg->dtype != MIXATTN_BF16 || cfg->head_dim != 128))
    return MIXATTN_ERR_UNSUPPORTED;
  return MIXATTN_OK;
}

// Enqueues the device side of an append the host bookkeeping has already applied.
int enqueue_append(mixattn_ctx* c, int layer, int n_seqs, const int32_t* seq_ids,
                   const int32_t* n_new, const std::vector<int32_t>& start_pos,
                   const std::vector<PageGrant>& grants, const void* k, const void* v,
                   cudaStream_t st, double rope_log2_theta = 0.0) {
  const LayerInfo& li = c->cm.layer(layer);
  const bool ring = li.kind == MIXATTN_SLIDING;
  bool single = true;
  for (int i = 0; i < n_seqs; ++i) single = single && (n_new == nullptr || n_new[i] == 1);
  const int stride = c->cm.max_blocks();
  if (!ring && !single && !grants.empty()) {
    // bulk append: the new table entries travel in kernel parameters (no host copy that would
    // wait for the stream or depend on pageable memory) and are set by a small kernel ahead of
    // the copy kernel, which reads the table
    TableSetParams tp;
    tp.table = c->dev_table();
    for (size_t a = 0; a < grants.size(); a += kTableSetMax) {
      const size_t n = grants.size() - a < (size_t)kTableSetMax ? grants.size() - a : (size_t)kTableSetMax;
      for (size_t i = 0; i < n; ++i) {
        tp.idx[i] = grants[a + i].seq * stride + grants[a + i].block;
        tp.page[i] = grants[a + i].page;
      }
      tp.n = (int32_t)n;
      cudaError_t e = launch_recorded(c, MIXATTN_K_APPEND, st, [&] { return launch_table_set(tp, st); });
      if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
    }
  }
  AppendParams p;
  p.k = k;
  p.v = v;
  p.pool = c->owner_storage(layer);
  p.table = c->dev_table();
  p.table_stride = stride;
  p.is_ring = ring;
  p.window = ring ? li.window : 0;
  p.ring_pages = ring ? ring_pages_of(li.window) : 0;
  p.geom = c->geom;
  p.rope_log2_theta = rope_log2_theta;
  int row = 0;
  size_t gi = 0;
  for (int i0 = 0; i0 < n_seqs; i0 += kMaxCallSeqs) {
    const int nb = n_seqs - i0 < kMaxCallSeqs ? n_seqs - i0 : kMaxCallSeqs;
    int max_new = 0;
    for (int j = 0; j < nb; ++j) {
      const int i = i0 + j;
      AppendEntry& e = p.e[j];
      e.seq = seq_ids[i];
      e.start_pos = start_pos[i];
      e.n_new = n_new ? n_new[i] : 1;
      e.src_row0 = row;
      e.page_hint = -1;
      e.tbl_idx = -1;
      if (!ring && single) {
        e.page_hint = c->cm.table_row(e.seq)[e.start_pos / kPage];
        // grants are in call order: at most one per sequence in single-token mode
        if (gi < grants.size() && grants[gi].seq == e.seq) {
          e.tbl_idx = e.seq * stride + grants[gi].block;
          ++gi;
        }
      }
      row += e.n_new;
      if (e.n_new > max_new) max_new = e.n_new;
    }
    p.n_entries = nb;
    if (max_new == 0) {
      bool any_tbl = false;
      for (int j = 0; j < nb; ++j) any_tbl = any_tbl || p.e[j].tbl_idx >= 0;
      if (!any_tbl) continue;
    }
    cudaError_t e = launch_recorded(c, MIXATTN_K_APPEND, st, [&] { return launch_append(p, max_new, st); });
    if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
  }
  return MIXATTN_OK;
}

}  // namespace

extern "C" {

int mixattn_arena_bytes(const mixattn_config* cfg, size_t* out_bytes) {
  if (out_bytes == nullptr) return MIXATTN_ERR_INVALID_ARG;
  CacheManager cm;
  int rc = validate_config(cfg, &cm, false);
  if (rc != MIXATTN_OK) return rc;
  *out_bytes = plan_arena(cm, *cfg).total;
  return MIXATTN_OK;
}

int mixattn_cache_bytes(const mixattn_config* cfg, size_t* out_bytes) {
  if (out_bytes == nullptr) return MIXATTN_ERR_INVALID_ARG;
  CacheManager cm;
  int rc = validate_config(cfg, &cm, false);
  if (rc != MIXATTN_OK) return rc;
  *out_bytes = plan_arena(cm, *cfg).cache_bytes;
  return MIXATTN_OK;
}

int mixattn_create(const mixattn_config* cfg, mixattn_ctx** out) {
  if (out == nullptr) return MIXATTN_ERR_INVALID_ARG;
  *out = nullptr;
  mixattn_ctx* c = new (std::nothrow) mixattn_ctx();
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  int rc = validate_config(cfg, &c->cm);
  if (rc != MIXATTN_OK) { delete c; return rc; }
  c->cfg = *cfg;
  c->cfg.layers = nullptr;
  c->cfg.free_order = nullptr;
  c->geom = make_geom(cfg->n_kv_heads, cfg->head_dim, cfg->dtype, cfg->kv_format);
  c->plan = plan_arena(c->cm, *cfg);
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
  c->host_only = cfg->device < 0;
  c->device = cfg->device;
  if (!c->host_only) {
    if (cfg->arena == nullptr || cfg->arena_bytes < c->plan.total ||
        (reinterpret_cast<uintptr_t>(cfg->arena) % kAlign) != 0) {
      delete c;
      return MIXATTN_ERR_INVALID_ARG;
    }
    c->arena = static_cast<char*>(cfg->arena);
    DeviceGuard g(c->device);
    cudaDeviceProp prop;
    if (!g.ok || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) { delete c; return MIXATTN_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    c->l2_bytes = prop.l2CacheSize;
    if (prepare_decode_bf16() != cudaSuccess || prepare_prefill_tc() != cudaSuccess) { delete c; return MIXATTN_ERR_CUDA; }
    if (cudaMemsetAsync(c->arena, 0, c->plan.total, 0) != cudaSuccess ||
        cudaStreamSynchronize(0) != cudaSuccess) {
      delete c;
      return MIXATTN_ERR_CUDA;
    }
  }
  *out = c;
  return MIXATTN_OK;
}

int mixattn_destroy(mixattn_ctx* c) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  if (!c->host_only) {
    DeviceGuard g(c->device);
    for (auto& r : c->records) {
      if (r.start) cudaEventDestroy(r.start);
      if (r.stop) cudaEventDestroy(r.stop);
    }
    for (auto e : c->event_pool) cudaEventDestroy(e);
  }
  delete c;
  return MIXATTN_OK;
}

int mixattn_seq_reset(mixattn_ctx* c, int32_t seq) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  c->cm.seq_reset(seq);
  ++c->cache_epoch;
  return MIXATTN_OK;
}

static int append_impl(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                       const int32_t* n_new, const void* k, const void* v, void* stream, double rope_log2_theta) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  int rc = c->cm.check_append(layer, n_seqs, seq_ids, n_new);
  if (rc != MIXATTN_OK) return rc;
  int64_t total = 0;
  for (int i = 0; i < n_seqs; ++i) total += n_new ? n_new[i] : 1;
  if (total > INT32_MAX) return MIXATTN_ERR_INVALID_ARG;
  if (!c->host_only) {
    if (total > 0 && (k == nullptr || v == nullptr)) return MIXATTN_ERR_INVALID_ARG;
    if (c->sticky_cuda_error) return MIXATTN_ERR_CUDA;
  }
  std::vector<int32_t> start(n_seqs);
  for (int i = 0; i < n_seqs; ++i) start[i] = c->cm.len(layer, seq_ids[i]);
  std::vector<PageGrant> grants;
  c->cm.apply_append(layer, n_seqs, seq_ids, n_new, &grants);
  ++c->cache_epoch;
  if (c->host_only) return MIXATTN_OK;
  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  return enqueue_append(c, layer, n_seqs, seq_ids, n_new, start, grants, k, v,
                        static_cast<cudaStream_t>(stream), rope_log2_theta);
}

int mixattn_append_kv(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                      const int32_t* n_new, const void* k, const void* v, void* stream) {
  return append_impl(c, layer, n_seqs, seq_ids, n_new, k, v, stream, 0.0);
}

int mixattn_append_kv_rope(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                           const int32_t* n_new, const void* k, const void* v, float rope_theta,
                           void* stream) {
  if (!(rope_theta > 1.f) || !isfinite(rope_theta)) return MIXATTN_ERR_INVALID_ARG;
  return append_impl(c, layer, n_seqs, seq_ids, n_new, k, v, stream, log2((double)rope_theta));
}

// L2 policy of a decode launch (see l2_policy_of in decode_bf16.cu).  Only a ring that a later
// layer reads again (Section 3's cache sharing makes consecutive layers read the same bytes) is
// worth keeping: the leading part of its storage, up to a share of the L2 that a cyclic scan was
// measured to keep resident.  The last layer that reads the ring lets go of it.
static void set_l2_policy(const mixattn_ctx* c, int layer, DecodeParams* p) {
  p->l2_keep_bytes = 0;
  p->l2_pool_bytes = 0;
  const LayerInfo& li = c->cm.layer(layer);
  if (li.kind != MIXATTN_SLIDING || c->l2_bytes <= 0) return;
  bool read_again = false;
  for (int l = layer + 1; l < c->cfg.n_layers; ++l) read_again = read_again || c->cm.layer(l).owner == li.owner;
  if (!read_again) return;
  const uint64_t pool = c->plan.owner_bytes[li.owner_slot];
  // (measured on a 126 MB L2: a 67 MB ring stays resident under plain LRU, a 134 MB ring does not
  // at all; keeping 0.4-0.5 of the L2 of it gave the shortest step)
  const uint64_t fits = (uint64_t)(kL2FitsShare * (double)c->l2_bytes);
  const uint64_t room = (uint64_t)(kL2KeepShare * (double)c->l2_bytes);
  const uint64_t window = pool < 0xFFFFFF00ull ? pool : 0xFFFFFF00ull;   // the policy's sizes are 32-bit
  p->l2_pool_bytes = (uint32_t)window;
  p->l2_keep_bytes = (uint32_t)(window <= fits ? window : room);
}

// Split plan of one decode launch over sequences ids[0 .. nb): fills the per-sequence fields of
// *p (seq_id, n_eff, chunk_len, chunk_base, n_seqs, total_items; group and head_chunks must be
// set) and returns the number of split slots the launch writes; *any_split tells whether a
// combine pass is needed.  Long caches are cut into splits of kSplitTokens keys (large splits
// keep the per-item epilogue negligible; thousands of items balance over the SMs).  When there
// are fewer (sequence, KV head) pairs than SMs, short caches are cut further, but only up to one
// item per SM, so the launch stays a single wave.  Both decode entry points use this one
// function, so they add the partial results in the same order.
static int plan_splits(const mixattn_ctx* c, int layer, const int32_t* ids, int nb, DecodeParams* p,
                       bool* any_split) {
  const int Hkv = c->cfg.n_kv_heads;
  int64_t total = 0;
  for (int j = 0; j < nb; ++j) {
    p->seq_id[j] = ids[j];
    p->n_eff[j] = c->cm.n_attended(layer, ids[j]);
    total += p->n_eff[j];
  }
  int64_t T = c->split_tokens > 0 ? (c->split_tokens + kPage - 1) / kPage * kPage : kSplitTokens;
  int64_t t_min = (total + kWsExtraChunks - 1) / kWsExtraChunks;
  t_min = (t_min + kPage - 1) / kPage * kPage;
  if (T < t_min) T = t_min;
  const int64_t pairs = (int64_t)nb * Hkv * p->head_chunks;
  int64_t nc_wave = c->split_tokens > 0 ? 1 : c->sm_count / pairs;
  if (nc_wave > kWsWaveChunks / nb) nc_wave = kWsWaveChunks / nb;   // the workspace bounds the extra splits
  int base = 0;
  *any_split = false;
  for (int j = 0; j < nb; ++j) {
    const int64_t n = p->n_eff[j];
    int64_t nc = (n + T - 1) / T;
    if (nc < nc_wave) {
      int64_t by_len = n / kMinSplitTokens;
      nc = by_len < nc_wave ? by_len : nc_wave;
      if (nc < 1) nc = 1;
    }
    int64_t len = (n + nc - 1) / nc;
    len = (len + kPage - 1) / kPage * kPage;
    nc = (n + len - 1) / len;
    p->chunk_base[j] = base;
    p->chunk_len[j] = (int32_t)len;
    base += (int)nc;
    *any_split = *any_split || nc > 1;
  }
  p->chunk_base[nb] = base;
  p->n_seqs = nb;
  p->total_items = base * Hkv * p->head_chunks;
  return base;
}

int mixattn_decode(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                   const void* q, void* out, void* stream) {
  if (c == nullptr || !c->cm.valid_layer(layer) || n_seqs < 0) return MIXATTN_ERR_INVALID_ARG;
  if (n_seqs > 0 && (seq_ids == nullptr || q == nullptr || out == nullptr)) return MIXATTN_ERR_INVALID_ARG;
  for (int i = 0; i < n_seqs; ++i) {
    if (!c->cm.valid_seq(seq_ids[i])) return MIXATTN_ERR_BAD_SEQ;
  }
  for (int i = 0; i < n_seqs; ++i) {
    if (c->cm.len(layer, seq_ids[i]) < 1) return MIXATTN_ERR_EMPTY_CONTEXT;
  }
  if (c->host_only || c->sticky_cuda_error) return MIXATTN_ERR_CUDA;
  if (n_seqs == 0) return MIXATTN_OK;
  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const LayerInfo& li = c->cm.layer(layer);
  const bool ring = li.kind == MIXATTN_SLIDING;
  const int Hq = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
  const size_t esz = c->geom.elem_bytes;

  DecodeParams p;
  p.pool = c->owner_storage(layer);
  p.table = ring ? nullptr : c->dev_table();
  p.table_stride = c->cm.max_blocks();
  p.ring_pages = ring ? ring_pages_of(li.window) : 0;
  p.geom = c->geom;
  p.n_q_heads = Hq;
  p.group = Hq / Hkv;
  p.head_chunks = (p.group + kMaxGroupRows - 1) / kMaxGroupRows;
  p.scale_log2e = c->scale * 1.4426950408889634f;
  p.part_o = reinterpret_cast<float*>(c->arena + c->plan.part_o_off);
  p.part_ml = reinterpret_cast<float2*>(c->arena + c->plan.part_ml_off);
  p.status = c->dev_status();
  set_l2_policy(c, layer, &p);

  for (int i0 = 0; i0 < n_seqs; i0 += kMaxCallSeqs) {
    const int nb = n_seqs - i0 < kMaxCallSeqs ? n_seqs - i0 : kMaxCallSeqs;
    bool any_split = false;
    const int base = plan_splits(c, layer, seq_ids + i0, nb, &p, &any_split);
    if (base > kWsChunks) return MIXATTN_ERR_UNSUPPORTED;   // (cannot happen: the plan is bounded by the workspace)
    p.q = static_cast<const char*>(q) + (size_t)i0 * Hq * D * esz;
    p.out = static_cast<char*>(out) + (size_t)i0 * Hq * D * esz;
    const int cls = ring ? MIXATTN_K_DECODE_SLIDING : MIXATTN_K_DECODE_FULL;
    cudaError_t e = launch_recorded(c, cls, st, [&] {
      return c->cfg.dtype == MIXATTN_BF16 ? launch_decode_split_bf16(p, c->sm_count, st)
                                          : launch_decode_split_f32(p, st);
    });
    if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
    if (any_split) {
      e = launch_recorded(c, MIXATTN_K_COMBINE, st,
                          [&] { return launch_decode_combine(p, c->cfg.dtype, st); });
      if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
    }
  }
  return MIXATTN_OK;
}

int mixattn_decode_layers(mixattn_ctx* c, int32_t layer_begin, int32_t layer_end, int32_t n_seqs,
                          const int32_t* seq_ids, const void* const* q, const void* const* k,
                          const void* const* v, void* const* out, void* stream, int32_t* layers_done) {
  if (layers_done != nullptr) *layers_done = 0;
  if (c == nullptr || layer_begin < 0 || layer_end < layer_begin || layer_end > c->cm.n_layers())
    return MIXATTN_ERR_INVALID_ARG;
  if (layer_end > layer_begin && (q == nullptr || out == nullptr || k == nullptr || v == nullptr))
    return MIXATTN_ERR_INVALID_ARG;
  for (int l = layer_begin; l < layer_end; ++l) {
    if (c->cm.layer(l).owner == l) {
      int rc = append_impl(c, l, n_seqs, seq_ids, nullptr, k[l], v[l], stream, 0.0);
      if (rc != MIXATTN_OK) return rc;
    }
    int rc = mixattn_decode(c, l, n_seqs, seq_ids, q[l], out[l], stream);
    if (rc != MIXATTN_OK) return rc;
    if (layers_done != nullptr) *layers_done = l - layer_begin + 1;
  }
  return MIXATTN_OK;
}

int mixattn_prefill(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                    const int32_t* seq_lens, const void* q, const void* k, const void* v,
                    void* out, void* stream) {
  if (c == nullptr || !c->cm.valid_layer(layer) || n_seqs < 0) return MIXATTN_ERR_INVALID_ARG;
  if (n_seqs > 0 && (seq_ids == nullptr || seq_lens == nullptr)) return MIXATTN_ERR_INVALID_ARG;
  const LayerInfo& li = c->cm.layer(layer);
  const bool owner = li.owner == layer;
  int64_t total = 0;
  int max_len = 0;
  {
    std::vector<char> seen(c->cm.max_seqs(), 0);
    for (int i = 0; i < n_seqs; ++i) {
      if (!c->cm.valid_seq(seq_ids[i])) return MIXATTN_ERR_BAD_SEQ;
      if (seen[seq_ids[i]]) return MIXATTN_ERR_INVALID_ARG;
      seen[seq_ids[i]] = 1;
      if (seq_lens[i] < 1) return MIXATTN_ERR_INVALID_ARG;
      total += seq_lens[i];
      if (seq_lens[i] > max_len) max_len = seq_lens[i];
    }
  }
  if (total > INT32_MAX) return MIXATTN_ERR_INVALID_ARG;
  if (owner) {
    for (int i = 0; i < n_seqs; ++i)
      if (c->cm.len(layer, seq_ids[i]) != 0) return MIXATTN_ERR_UNSUPPORTED;
    int rc = c->cm.check_append(layer, n_seqs, seq_ids, seq_lens);
    if (rc != MIXATTN_OK) return rc;
  }
  if (c->host_only || c->sticky_cuda_error) return MIXATTN_ERR_CUDA;
  if (n_seqs == 0) return MIXATTN_OK;
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return MIXATTN_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int Hq = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
  const size_t esz = c->geom.elem_bytes;
  PrefillParams p;
  p.n_q_heads = Hq;
  p.n_kv_heads = Hkv;
  p.head_dim = D;
  p.window = li.kind == MIXATTN_SLIDING ? li.window : 0;
  p.scale_log2e = c->scale * 1.4426950408889634f;
  p.status = c->dev_status();
  int64_t row = 0;
  for (int i0 = 0; i0 < n_seqs; i0 += kMaxCallSeqs) {
    const int nb = n_seqs - i0 < kMaxCallSeqs ? n_seqs - i0 : kMaxCallSeqs;
    int r = 0, mlen = 0;
    for (int j = 0; j < nb; ++j) {
      p.row0[j] = r;
      p.krow0[j] = r;
      p.prefix[j] = 0;
      r += seq_lens[i0 + j];
      if (seq_lens[i0 + j] > mlen) mlen = seq_lens[i0 + j];
    }
    p.row0[nb] = r;
    p.n_seqs = nb;
    p.q = static_cast<const char*>(q) + (size_t)row * Hq * D * esz;
    p.out = static_cast<char*>(out) + (size_t)row * Hq * D * esz;
    p.k = static_cast<const char*>(k) + (size_t)row * Hkv * D * esz;
    p.v = static_cast<const char*>(v) + (size_t)row * Hkv * D * esz;
    row += r;
    const int cls = p.window ? MIXATTN_K_PREFILL_SLIDING : MIXATTN_K_PREFILL_FULL;
    // bf16 runs on the tensor-core kernel, fp32 mode on the exact CUDA-core kernel
    const bool tc = prefill_tc_supported(c->cfg.dtype, D, p.q, p.k, p.v) && (((size_t)p.out) & 15) == 0;
    cudaError_t e = launch_recorded(c, cls, st, [&] {
      return tc ? launch_prefill_tc(p, mlen, c->sm_count, st) : launch_prefill_simple(p, c->cfg.dtype, mlen, st);
    });
    if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
  }
  // The attention reads the caller's tensors, not the cache, so the cache is written after it:
  // the bookkeeping moves only once every attention launch (tensor maps included) has been
  // accepted.  A CUDA failure past this point leaves the context unusable (see the header).
  if (owner) {
    std::vector<int32_t> start(n_seqs, 0);
    std::vector<PageGrant> grants;
    c->cm.apply_append(layer, n_seqs, seq_ids, seq_lens, &grants);
    ++c->cache_epoch;
    int rc = enqueue_append(c, layer, n_seqs, seq_ids, seq_lens, start, grants, k, v, st);
    if (rc != MIXATTN_OK) return rc;
  }
  return MIXATTN_OK;
}

int mixattn_attend_chunk(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                         const int32_t* seq_lens, const void* q, const void* k, const void* v,
                         void* out, void* stream) {
  if (c == nullptr || !c->cm.valid_layer(layer) || n_seqs < 0) return MIXATTN_ERR_INVALID_ARG;
  if (n_seqs > 0 && (seq_ids == nullptr || seq_lens == nullptr)) return MIXATTN_ERR_INVALID_ARG;
  const LayerInfo& li = c->cm.layer(layer);
  const bool ring = li.kind == MIXATTN_SLIDING;
  const int scratch = c->cfg.chunk_scratch_tokens;
  // cached keys each sequence's chunk needs: all of a paged cache, the last window - 1 of a ring
  std::vector<int32_t> n_prefix(n_seqs > 0 ? n_seqs : 0);
  {
    std::vector<char> seen(c->cm.max_seqs(), 0);
    int64_t total = 0;
    for (int i = 0; i < n_seqs; ++i) {
      if (!c->cm.valid_seq(seq_ids[i])) return MIXATTN_ERR_BAD_SEQ;
      if (seen[seq_ids[i]]) return MIXATTN_ERR_INVALID_ARG;
      seen[seq_ids[i]] = 1;
      if (seq_lens[i] < 1) return MIXATTN_ERR_INVALID_ARG;
      const int64_t n = c->cm.len(layer, seq_ids[i]);
      if (n + seq_lens[i] > c->cm.max_seq_len()) return MIXATTN_ERR_INVALID_ARG;
      total += seq_lens[i];
      n_prefix[i] = (int32_t)(ring ? (n < li.window - 1 ? n : li.window - 1) : n);
    }
    if (total > INT32_MAX) return MIXATTN_ERR_INVALID_ARG;
  }
  if (scratch <= 0) return MIXATTN_ERR_UNSUPPORTED;
  for (int i = 0; i < n_seqs; ++i)
    if ((int64_t)n_prefix[i] + seq_lens[i] > scratch) return MIXATTN_ERR_TOO_LARGE;
  if (c->host_only || c->sticky_cuda_error) return MIXATTN_ERR_CUDA;
  if (n_seqs == 0) return MIXATTN_OK;
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return MIXATTN_ERR_INVALID_ARG;
  if ((((size_t)k) | ((size_t)v)) & 15) return MIXATTN_ERR_INVALID_ARG;
  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int Hq = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
  const size_t esz = c->geom.elem_bytes;
  char* ks = c->arena + c->plan.chunk_k_off;
  char* vs = c->arena + c->plan.chunk_v_off;

  GatherParams gp;
  gp.k_out = ks;
  gp.v_out = vs;
  gp.pool = c->owner_storage(layer);
  gp.table = c->dev_table();
  gp.table_stride = c->cm.max_blocks();
  gp.is_ring = ring;
  gp.window = ring ? li.window : 0;
  gp.ring_pages = ring ? ring_pages_of(li.window) : 0;
  gp.geom = c->geom;
  PrefillParams p;
  p.n_q_heads = Hq;
  p.n_kv_heads = Hkv;
  p.head_dim = D;
  p.window = ring ? li.window : 0;
  p.scale_log2e = c->scale * 1.4426950408889634f;
  p.status = c->dev_status();
  p.k = ks;
  p.v = vs;

  // The rows this call would copy are already in the scratch when the previous chunk call read
  // the same cache for the same sequences with the same chunk K/V, in one piece, on this stream,
  // and no cache has changed since (a reader layer right after its owner, or after another reader).
  bool one_piece = n_seqs <= kMaxCallSeqs;
  {
    int64_t rows = 0;
    for (int i = 0; i < n_seqs; ++i) rows += (int64_t)n_prefix[i] + seq_lens[i];
    one_piece = one_piece && rows <= scratch;
  }
  // A ring whose window is a whole number of key tiles is read where it is: a key tile of the
  // cached positions is eight consecutive pages of the sequence's ring, in the layout the tensor
  // cores take.  K / V of the chunk itself then come from the caller's tensors.
  const bool direct = ring && c->chunk_ring_direct && prefill_tc_ring_direct_supported(c->geom, li.window) &&
                      prefill_tc_supported(c->cfg.dtype, D, q, k, v) && (((size_t)out) & 15) == 0;
  mixattn_ctx::GatherKey dummy;
  mixattn_ctx::GatherKey& held = direct ? dummy : c->scratch_holds;
  const bool reuse = !direct && c->chunk_reuse && one_piece && held.valid && held.owner == li.owner &&
                     held.epoch == c->cache_epoch && held.k == k && held.v == v && held.st == st &&
                     held.ids.size() == (size_t)n_seqs &&
                     std::equal(held.ids.begin(), held.ids.end(), seq_ids) &&
                     std::equal(held.lens.begin(), held.lens.end(), seq_lens);
  if (!reuse) {
    held.valid = false;   // set again below, once the copy of a one-piece call has been issued
    held.owner = li.owner;
    held.epoch = c->cache_epoch;
    held.k = k;
    held.v = v;
    held.st = st;
    held.ids.assign(seq_ids, seq_ids + n_seqs);
    held.lens.assign(seq_lens, seq_lens + n_seqs);
  }

  // groups of consecutive sequences whose keys fit the scratch together; the stream orders
  // each group's attention before the next group's copy reuses the scratch
  int64_t row = 0;   // first chunk row of the group in q / k / v / out
  for (int i0 = 0; i0 < n_seqs;) {
    int nb = 0, mlen = 0, max_rows = 0;
    int32_t krow = 0, qrow = 0;
    while (i0 + nb < n_seqs && nb < kMaxCallSeqs) {
      const int i = i0 + nb;
      const int rows = n_prefix[i] + seq_lens[i];
      if (krow + rows > scratch) break;
      GatherEntry& e = gp.e[nb];
      e.seq = seq_ids[i];
      e.n_prefix = n_prefix[i];
      e.pos0 = c->cm.len(layer, seq_ids[i]) - n_prefix[i];
      e.n_chunk = seq_lens[i];
      e.src_row0 = qrow;
      e.dst_row0 = krow;
      p.row0[nb] = qrow;
      p.krow0[nb] = direct ? qrow : krow;
      p.prefix[nb] = direct ? c->cm.len(layer, seq_ids[i]) : n_prefix[i];
      p.cached[nb] = p.prefix[nb];
      p.ring_page0[nb] = seq_ids[i] * ring_pages_of(li.window);
      krow += rows;
      qrow += seq_lens[i];
      if (seq_lens[i] > mlen) mlen = seq_lens[i];
      if (rows > max_rows) max_rows = rows;
      ++nb;
    }
    p.row0[nb] = qrow;
    p.n_seqs = nb;
    gp.n_entries = nb;
    gp.k_chunk = static_cast<const char*>(k) + (size_t)row * Hkv * D * esz;
    gp.v_chunk = static_cast<const char*>(v) + (size_t)row * Hkv * D * esz;
    p.q = static_cast<const char*>(q) + (size_t)row * Hq * D * esz;
    p.out = static_cast<char*>(out) + (size_t)row * Hq * D * esz;
    if (direct) {
      p.k = gp.k_chunk;
      p.v = gp.v_chunk;
      p.ring_pool = gp.pool;
      p.ring_pages = gp.ring_pages;
      p.ring_total_pages = (int64_t)c->cm.max_seqs() * gp.ring_pages;
      p.geom = c->geom;
    }
    cudaError_t e = cudaSuccess;
    if (!reuse && !direct) {
      e = launch_recorded(c, MIXATTN_K_GATHER, st, [&] { return launch_gather(gp, max_rows, st); });
      if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
      held.valid = one_piece;
    }
    const int cls = p.window ? MIXATTN_K_PREFILL_SLIDING : MIXATTN_K_PREFILL_FULL;
    const bool tc = prefill_tc_supported(c->cfg.dtype, D, p.q, p.k, p.v) && (((size_t)p.out) & 15) == 0;
    if (direct && !tc) return MIXATTN_ERR_INVALID_ARG;   // (not reachable: the pointers were checked above)
    e = launch_recorded(c, cls, st, [&] {
      return tc ? launch_prefill_tc(p, mlen, c->sm_count, st) : launch_prefill_simple(p, c->cfg.dtype, mlen, st);
    });
    if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
    row += qrow;
    i0 += nb;
  }
  return MIXATTN_OK;
}

int mixattn_get_len(mixattn_ctx* c, int32_t layer, int32_t seq, int32_t* len) {
  if (c == nullptr || len == nullptr || !c->cm.valid_layer(layer)) return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  *len = c->cm.len(layer, seq);
  return MIXATTN_OK;
}

int mixattn_get_block_table(mixattn_ctx* c, int32_t seq, int32_t* out, int32_t cap, int32_t* n_blocks) {
  if (c == nullptr || n_blocks == nullptr || cap < 0 || (cap > 0 && out == nullptr))
    return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  const int n = c->cm.n_blocks(seq);
  *n_blocks = n;
  const int m = n < cap ? n : cap;
  if (m > 0) memcpy(out, c->cm.table_row(seq), (size_t)m * sizeof(int32_t));
  return MIXATTN_OK;
}

int mixattn_get_n_free_pages(mixattn_ctx* c, int32_t* n_free) {
  if (c == nullptr || n_free == nullptr) return MIXATTN_ERR_INVALID_ARG;
  *n_free = c->cm.n_free();
  return MIXATTN_OK;
}

int mixattn_get_ring_state(mixattn_ctx* c, int32_t layer, int32_t seq, int32_t* next_slot, int32_t* n_valid) {
  if (c == nullptr || next_slot == nullptr || n_valid == nullptr || !c->cm.valid_layer(layer))
    return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  const LayerInfo& li = c->cm.layer(layer);
  if (li.kind != MIXATTN_SLIDING) return MIXATTN_ERR_INVALID_ARG;
  const int32_t n = c->cm.len(layer, seq);
  *next_slot = n % li.window;
  *n_valid = n < li.window ? n : li.window;
  return MIXATTN_OK;
}

int mixattn_locate(mixattn_ctx* c, int32_t layer, int32_t seq, int32_t pos, int32_t* page, int32_t* slot) {
  if (c == nullptr || page == nullptr || slot == nullptr || !c->cm.valid_layer(layer))
    return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  return c->cm.locate(layer, seq, pos, page, slot) ? MIXATTN_OK : MIXATTN_ERR_INVALID_ARG;
}

// Physical page (looked up in the DEVICE copy of the block table for a paged cache) and slot
// within it of a stored token; `slot` comes in as CacheManager::locate returned it.
static int stored_page_of(mixattn_ctx* c, int layer, int seq, int pos, int64_t* phys, int32_t* slot) {
  const LayerInfo& li = c->cm.layer(layer);
  if (li.kind == MIXATTN_FULL) {
    int32_t dev_page = -1;
    if (cudaMemcpy(&dev_page, c->dev_table() + (size_t)seq * c->cm.max_blocks() + pos / kPage,
                   sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
      return MIXATTN_ERR_CUDA;
    *phys = dev_page;
  } else {
    *phys = (int64_t)seq * ring_pages_of(li.window) + *slot / kPage;
    *slot = *slot % kPage;
  }
  return MIXATTN_OK;
}

// Copies one stored row (its 16-byte chunks put back in order) to `dst` (st_row_bytes bytes) and,
// for quantised storage, its shared exponent to *X.
static int read_stored_row(mixattn_ctx* c, const char* pool, int64_t phys, int gh, int which, int slot,
                           void* dst, int32_t* X) {
  const KvGeom& ge = c->geom;
  if (ge.fp8 && which == 1) {
    // quantised V is stored transposed: fetch the page's V^T and pick this token's column
    std::vector<unsigned char> vt((size_t)ge.head_dim * kPage);
    if (cudaMemcpy(vt.data(), pool + kv_fp8_v_offset(ge, phys, gh, 0, 0), vt.size(), cudaMemcpyDeviceToHost) != cudaSuccess)
      return MIXATTN_ERR_CUDA;
    for (int d = 0; d < ge.head_dim; ++d) static_cast<unsigned char*>(dst)[d] = vt[(size_t)d * kPage + slot];
  } else {
    unsigned char row[512];
    if (ge.st_row_bytes > (int)sizeof(row)) return MIXATTN_ERR_UNSUPPORTED;
    // start of the stored row; its 16-byte chunks are permuted unless the cache is fp32
    const char* src = pool + phys * ge.page_bytes + (int64_t)gh * ge.blk_bytes +
                      (int64_t)(which * kPage + slot) * ge.st_row_bytes;
    if (cudaMemcpy(row, src, ge.st_row_bytes, cudaMemcpyDeviceToHost) != cudaSuccess) return MIXATTN_ERR_CUDA;
    const int chunks = ge.st_row_bytes / 16;
    for (int ch = 0; ch < chunks; ++ch) {
      const int phys_ch = !ge.swizzle ? ch : ge.fp8 ? (ch ^ fp8_k_swizzle(slot)) : (ch ^ (slot & 7));
      memcpy(static_cast<char*>(dst) + ch * 16, row + phys_ch * 16, 16);
    }
  }
  if (ge.fp8 && X != nullptr) {
    unsigned char xb = 0;
    if (cudaMemcpy(&xb, pool + kv_exp_offset(ge, phys, gh, which, slot), 1, cudaMemcpyDeviceToHost) != cudaSuccess)
      return MIXATTN_ERR_CUDA;
    *X = (int32_t)xb - 127;
  }
  return MIXATTN_OK;
}

// bf16 bit pattern of an E4M3 code times 2^X (host side of the debug read; the format is the
// OCP 8-bit float: exponent bias 7, subnormals m/8 * 2^-6, no infinity).
static uint16_t bf16_bits_of_e4m3(unsigned char code, int X) {
  const int e = (code >> 3) & 0xF, m = code & 7;
  float v = e == 0 ? ldexpf((float)m, -9) : ldexpf(1.0f + (float)m / 8.0f, e - 7);
  v = ldexpf(v, X);
  if (code & 0x80) v = -v;
  uint32_t bits;
  memcpy(&bits, &v, 4);
  return (uint16_t)(bits >> 16);   // exact: four significant bits
}

int mixattn_debug_read_kv(mixattn_ctx* c, int32_t layer, int32_t seq, int32_t pos, void* k_host, void* v_host) {
  if (c == nullptr || k_host == nullptr || v_host == nullptr || !c->cm.valid_layer(layer))
    return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  int32_t page, slot;
  if (!c->cm.locate(layer, seq, pos, &page, &slot)) return MIXATTN_ERR_INVALID_ARG;
  if (c->host_only) return MIXATTN_ERR_CUDA;
  DeviceGuard g(c->device);
  if (!g.ok || cudaDeviceSynchronize() != cudaSuccess) return MIXATTN_ERR_CUDA;
  const KvGeom& ge = c->geom;
  int64_t phys;
  if (stored_page_of(c, layer, seq, pos, &phys, &slot) != MIXATTN_OK) return MIXATTN_ERR_CUDA;
  const char* pool = c->owner_storage(layer);
  std::vector<unsigned char> codes(ge.st_row_bytes);
  for (int which = 0; which < 2; ++which) {
    char* dst = static_cast<char*>(which ? v_host : k_host);
    for (int gh = 0; gh < ge.n_kv_heads; ++gh) {
      if (!ge.fp8) {
        if (read_stored_row(c, pool, phys, gh, which, slot, dst + (size_t)gh * ge.row_bytes, nullptr) != MIXATTN_OK)
          return MIXATTN_ERR_CUDA;
        continue;
      }
      // quantised storage: element * 2^X, which is a bf16 number
      int32_t X = 0;
      if (read_stored_row(c, pool, phys, gh, which, slot, codes.data(), &X) != MIXATTN_OK) return MIXATTN_ERR_CUDA;
      uint16_t* out = reinterpret_cast<uint16_t*>(dst + (size_t)gh * ge.row_bytes);
      for (int d = 0; d < ge.head_dim; ++d) out[d] = bf16_bits_of_e4m3(codes[d], X);
    }
  }
  return MIXATTN_OK;
}

int mixattn_debug_read_kv_fp8(mixattn_ctx* c, int32_t layer, int32_t seq, int32_t pos, uint8_t* k_codes,
                              int32_t* k_exp, uint8_t* v_codes, int32_t* v_exp) {
  if (c == nullptr || k_codes == nullptr || k_exp == nullptr || v_codes == nullptr || v_exp == nullptr ||
      !c->cm.valid_layer(layer))
    return MIXATTN_ERR_INVALID_ARG;
  if (!c->cm.valid_seq(seq)) return MIXATTN_ERR_BAD_SEQ;
  if (!c->geom.fp8) return MIXATTN_ERR_UNSUPPORTED;
  int32_t page, slot;
  if (!c->cm.locate(layer, seq, pos, &page, &slot)) return MIXATTN_ERR_INVALID_ARG;
  if (c->host_only) return MIXATTN_ERR_CUDA;
  DeviceGuard g(c->device);
  if (!g.ok || cudaDeviceSynchronize() != cudaSuccess) return MIXATTN_ERR_CUDA;
  int64_t phys;
  if (stored_page_of(c, layer, seq, pos, &phys, &slot) != MIXATTN_OK) return MIXATTN_ERR_CUDA;
  const KvGeom& ge = c->geom;
  const char* pool = c->owner_storage(layer);
  for (int gh = 0; gh < ge.n_kv_heads; ++gh) {
    if (read_stored_row(c, pool, phys, gh, 0, slot, k_codes + (size_t)gh * ge.head_dim, &k_exp[gh]) != MIXATTN_OK ||
        read_stored_row(c, pool, phys, gh, 1, slot, v_codes + (size_t)gh * ge.head_dim, &v_exp[gh]) != MIXATTN_OK)
      return MIXATTN_ERR_CUDA;
  }
  return MIXATTN_OK;
}

int mixattn_get_device_status(mixattn_ctx* c, int32_t* status) {
  if (c == nullptr || status == nullptr) return MIXATTN_ERR_INVALID_ARG;
  if (c->host_only) return MIXATTN_ERR_CUDA;
  DeviceGuard g(c->device);
  if (!g.ok || cudaDeviceSynchronize() != cudaSuccess) return MIXATTN_ERR_CUDA;
  if (cudaMemcpy(status, c->dev_status(), sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
    return MIXATTN_ERR_CUDA;
  return MIXATTN_OK;
}

int mixattn_set_split_tokens(mixattn_ctx* c, int32_t tokens) {
  if (c == nullptr || tokens < 0) return MIXATTN_ERR_INVALID_ARG;
  c->split_tokens = tokens;
  return MIXATTN_OK;
}

int mixattn_set_chunk_gather_reuse(mixattn_ctx* c, int32_t enable) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  c->chunk_reuse = enable != 0;
  c->scratch_holds.valid = false;
  return MIXATTN_OK;
}

int mixattn_set_chunk_ring_direct(mixattn_ctx* c, int32_t enable) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  c->chunk_ring_direct = enable != 0;
  return MIXATTN_OK;
}

int mixattn_profile_enable(mixattn_ctx* c, int32_t enable) {
  if (c == nullptr) return MIXATTN_ERR_INVALID_ARG;
  if (c->host_only) return MIXATTN_ERR_CUDA;
  for (auto& r : c->records) {
    if (r.start) c->event_pool.push_back(r.start);
    if (r.stop) c->event_pool.push_back(r.stop);
  }
  c->records.clear();
  c->profiling = enable != 0;
  return MIXATTN_OK;
}

int mixattn_profile_read(mixattn_ctx* c, int32_t cls, int32_t* launches, float* ms) {
  if (c == nullptr || launches == nullptr || ms == nullptr || cls < 0 || cls >= MIXATTN_K_COUNT)
    return MIXATTN_ERR_INVALID_ARG;
  if (c->host_only) return MIXATTN_ERR_CUDA;
  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  int n = 0;
  float total = 0.f;
  for (auto& r : c->records) {
    if (r.cls != cls || !r.start || !r.stop) continue;
    if (cudaEventSynchronize(r.stop) != cudaSuccess) return MIXATTN_ERR_CUDA;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.start, r.stop) != cudaSuccess) return MIXATTN_ERR_CUDA;
    total += t;
    ++n;
  }
  *launches = n;
  *ms = total;
  return MIXATTN_OK;
}

// ---------------------------------------------------------------------------
// Decode with the split-KV scratch in a static device array (no arena workspace used).
// ---------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = MIXATTN_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Lives in every GPU context that loads this library, until the process exits.
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

// Device address of g_decode_scratch per device ordinal.  In host code the array's name
// is only a handle for the runtime; the address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
// Contexts on several threads may make their first call at once: the slots are atomic (every
// thread that asks gets the same address, so a relaxed load / store is enough).  The address is
// kept until the process exits; it does not survive a cudaDeviceReset of that device.
std::atomic<void*> g_decode_scratch_ptr[kMaxDevices];

int static_scratch_for_current_device(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return MIXATTN_ERR_INVALID_ARG;
  void* ptr = g_decode_scratch_ptr[device].load(std::memory_order_relaxed);
  if (ptr == nullptr) {
    if (cudaGetSymbolAddress(&ptr, g_decode_scratch) != cudaSuccess || ptr == nullptr) return MIXATTN_ERR_CUDA;
    g_decode_scratch_ptr[device].store(ptr, std::memory_order_relaxed);
  }
  *out = ptr;
  return MIXATTN_OK;
}

}  // namespace

int mixattn_decode_static_scratch(mixattn_ctx* c, int32_t layer, int32_t n_seqs, const int32_t* seq_ids,
                                  const void* q, void* out, void* stream) {
  if (c == nullptr || !c->cm.valid_layer(layer) || n_seqs < 0) return MIXATTN_ERR_INVALID_ARG;
  if (n_seqs > 0 && (seq_ids == nullptr || q == nullptr || out == nullptr)) return MIXATTN_ERR_INVALID_ARG;
  for (int i = 0; i < n_seqs; ++i) {
    if (!c->cm.valid_seq(seq_ids[i])) return MIXATTN_ERR_BAD_SEQ;
  }
  for (int i = 0; i < n_seqs; ++i) {
    if (c->cm.len(layer, seq_ids[i]) < 1) return MIXATTN_ERR_EMPTY_CONTEXT;
  }
  if (c->host_only || c->sticky_cuda_error) return MIXATTN_ERR_CUDA;
  if (n_seqs == 0) return MIXATTN_OK;
  if (n_seqs > kMaxCallSeqs) return MIXATTN_ERR_TOO_LARGE;

  const LayerInfo& li = c->cm.layer(layer);
  const bool ring = li.kind == MIXATTN_SLIDING;
  const int Hq = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;

  DecodeParams p;
  p.group = Hq / Hkv;
  p.head_chunks = (p.group + kMaxGroupRows - 1) / kMaxGroupRows;
  // the split plan of mixattn_decode (one function), so both calls add the partial results in
  // the same order and give the same bits
  bool any_split = false;
  const int base = plan_splits(c, layer, seq_ids, n_seqs, &p, &any_split);
  // scratch needed: per split and query head, D partial outputs + (max, sum)
  const size_t part_o_bytes = align_up((size_t)base * Hq * D * sizeof(float));
  const size_t need = part_o_bytes + (size_t)base * Hq * sizeof(float2);
  if (need > kStaticScratchBytes) return MIXATTN_ERR_TOO_LARGE;

  DeviceGuard g(c->device);
  if (!g.ok) return MIXATTN_ERR_CUDA;
  void* scratch = nullptr;
  int rc = static_scratch_for_current_device(c->device, &scratch);
  if (rc != MIXATTN_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  p.q = q;
  p.out = out;
  p.pool = c->owner_storage(layer);
  p.table = ring ? nullptr : c->dev_table();
  p.table_stride = c->cm.max_blocks();
  p.ring_pages = ring ? ring_pages_of(li.window) : 0;
  p.geom = c->geom;
  p.n_q_heads = Hq;
  p.scale_log2e = c->scale * 1.4426950408889634f;
  set_l2_policy(c, layer, &p);
  // every partial slot that the combine pass reads is written by the split pass of the
  // same call first, so nothing in the array has to start at zero
  p.part_o = reinterpret_cast<float*>(scratch);
  p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(scratch) + part_o_bytes);
  p.status = c->dev_status();
  const int cls = ring ? MIXATTN_K_DECODE_SLIDING : MIXATTN_K_DECODE_FULL;
  cudaError_t e = launch_recorded(c, cls, st, [&] {
    return c->cfg.dtype == MIXATTN_BF16 ? launch_decode_split_bf16(p, c->sm_count, st)
                                        : launch_decode_split_f32(p, st);
  });
  if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
  if (any_split) {
    e = launch_recorded(c, MIXATTN_K_COMBINE, st, [&] { return launch_decode_combine(p, c->cfg.dtype, st); });
    if (e != cudaSuccess) return MIXATTN_ERR_CUDA;
  }
  return MIXATTN_OK;
}

int mixattn_get_launch_count(mixattn_ctx* c, int64_t* launches) {
  if (c == nullptr || launches == nullptr) return MIXATTN_ERR_INVALID_ARG;
  *launches = c->launches;
  return MIXATTN_OK;
}

const char* mixattn_strerror(int code) {
  switch (code) {
    case MIXATTN_OK: return "ok";
    case MIXATTN_ERR_INVALID_ARG: return "invalid argument";
    case MIXATTN_ERR_INVALID_LAYOUT: return "invalid layer layout";
    case MIXATTN_ERR_NOT_OWNER: return "layer reuses another layer's KV cache and takes no K/V";
    case MIXATTN_ERR_OUT_OF_PAGES: return "not enough free pages";
    case MIXATTN_ERR_EMPTY_CONTEXT: return "sequence has no cached token";
    case MIXATTN_ERR_BAD_SEQ: return "sequence id out of range";
    case MIXATTN_ERR_UNSUPPORTED: return "unsupported request";
    case MIXATTN_ERR_CUDA: return "CUDA error or host-only context";
    case MIXATTN_ERR_TOO_LARGE: return "request needs more scratch than the static array holds";
    default: return "unknown status";
  }
}

}  // extern "C"

// Host-side KV-cache bookkeeping: layout resolution, the FIFO page allocator, block
// tables, ring positions and per-owner length counters.  Pure C++ (no CUDA): the host
// copy is authoritative, the device only mirrors the block tables.
//
// Paper, Section 3: a layer either computes its own KV cache or reuses the cache of an
// earlier layer; a sliding-window cache keeps the past `window` tokens.
#pragma once

#include <stdint.h>

#include <deque>
#include <vector>

#include "mixattn.h"

namespace mixattn {

struct LayerInfo {
  int32_t kind;
  int32_t window;
  int32_t owner;       // layer whose cache this layer reads
  int32_t owner_slot;  // index of that owner among owners (storage handle)
};

struct PageGrant {     // a block-table entry set during an append
  int32_t seq;
  int32_t block;
  int32_t page;
};

class CacheManager {
 public:
  static constexpr int kPageSize = 16;

  // Validates the config; returns MIXATTN_OK or an error code (then *this is unusable).
  // `allocate` false: only resolve the layout and sizes (for the byte-count queries).
  int init(const mixattn_config& cfg, bool allocate = true) {
    if (cfg.n_layers <= 0 || cfg.layers == nullptr) return MIXATTN_ERR_INVALID_LAYOUT;
    if (cfg.n_q_heads <= 0 || cfg.n_kv_heads <= 0 || cfg.n_q_heads % cfg.n_kv_heads != 0)
      return MIXATTN_ERR_INVALID_ARG;
    if (cfg.head_dim != 64 && cfg.head_dim != 128) return MIXATTN_ERR_INVALID_ARG;
    if (cfg.dtype != MIXATTN_F32 && cfg.dtype != MIXATTN_BF16) return MIXATTN_ERR_INVALID_ARG;
    if (cfg.page_size != kPageSize || cfg.max_seqs <= 0 || cfg.n_pages < 0 || cfg.max_seq_len < 0)
      return MIXATTN_ERR_INVALID_ARG;
    layers_.clear();
    owners_.clear();
    for (int l = 0; l < cfg.n_layers; ++l) {
      const mixattn_layer_desc& d = cfg.layers[l];
      if (d.kind != MIXATTN_FULL && d.kind != MIXATTN_SLIDING) return MIXATTN_ERR_INVALID_LAYOUT;
      if (d.kind == MIXATTN_SLIDING && d.window < 1) return MIXATTN_ERR_INVALID_LAYOUT;
      if (d.kv_owner_layer < 0 || d.kv_owner_layer > l) return MIXATTN_ERR_INVALID_LAYOUT;
      const mixattn_layer_desc& o = cfg.layers[d.kv_owner_layer];
      if (o.kv_owner_layer != d.kv_owner_layer) return MIXATTN_ERR_INVALID_LAYOUT;
      if (o.kind != d.kind) return MIXATTN_ERR_INVALID_LAYOUT;
      if (d.kind == MIXATTN_SLIDING && o.window != d.window) return MIXATTN_ERR_INVALID_LAYOUT;
      layers_.push_back(LayerInfo{d.kind, d.kind == MIXATTN_SLIDING ? d.window : 0, d.kv_owner_layer, -1});
    }
    for (int l = 0; l < cfg.n_layers; ++l) {
      if (layers_[l].owner == l) {
        layers_[l].owner_slot = (int32_t)owners_.size();
        owners_.push_back(l);
      }
    }
    for (auto& li : layers_) li.owner_slot = layers_[li.owner].owner_slot;
    n_full_owners_ = 0;
    for (int o : owners_) n_full_owners_ += layers_[o].kind == MIXATTN_FULL;
    max_seqs_ = cfg.max_seqs;
    n_pages_ = cfg.n_pages;
    int64_t cap = (int64_t)cfg.n_pages * kPageSize;
    int64_t msl = cfg.max_seq_len > 0 ? cfg.max_seq_len : cap;
    if (msl > INT32_MAX - kPageSize) return MIXATTN_ERR_INVALID_ARG;
    if (msl < 1) msl = 1;
    max_seq_len_ = (int32_t)msl;
    max_blocks_ = (max_seq_len_ + kPageSize - 1) / kPageSize;
    if ((int64_t)max_seqs_ * max_blocks_ > INT32_MAX) return MIXATTN_ERR_INVALID_ARG;   // table entries are indexed in 32 bits
    free_.clear();
    if (cfg.free_order) {
      std::vector<char> seen(cfg.n_pages, 0);
      for (int i = 0; i < cfg.n_pages; ++i) {
        int32_t pg = cfg.free_order[i];
        if (pg < 0 || pg >= cfg.n_pages || seen[pg]) return MIXATTN_ERR_INVALID_ARG;
        seen[pg] = 1;
        if (allocate) free_.push_back(pg);
      }
    } else if (allocate) {
      for (int i = 0; i < cfg.n_pages; ++i) free_.push_back(i);
    }
    if (allocate) {
      table_.assign((size_t)max_seqs_ * max_blocks_, -1);
      n_blocks_.assign(max_seqs_, 0);
      len_.assign(owners_.size() * (size_t)max_seqs_, 0);
    }
    return MIXATTN_OK;
  }

  int n_layers() const { return (int)layers_.size(); }
  const LayerInfo& layer(int l) const { return layers_[l]; }
  const std::vector<int>& owners() const { return owners_; }
  int n_full_owners() const { return n_full_owners_; }
  int max_seqs() const { return max_seqs_; }
  int n_pages() const { return n_pages_; }
  int max_blocks() const { return max_blocks_; }
  int max_seq_len() const { return max_seq_len_; }
  int n_free() const { return (int)free_.size(); }
  bool valid_layer(int l) const { return l >= 0 && l < (int)layers_.size(); }
  bool valid_seq(int s) const { return s >= 0 && s < max_seqs_; }

  int32_t len(int layer, int seq) const {
    return len_[(size_t)layers_[layer].owner_slot * max_seqs_ + seq];
  }
  int32_t n_blocks(int seq) const { return n_blocks_[seq]; }
  const int32_t* table_row(int seq) const { return &table_[(size_t)seq * max_blocks_]; }

  // Keys a decode of `layer` attends to for `seq`: all of them, or the last `window`.
  int32_t n_attended(int layer, int seq) const {
    int32_t n = len(layer, seq);
    const LayerInfo& li = layers_[layer];
    return li.kind == MIXATTN_SLIDING && n > li.window ? li.window : n;
  }

  // Checks an append call; nothing changes.
  int check_append(int layer, int n_seqs, const int32_t* seq_ids, const int32_t* n_new) const {
    if (!valid_layer(layer) || n_seqs < 0 || (n_seqs > 0 && seq_ids == nullptr))
      return MIXATTN_ERR_INVALID_ARG;
    const LayerInfo& li = layers_[layer];
    if (li.owner != layer) return MIXATTN_ERR_NOT_OWNER;
    std::vector<char> seen(max_seqs_, 0);
    int64_t need = 0;
    for (int i = 0; i < n_seqs; ++i) {
      int s = seq_ids[i];
      if (!valid_seq(s)) return MIXATTN_ERR_BAD_SEQ;
      if (seen[s]) return MIXATTN_ERR_INVALID_ARG;
      seen[s] = 1;
      int64_t n = n_new ? n_new[i] : 1;
      if (n < 0) return MIXATTN_ERR_INVALID_ARG;
      int64_t end = (int64_t)len(layer, s) + n;
      if (end > max_seq_len_) return MIXATTN_ERR_INVALID_ARG;
      if (li.kind == MIXATTN_FULL) {
        int64_t blocks = (end + kPageSize - 1) / kPageSize;
        if (blocks > n_blocks_[s]) need += blocks - n_blocks_[s];
      }
    }
    if (need > (int64_t)free_.size()) return MIXATTN_ERR_OUT_OF_PAGES;
    return MIXATTN_OK;
  }

  // Applies an append that check_append accepted.  Pages are popped from the FIFO head,
  // sequences in call order, blocks in position order; every new table entry is
  // reported in `grants`.
  void apply_append(int layer, int n_seqs, const int32_t* seq_ids, const int32_t* n_new,
                    std::vector<PageGrant>* grants) {
    const LayerInfo& li = layers_[layer];
    for (int i = 0; i < n_seqs; ++i) {
      int s = seq_ids[i];
      int32_t n = n_new ? n_new[i] : 1;
      int32_t& L = len_[(size_t)li.owner_slot * max_seqs_ + s];
      int32_t end = L + n;
      if (li.kind == MIXATTN_FULL) {
        int32_t blocks = (end + kPageSize - 1) / kPageSize;
        while (n_blocks_[s] < blocks) {
          int32_t pg = free_.front();
          free_.pop_front();
          table_[(size_t)s * max_blocks_ + n_blocks_[s]] = pg;
          if (grants) grants->push_back(PageGrant{s, n_blocks_[s], pg});
          ++n_blocks_[s];
        }
      }
      L = end;
    }
  }

  void seq_reset(int seq) {
    for (size_t o = 0; o < owners_.size(); ++o) len_[o * max_seqs_ + seq] = 0;
    for (int b = 0; b < n_blocks_[seq]; ++b) {
      free_.push_back(table_[(size_t)seq * max_blocks_ + b]);
      table_[(size_t)seq * max_blocks_ + b] = -1;
    }
    n_blocks_[seq] = 0;
  }

  // Page and slot of a stored token; false if it is not stored (any more).
  bool locate(int layer, int seq, int pos, int32_t* page, int32_t* slot) const {
    const LayerInfo& li = layers_[layer];
    int32_t n = len(layer, seq);
    int32_t lo = li.kind == MIXATTN_SLIDING && n > li.window ? n - li.window : 0;
    if (pos < lo || pos >= n) return false;
    if (li.kind == MIXATTN_FULL) {
      *page = table_[(size_t)seq * max_blocks_ + pos / kPageSize];
      *slot = pos % kPageSize;
    } else {
      *page = -1;
      *slot = pos % li.window;
    }
    return true;
  }

 private:
  std::vector<LayerInfo> layers_;
  std::vector<int> owners_;
  int n_full_owners_ = 0;
  int max_seqs_ = 0, n_pages_ = 0, max_seq_len_ = 0, max_blocks_ = 0;
  std::deque<int32_t> free_;
  std::vector<int32_t> table_;
  std::vector<int32_t> n_blocks_;
  std::vector<int32_t> len_;
};

}  // namespace mixattn

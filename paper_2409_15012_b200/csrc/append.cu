// KV append: writes new tokens' K/V into a paged pool (through the block table) or a ring
// buffer (slot = position mod window), in the page format described in internal.h.
//
// Paper, Section 1 (keys/values of earlier tokens are cached) and Section 3 (a window-s
// cache keeps the past s tokens).  HBM-bound copy; 16-byte vector accesses.
#include "internal.h"

namespace mixattn {

namespace {

constexpr int kThreads = 256;
constexpr int kTokensPerBlock = 8;

__global__ void __launch_bounds__(kThreads) append_kernel(const __grid_constant__ AppendParams p) {
  const AppendEntry& e = p.e[blockIdx.y];
  const KvGeom& ge = p.geom;
  if (blockIdx.x == 0 && threadIdx.x == 0 && e.tbl_idx >= 0) p.table[e.tbl_idx] = e.page_hint;
  const int tok0 = blockIdx.x * kTokensPerBlock;
  if (tok0 >= e.n_new) return;
  // a ring only keeps the last `window` tokens: older ones of this call would be
  // overwritten by newer ones of the same call, so they are skipped outright
  const int first_kept = (p.is_ring && e.n_new > p.window) ? e.n_new - p.window : 0;
  const int chunks_row = ge.row_bytes / 16;
  const int chunks_tok = 2 * ge.n_kv_heads * chunks_row;  // K and V
  const int n_tok = min(kTokensPerBlock, e.n_new - tok0);
  for (int w = threadIdx.x; w < n_tok * chunks_tok; w += kThreads) {
    const int t = tok0 + w / chunks_tok;
    if (t < first_kept) continue;
    int r = w % chunks_tok;
    const int which = r / (ge.n_kv_heads * chunks_row);
    r -= which * ge.n_kv_heads * chunks_row;
    const int g = r / chunks_row;
    const int chunk = r - g * chunks_row;
    const int pos = e.start_pos + t;
    int64_t page;
    int slot;
    if (p.is_ring) {
      const int rs = pos % p.window;
      page = (int64_t)e.seq * p.ring_pages + rs / kPage;
      slot = rs % kPage;
    } else {
      page = e.page_hint >= 0 ? e.page_hint
                              : p.table[(int64_t)e.seq * p.table_stride + pos / kPage];
      slot = pos % kPage;
    }
    const char* src = (const char*)(which ? p.v : p.k) +
                      ((int64_t)(e.src_row0 + t) * ge.n_kv_heads + g) * ge.row_bytes + chunk * 16;
    char* dst = p.pool + kv_chunk_offset(ge, page, g, which, slot, chunk);
    *reinterpret_cast<int4*>(dst) = *reinterpret_cast<const int4*>(src);
  }
}

}  // namespace

cudaError_t launch_append(const AppendParams& p, int max_n_new, cudaStream_t st) {
  if (p.n_entries <= 0) return cudaSuccess;
  int bx = (max_n_new + kTokensPerBlock - 1) / kTokensPerBlock;
  if (bx < 1) bx = 1;
  dim3 grid(bx, p.n_entries);
  append_kernel<<<grid, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace mixattn

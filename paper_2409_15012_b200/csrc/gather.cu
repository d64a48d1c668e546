// Gathers the cached keys and values that a chunk of queries attends to, followed by the
// chunk's own, into plain [rows, Hkv, D] tensors.
//
// Paper, Section 3: a query attends to every earlier key (standard layer) or to the last
// `window` keys (sliding window); Section 5 serves long prompts, which arrive in chunks.
// The prompt kernels read contiguous row-major K / V; this copy undoes the page format
// (block table or ring slot, chunk swizzle).  HBM-bound; 16-byte vector accesses; its
// bytes are a few percent of the time of the attention that follows.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kThreads = 256;
constexpr int kTokensPerBlock = 8;

__global__ void __launch_bounds__(kThreads) gather_kernel(const __grid_constant__ GatherParams p) {
  const GatherEntry& e = p.e[blockIdx.y];
  const KvGeom& ge = p.geom;
  const int n_rows = e.n_prefix + e.n_chunk;
  const int tok0 = blockIdx.x * kTokensPerBlock;
  if (tok0 >= n_rows) return;
  const int chunks_row = ge.row_bytes / 16;
  const int chunks_tok = 2 * ge.n_kv_heads * chunks_row;  // K and V
  const int n_tok = min(kTokensPerBlock, n_rows - tok0);
  for (int w = threadIdx.x; w < n_tok * chunks_tok; w += kThreads) {
    const int t = tok0 + w / chunks_tok;
    int r = w % chunks_tok;
    const int which = r / (ge.n_kv_heads * chunks_row);
    r -= which * ge.n_kv_heads * chunks_row;
    const int g = r / chunks_row;
    const int chunk = r - g * chunks_row;
    const char* src;
    if (t < e.n_prefix) {
      const int pos = e.pos0 + t;
      int64_t page;
      int slot;
      if (p.is_ring) {
        const int rs = pos % p.window;
        page = (int64_t)e.seq * p.ring_pages + rs / kPage;
        slot = rs % kPage;
      } else {
        page = p.table[(int64_t)e.seq * p.table_stride + pos / kPage];
        slot = pos % kPage;
      }
      src = p.pool + kv_chunk_offset(ge, page, g, which, slot, chunk);
    } else {
      src = (const char*)(which ? p.v_chunk : p.k_chunk) +
            ((int64_t)(e.src_row0 + t - e.n_prefix) * ge.n_kv_heads + g) * ge.row_bytes + chunk * 16;
    }
    char* dst = (char*)(which ? p.v_out : p.k_out) +
                ((int64_t)(e.dst_row0 + t) * ge.n_kv_heads + g) * ge.row_bytes + chunk * 16;
    *reinterpret_cast<int4*>(dst) = *reinterpret_cast<const int4*>(src);
  }
}

// Quantised storage: a cached element reads as code * 2^X, which is a bf16 number, so the copy
// dequantises exactly; the chunk's own rows are bf16 already.  One thread per 16 bytes written.
__global__ void __launch_bounds__(kThreads) gather_fp8_kernel(const __grid_constant__ GatherParams p) {
  const GatherEntry& e = p.e[blockIdx.y];
  const KvGeom& ge = p.geom;
  const int n_rows = e.n_prefix + e.n_chunk;
  const int tok0 = blockIdx.x * kTokensPerBlock;
  if (tok0 >= n_rows) return;
  const int chunks_row = ge.row_bytes / 16;               // 16-byte pieces of a bf16 row (8 channels each)
  const int chunks_tok = 2 * ge.n_kv_heads * chunks_row;
  const int n_tok = min(kTokensPerBlock, n_rows - tok0);
  for (int w = threadIdx.x; w < n_tok * chunks_tok; w += kThreads) {
    const int t = tok0 + w / chunks_tok;
    int r = w % chunks_tok;
    const int which = r / (ge.n_kv_heads * chunks_row);
    r -= which * ge.n_kv_heads * chunks_row;
    const int g = r / chunks_row;
    const int chunk = r - g * chunks_row;
    int4 val;
    if (t < e.n_prefix) {
      const int pos = e.pos0 + t;
      int64_t page;
      int slot;
      if (p.is_ring) {
        const int rs = pos % p.window;
        page = (int64_t)e.seq * p.ring_pages + rs / kPage;
        slot = rs % kPage;
      } else {
        page = p.table[(int64_t)e.seq * p.table_stride + pos / kPage];
        slot = pos % kPage;
      }
      uint2 codes;
      if (which == 0) {   // 8 codes = half of a stored 16-byte chunk
        codes = *reinterpret_cast<const uint2*>(p.pool + kv_chunk_offset(ge, page, g, 0, slot, chunk >> 1) + (chunk & 1) * 8);
      } else {            // V is stored transposed: one byte per channel row
        const unsigned char* src = reinterpret_cast<const unsigned char*>(p.pool) + kv_fp8_v_offset(ge, page, g, chunk * 8, slot);
        uint32_t w[2] = {0u, 0u};
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i >> 2] |= (uint32_t)src[i * kPage] << (8 * (i & 3));
        codes = make_uint2(w[0], w[1]);
      }
      const int X = (int)*reinterpret_cast<const unsigned char*>(p.pool + kv_exp_offset(ge, page, g, which, slot)) - 127;
      const float scale = X > -127 ? __int_as_float((X + 127) << 23) : __int_as_float(0x00400000);   // 2^X (2^-127 is subnormal)
      const uint32_t cw[2] = {codes.x, codes.y};
      int out[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(cw[i >> 1] >> (16 * (i & 1))), __NV_E4M3);
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hr));
        const __nv_bfloat162 b = __floats2bfloat162_rn(f.x * scale, f.y * scale);
        out[i] = *reinterpret_cast<const int*>(&b);
      }
      val = make_int4(out[0], out[1], out[2], out[3]);
    } else {
      val = *reinterpret_cast<const int4*>((const char*)(which ? p.v_chunk : p.k_chunk) +
            ((int64_t)(e.src_row0 + t - e.n_prefix) * ge.n_kv_heads + g) * ge.row_bytes + chunk * 16);
    }
    char* dst = (char*)(which ? p.v_out : p.k_out) +
                ((int64_t)(e.dst_row0 + t) * ge.n_kv_heads + g) * ge.row_bytes + chunk * 16;
    *reinterpret_cast<int4*>(dst) = val;
  }
}

}  // namespace

cudaError_t launch_gather(const GatherParams& p, int max_rows, cudaStream_t st) {
  if (p.n_entries <= 0 || max_rows <= 0) return cudaSuccess;
  dim3 grid((max_rows + kTokensPerBlock - 1) / kTokensPerBlock, p.n_entries);
  if (p.geom.fp8) gather_fp8_kernel<<<grid, kThreads, 0, st>>>(p);
  else gather_kernel<<<grid, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace mixattn

// Split-KV decode for fp32 caches (true fp32 FMAs, no tensor cores) and the split-combine
// pass shared by both dtypes.
//
// Paper, Section 3 (standard and sliding-window attention over the cache a layer reads).
// The fp32 path exists for exact-arithmetic checks; it streams K/V rows straight from
// HBM with one warp per key and warp-shuffle reductions.
#include <cuda_bf16.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kWarps = 4;
constexpr int kRowsPerPass = 4;  // query heads kept in registers per pass over the keys

// one work item = (split, KV head, chunk of 16 heads); grid.x = total_items
template <int D>
__global__ void __launch_bounds__(kWarps * 32) decode_split_f32_kernel(const __grid_constant__ DecodeParams p) {
  constexpr int V = D / 32;  // floats per lane per row
  __shared__ float sm_o[kWarps][kRowsPerPass][D];
  __shared__ float sm_ml[kWarps][kRowsPerPass][2];

  const int it = blockIdx.x;
  const int hc = it % p.head_chunks;
  int r_ = it / p.head_chunks;
  const int g = r_ % p.geom.n_kv_heads;
  const int cg = r_ / p.geom.n_kv_heads;
  int lo = 0, hi = p.n_seqs;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.chunk_base[mid] <= cg) lo = mid; else hi = mid;
  }
  const int i = lo;
  const int c = cg - p.chunk_base[i];
  const int n_splits = p.chunk_base[i + 1] - p.chunk_base[i];
  const int t0 = c * p.chunk_len[i];
  const int t1 = min(p.n_eff[i], t0 + p.chunk_len[i]);
  const int seq = p.seq_id[i];
  const int rows = min(kMaxGroupRows, p.group - hc * kMaxGroupRows);
  const int h0 = g * p.group + hc * kMaxGroupRows;
  const KvGeom& ge = p.geom;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int32_t* tbl = p.table ? p.table + (int64_t)seq * p.table_stride : nullptr;

  for (int r0 = 0; r0 < rows; r0 += kRowsPerPass) {
    const int nr = min(kRowsPerPass, rows - r0);
    float q[kRowsPerPass][V], o[kRowsPerPass][V], m[kRowsPerPass], l[kRowsPerPass];
#pragma unroll
    for (int r = 0; r < kRowsPerPass; ++r) {
      m[r] = -INFINITY;
      l[r] = 0.f;
#pragma unroll
      for (int e = 0; e < V; ++e) {
        o[r][e] = 0.f;
        q[r][e] = r < nr ? reinterpret_cast<const float*>(p.q)[((int64_t)i * p.n_q_heads + h0 + r0 + r) * D +
                                                                 lane * V + e]
                         : 0.f;
      }
    }
    for (int t = t0 + warp; t < t1; t += kWarps) {
      const int64_t page = tbl ? (int64_t)tbl[t / kPage] : (int64_t)seq * p.ring_pages + t / kPage;
      const char* blk = p.pool + page * ge.page_bytes + (int64_t)g * ge.blk_bytes;
      const float* kr = reinterpret_cast<const float*>(blk + (int64_t)(t % kPage) * ge.row_bytes) + lane * V;
      const float* vr = kr + kPage * D;
      float kv[V], vv[V];
#pragma unroll
      for (int e = 0; e < V; ++e) {
        kv[e] = kr[e];
        vv[e] = vr[e];
      }
#pragma unroll
      for (int r = 0; r < kRowsPerPass; ++r) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < V; ++e) s = fmaf(q[r][e], kv[e], s);
#pragma unroll
        for (int sh = 16; sh > 0; sh >>= 1) s += __shfl_xor_sync(0xffffffffu, s, sh);
        s *= p.scale_log2e;
        const float mn = fmaxf(m[r], s);
        const float a = exp2f(m[r] - mn);
        const float pe = exp2f(s - mn);
        m[r] = mn;
        l[r] = l[r] * a + pe;
#pragma unroll
        for (int e = 0; e < V; ++e) o[r][e] = fmaf(pe, vv[e], o[r][e] * a);
      }
    }
#pragma unroll
    for (int r = 0; r < kRowsPerPass; ++r) {
#pragma unroll
      for (int e = 0; e < V; ++e) sm_o[warp][r][lane * V + e] = o[r][e];
      if (lane == 0) {
        sm_ml[warp][r][0] = m[r];
        sm_ml[warp][r][1] = l[r];
      }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < nr * D; e += kWarps * 32) {
      const int r = e / D, d = e - r * D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_ml[w][r][0]);
      float L = 0.f, acc = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float sc = exp2f(sm_ml[w][r][0] - M);
        L += sm_ml[w][r][1] * sc;
        acc += sm_o[w][r][d] * sc;
      }
      const int h = h0 + r0 + r;
      if (n_splits == 1) {
        reinterpret_cast<float*>(p.out)[((int64_t)i * p.n_q_heads + h) * D + d] = acc / L;
      } else {
        const int64_t slot = (int64_t)(p.chunk_base[i] + c) * p.n_q_heads + h;
        p.part_o[slot * D + d] = acc;
        if (d == 0) p.part_ml[slot] = make_float2(M, L);
      }
    }
    __syncthreads();
  }
}

// out[i, h, :] = sum_c o_c * 2^(m_c - M) / sum_c l_c * 2^(m_c - M) over the splits of a
// sequence; sequences with a single split were already written by the split pass.
template <typename T>
__global__ void decode_combine_kernel(const __grid_constant__ DecodeParams p) {
  const int i = blockIdx.y, h = blockIdx.x, d = threadIdx.x;
  const int D = p.geom.head_dim;
  const int c0 = p.chunk_base[i], n = p.chunk_base[i + 1] - c0;
  if (n <= 1) return;
  float M = -INFINITY;
  for (int c = 0; c < n; ++c) M = fmaxf(M, p.part_ml[(int64_t)(c0 + c) * p.n_q_heads + h].x);
  float L = 0.f, acc = 0.f;
  for (int c = 0; c < n; ++c) {
    const int64_t slot = (int64_t)(c0 + c) * p.n_q_heads + h;
    const float2 ml = p.part_ml[slot];
    const float sc = exp2f(ml.x - M);
    L += ml.y * sc;
    acc += p.part_o[slot * D + d] * sc;
  }
  const float r = acc / L;
  T* out = reinterpret_cast<T*>(p.out) + ((int64_t)i * p.n_q_heads + h) * D + d;
  if constexpr (sizeof(T) == 2) *out = __float2bfloat16_rn(r); else *out = r;
}

}  // namespace

cudaError_t launch_decode_split_f32(const DecodeParams& p, cudaStream_t st) {
  if (p.total_items <= 0) return cudaSuccess;
  if (p.geom.head_dim == 128)
    decode_split_f32_kernel<128><<<p.total_items, kWarps * 32, 0, st>>>(p);
  else
    decode_split_f32_kernel<64><<<p.total_items, kWarps * 32, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_decode_combine(const DecodeParams& p, int dtype, cudaStream_t st) {
  dim3 grid(p.n_q_heads, p.n_seqs);
  if (dtype == MIXATTN_BF16)
    decode_combine_kernel<__nv_bfloat16><<<grid, p.geom.head_dim, 0, st>>>(p);
  else
    decode_combine_kernel<float><<<grid, p.geom.head_dim, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace mixattn

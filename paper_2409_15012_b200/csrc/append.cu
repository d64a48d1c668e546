// KV append: writes new tokens' K/V into a paged pool (through the block table) or a ring
// buffer (slot = position mod window), in the page format described in internal.h.
//
// Paper, Section 1 (keys/values of earlier tokens are cached) and Section 3 (a window-s
// cache keeps the past s tokens).  HBM-bound copy; 16-byte vector accesses.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kThreads = 256;
constexpr int kTokensPerBlock = 8;

// Rotary position embedding of one 16-byte chunk of a key row (RoFormer's definition, which
// Section 3 of the paper cites): channel pair (2i, 2i+1) at position m turns by the angle
// m * theta^(-2i/d).  The angle is formed and reduced modulo 2 pi in double precision
// (positions reach 10^5 and the first pairs turn by about a radian per position), the
// rotation itself runs in fp32, and bf16 rows are rounded once.
__device__ __forceinline__ void rope_pair(float& a, float& b, int pair, int pos, int head_dim, double log2_theta) {
  const double freq = exp2(-2.0 * (double)pair / (double)head_dim * log2_theta);
  double ang = (double)pos * freq;
  ang -= 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
  float sn, cs;
  sincosf((float)ang, &sn, &cs);
  const float x = a, y = b;
  a = x * cs - y * sn;
  b = x * sn + y * cs;
}
__device__ __forceinline__ int4 rope_chunk(int4 v, const KvGeom& ge, int chunk, int pos, double log2_theta) {
  if (ge.elem_bytes == 4) {   // 4 fp32 = pairs 2 chunk, 2 chunk + 1
    float f[4] = {__int_as_float(v.x), __int_as_float(v.y), __int_as_float(v.z), __int_as_float(v.w)};
    rope_pair(f[0], f[1], 2 * chunk, pos, ge.head_dim, log2_theta);
    rope_pair(f[2], f[3], 2 * chunk + 1, pos, ge.head_dim, log2_theta);
    return make_int4(__float_as_int(f[0]), __float_as_int(f[1]), __float_as_int(f[2]), __float_as_int(f[3]));
  }
  int w[4] = {v.x, v.y, v.z, v.w};   // 8 bf16 = pairs 4 chunk .. 4 chunk + 3, one pair per word
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = *reinterpret_cast<__nv_bfloat162*>(&w[i]);
    float a = __low2float(h), b = __high2float(h);
    rope_pair(a, b, 4 * chunk + i, pos, ge.head_dim, log2_theta);
    h = __floats2bfloat162_rn(a, b);
    w[i] = *reinterpret_cast<int*>(&h);
  }
  return make_int4(w[0], w[1], w[2], w[3]);
}

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
    int4 val = *reinterpret_cast<const int4*>(src);
    if (p.rope_log2_theta > 0.0 && which == 0) val = rope_chunk(val, ge, chunk, pos, p.rope_log2_theta);
    *reinterpret_cast<int4*>(dst) = val;
  }
}

// Quantised storage (paper, Section 2, "KV Quantization"; the format is described in
// internal.h and in the public header): each head vector of 128 bf16 values is handled by 16
// lanes with 8 values each.  The shared exponent is X = floor(log2(max |x|)) - 8, read off the
// maximum's exponent field; x / 2^X is exact, and the conversion to E4M3 rounds to nearest even
// and saturates at 448, so codes and exponents are a function of exact values.
__global__ void __launch_bounds__(kThreads) append_fp8_kernel(const __grid_constant__ AppendParams p) {
  const AppendEntry& e = p.e[blockIdx.y];
  const KvGeom& ge = p.geom;
  if (blockIdx.x == 0 && threadIdx.x == 0 && e.tbl_idx >= 0) p.table[e.tbl_idx] = e.page_hint;
  const int tok0 = blockIdx.x * kTokensPerBlock;
  if (tok0 >= e.n_new) return;
  const int first_kept = (p.is_ring && e.n_new > p.window) ? e.n_new - p.window : 0;
  const int rows_tok = 2 * ge.n_kv_heads;                 // head vectors per token: K and V
  const int n_tok = min(kTokensPerBlock, e.n_new - tok0);
  const int sub = threadIdx.x & 15;                       // this lane's 8 channels of the vector
  // (the loop bound is uniform over each group of 16 lanes, which shuffle among themselves)
  for (int r = threadIdx.x >> 4; r < n_tok * rows_tok; r += kThreads / 16) {
    const int t = tok0 + r / rows_tok;
    const int rr = r % rows_tok;
    const int which = rr / ge.n_kv_heads;
    const int g = rr - which * ge.n_kv_heads;
    const int pos = e.start_pos + t;
    const char* src = (const char*)(which ? p.v : p.k) +
                      ((int64_t)(e.src_row0 + t) * ge.n_kv_heads + g) * ge.row_bytes + sub * 16;
    int4 val = *reinterpret_cast<const int4*>(src);
    if (p.rope_log2_theta > 0.0 && which == 0) val = rope_chunk(val, ge, sub, pos, p.rope_log2_theta);
    const int w[4] = {val.x, val.y, val.z, val.w};
    float f[8];
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&w[i]);
      f[2 * i] = __low2float(h);
      f[2 * i + 1] = __high2float(h);
      amax = fmaxf(amax, fmaxf(fabsf(f[2 * i]), fabsf(f[2 * i + 1])));
    }
#pragma unroll
    for (int sh = 8; sh >= 1; sh >>= 1)
      amax = fmaxf(amax, __shfl_xor_sync(0xffffu << (threadIdx.x & 16), amax, sh, 16));
    const int ef = (__float_as_int(amax) >> 23) & 0xff;   // amax = 1.m * 2^(ef - 127); ef 0: zero (or below fp32's normals)
    int X = ef == 0 ? -127 : ef - 127 - 8;
    X = max(-127, min(127, X));
    const float inv = __int_as_float((127 - X) << 23);    // 2^-X, exact
    uint32_t lo = 0, hi = 0;                              // 8 codes, channel order
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t two = __nv_cvt_float2_to_fp8x2(make_float2(f[2 * i] * inv, f[2 * i + 1] * inv), __NV_SATFINITE, __NV_E4M3);
      if (i < 2) lo |= two << (16 * i);
      else hi |= two << (16 * (i - 2));
    }
    if (t < first_kept) continue;   // (a ring keeps the last `window` tokens of the call)
    int64_t page;
    int slot;
    if (p.is_ring) {
      const int rs = pos % p.window;
      page = (int64_t)e.seq * p.ring_pages + rs / kPage;
      slot = rs % kPage;
    } else {
      page = e.page_hint >= 0 ? e.page_hint : p.table[(int64_t)e.seq * p.table_stride + pos / kPage];
      slot = pos % kPage;
    }
    if (which == 0) {   // K: two lanes share a 16-byte chunk of the stored row
      char* dst = p.pool + kv_chunk_offset(ge, page, g, 0, slot, sub >> 1) + (sub & 1) * 8;
      *reinterpret_cast<uint2*>(dst) = make_uint2(lo, hi);
    } else {            // V is stored transposed: this token's byte of each channel row
      unsigned char* dst = reinterpret_cast<unsigned char*>(p.pool) + kv_fp8_v_offset(ge, page, g, sub * 8, slot);
#pragma unroll
      for (int i = 0; i < 8; ++i) dst[i * kPage] = (unsigned char)((i < 4 ? lo >> (8 * i) : hi >> (8 * (i - 4))) & 0xffu);
    }
    if (sub == 0) *reinterpret_cast<unsigned char*>(p.pool + kv_exp_offset(ge, page, g, which, slot)) = (unsigned char)(X + 127);
  }
}

__global__ void __launch_bounds__(kThreads) table_set_kernel(const __grid_constant__ TableSetParams p) {
  const int i = blockIdx.x * kThreads + threadIdx.x;
  if (i < p.n) p.table[p.idx[i]] = p.page[i];
}

}  // namespace

cudaError_t launch_table_set(const TableSetParams& p, cudaStream_t st) {
  if (p.n <= 0) return cudaSuccess;
  table_set_kernel<<<(p.n + kThreads - 1) / kThreads, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, int max_n_new, cudaStream_t st) {
  if (p.n_entries <= 0) return cudaSuccess;
  int bx = (max_n_new + kTokensPerBlock - 1) / kTokensPerBlock;
  if (bx < 1) bx = 1;
  dim3 grid(bx, p.n_entries);
  if (p.geom.fp8) append_fp8_kernel<<<grid, kThreads, 0, st>>>(p);
  else append_kernel<<<grid, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace mixattn

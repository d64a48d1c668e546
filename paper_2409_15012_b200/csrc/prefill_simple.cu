// Prompt attention on CUDA cores with exact fp32 arithmetic (fp32 or bf16 tensors).
//
// Paper, Section 3 with the causal order of Section 1: query i attends to keys j <= i
// (standard layer) or i - window < j <= i (sliding window).  This is the fp32-mode
// prefill and the fallback for shapes the tensor-core kernel does not take.  A sequence's
// queries may sit behind `prefix` keys that earlier calls cached: query row r then has
// position prefix + r among the sequence's prefix + S key rows.
// Flash-attention tiling (32 queries x 32 keys per step, online softmax in base 2); key
// tiles outside the band are skipped.
#include <cuda_bf16.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kBM = 32, kBN = 32, kThreads = 128;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) prefill_simple_kernel(const __grid_constant__ PrefillParams p) {
  extern __shared__ float sm[];
  float* Qs = sm;                      // [kBM][D + 1]
  float* Ks = Qs + kBM * (D + 1);      // [kBN][D + 1]
  float* Vs = Ks + kBN * (D + 1);      // [kBN][D]
  float* Ps = Vs + kBN * D;            // [kBM][kBN + 1]

  const int b = blockIdx.z, h = blockIdx.y;
  const int S = p.row0[b + 1] - p.row0[b];
  const int i0 = blockIdx.x * kBM;
  if (i0 >= S) return;
  const int g = h / (p.n_q_heads / p.n_kv_heads);
  const int64_t base = p.row0[b], kbase = p.krow0[b];
  const int P = p.prefix[b];            // key rows before the first query
  const T* q = reinterpret_cast<const T*>(p.q);
  const T* k = reinterpret_cast<const T*>(p.k);
  const T* v = reinterpret_cast<const T*>(p.v);
  const int tid = threadIdx.x, r = tid >> 2, c = tid & 3;

  for (int e = tid; e < kBM * D; e += kThreads) {
    const int rr = e / D, d = e - rr * D;
    Qs[rr * (D + 1) + d] = i0 + rr < S ? to_f32(q[((base + i0 + rr) * p.n_q_heads + h) * D + d]) : 0.f;
  }
  float o[D / 4];
#pragma unroll
  for (int e = 0; e < D / 4; ++e) o[e] = 0.f;
  float m = -INFINITY, l = 0.f;
  const int i = P + i0 + r;  // this thread's query position
  const bool row_ok = i0 + r < S;

  const int n_keys = P + S;
  const int i_last = P + min(S, i0 + kBM) - 1;
  int j_lo = 0;
  if (p.window > 0) j_lo = max(0, P + i0 - p.window + 1) / kBN * kBN;
  for (int j0 = j_lo; j0 <= i_last; j0 += kBN) {
    __syncthreads();
    for (int e = tid; e < kBN * D; e += kThreads) {
      const int jj = e / D, d = e - jj * D;
      const bool in = j0 + jj < n_keys;
      Ks[jj * (D + 1) + d] = in ? to_f32(k[((kbase + j0 + jj) * p.n_kv_heads + g) * D + d]) : 0.f;
      Vs[jj * D + d] = in ? to_f32(v[((kbase + j0 + jj) * p.n_kv_heads + g) * D + d]) : 0.f;
    }
    __syncthreads();
    float s[kBN / 4];
    float mx = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < kBN / 4; ++jj) {
      const int j = j0 + c + 4 * jj;
      float acc = 0.f;
      for (int d = 0; d < D; ++d) acc = fmaf(Qs[r * (D + 1) + d], Ks[(c + 4 * jj) * (D + 1) + d], acc);
      const bool seen = j <= i && row_ok && (p.window == 0 || i - j < p.window);
      s[jj] = seen ? acc * p.scale_log2e : -INFINITY;
      mx = fmaxf(mx, s[jj]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float mn = fmaxf(m, mx);
    // a row that has seen no key yet keeps m = -inf: its weights are 0, not NaN
    const float a = mn == -INFINITY ? 1.f : exp2f(m - mn);
    float sum = 0.f;
#pragma unroll
    for (int jj = 0; jj < kBN / 4; ++jj) {
      const float pe = mn == -INFINITY ? 0.f : exp2f(s[jj] - mn);
      Ps[r * (kBN + 1) + c + 4 * jj] = pe;
      sum += pe;
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    l = l * a + sum;
    m = mn;
    __syncwarp();
#pragma unroll
    for (int e = 0; e < D / 4; ++e) o[e] *= a;
    for (int jj = 0; jj < kBN; ++jj) {
      const float pe = Ps[r * (kBN + 1) + jj];
#pragma unroll
      for (int e = 0; e < D / 4; ++e) o[e] = fmaf(pe, Vs[jj * D + c + 4 * e], o[e]);
    }
  }
  if (row_ok) {
    T* out = reinterpret_cast<T*>(p.out) + ((base + i0 + r) * p.n_q_heads + h) * D;
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < D / 4; ++e) store_out(out + c + 4 * e, o[e] * inv);
  }
}

template <typename T, int D>
cudaError_t launch(const PrefillParams& p, int max_len, cudaStream_t st) {
  const size_t smem = (size_t)(kBM * (D + 1) + kBN * (D + 1) + kBN * D + kBM * (kBN + 1)) * 4;
  cudaError_t e = cudaFuncSetAttribute(prefill_simple_kernel<T, D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((max_len + kBM - 1) / kBM, p.n_q_heads, p.n_seqs);
  prefill_simple_kernel<T, D><<<grid, kThreads, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_simple(const PrefillParams& p, int dtype, int max_len, cudaStream_t st) {
  if (p.n_seqs <= 0 || max_len <= 0) return cudaSuccess;
  if (dtype == MIXATTN_BF16)
    return p.head_dim == 128 ? launch<__nv_bfloat16, 128>(p, max_len, st)
                             : launch<__nv_bfloat16, 64>(p, max_len, st);
  return p.head_dim == 128 ? launch<float, 128>(p, max_len, st) : launch<float, 64>(p, max_len, st);
}

}  // namespace mixattn

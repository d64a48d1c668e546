// Split-KV flash decoding, bf16 cache, fp32 softmax and accumulation (sm_100a).
//
// Paper, Section 3: a decode query attends to all cached keys (standard layer) or to the
// last `window` keys (sliding-window layer); Section 1: the cost is moving the KV cache
// from HBM to shared memory, so this kernel is built around that stream:
//
//   * persistent CTAs (one per SM) walk a static list of work items
//     (sequence, split of its keys, KV head); the GQA query heads of that KV head
//     (up to 16) are the rows of one tensor-core tile, so K/V is read once per group;
//   * one producer warp streams (page, head) blocks -- 16 keys of K and V, contiguous in
//     HBM, already in the swizzled shared-memory image -- with one bulk async copy each
//     into a ring of 64-key stages guarded by full/empty mbarriers; the ring keeps
//     running across work items, so the next item's keys arrive during this item's
//     epilogue;
//   * eight consumer warps, two groups alternating stages, one 16-key page per warp:
//     S = Q K^T and O += P V on mma.sync m16n8k16 (bf16 in, fp32 out), online softmax in
//     base 2 with quad shuffles, private running (max, sum, O) per warp;
//   * per item the warps merge through shared memory and write either the final output
//     (sequence not split) or an unnormalised partial + (max, sum) for the combine pass.
//
// Every mbarrier wait is bounded: on time-out the kernel raises a status word and all
// roles leave.
#include <cuda_bf16.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kGroupWarps = 4;                      // warps (= pages) per stage
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kTileKeys = kGroupWarps * kPage;      // 64 keys per stage
constexpr int kMaxStages = 8;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false after kWaitLimitNs or when another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                        uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                          uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
// (x, y) -> packed bf16 pair `hi` and packed bf16 pair `lo` of the rounding residuals
__device__ __forceinline__ void split_bf16(float x, float y, uint32_t& hi, uint32_t& lo) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  hi = *reinterpret_cast<uint32_t*>(&h);
  lo = pack_bf16(x - __low2float(h), y - __high2float(h));
}
__device__ __forceinline__ void consumer_bar() {  // the 256 consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

struct Item {
  int i;        // sequence index within the call
  int g;        // KV head
  int hc;       // chunk of 16 query heads within the group
  int c;        // split index within the sequence
  int t0, t1;   // keys [t0, t1)
  int n_splits;
};

__device__ __forceinline__ Item decode_item(const DecodeParams& p, int it) {
  Item x;
  x.hc = it % p.head_chunks;
  int r = it / p.head_chunks;
  x.g = r % p.geom.n_kv_heads;
  const int cg = r / p.geom.n_kv_heads;  // global split index
  int lo = 0, hi = p.n_seqs;             // last i with chunk_base[i] <= cg
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.chunk_base[mid] <= cg) lo = mid; else hi = mid;
  }
  x.i = lo;
  x.c = cg - p.chunk_base[lo];
  x.n_splits = p.chunk_base[lo + 1] - p.chunk_base[lo];
  x.t0 = x.c * p.chunk_len[lo];
  x.t1 = min(p.n_eff[lo], x.t0 + p.chunk_len[lo]);
  return x;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
decode_split_bf16_kernel(const __grid_constant__ DecodeParams p, const int n_stages) {
  constexpr int kRowBytes = D * 2;
  constexpr int kBlkBytes = 2 * kPage * kRowBytes;       // K+V of one (page, head)
  constexpr int kStageBytes = kGroupWarps * kBlkBytes;
  constexpr int kKSteps = D / 16;

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stages = smem;
  float* merge = reinterpret_cast<float*>(smem + (size_t)n_stages * kStageBytes);
  const int rows_cap = min(p.group, kMaxGroupRows);
  float* merge_ml = merge + kConsumerWarps * rows_cap * D;            // [warp][row][2]
  uint64_t* bars = reinterpret_cast<uint64_t*>(merge_ml + kConsumerWarps * rows_cap * 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kMaxStages);
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = smem_u32(bars + kMaxStages);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kGroupWarps);
    }
    abort_flag[0] = 0;   // any role gave up
    abort_flag[1] = 0;   // never set: lets the producer's drain wait run to its own limit
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const KvGeom& ge = p.geom;

  if (warp == kConsumerWarps) {
    // ------------------------------ producer ------------------------------
    int K = 0;  // tiles issued by this CTA so far
    bool ok = true;
    for (int it = blockIdx.x; ok && it < p.total_items; it += gridDim.x) {
      const Item x = decode_item(p, it);
      const int seq = p.seq_id[x.i];
      const int32_t* tbl = p.table ? p.table + (int64_t)seq * p.table_stride : nullptr;
      const int64_t ring_page0 = (int64_t)seq * p.ring_pages;
      const int page_lo = x.t0 / kPage;
      const int page_hi = (x.t1 + kPage - 1) / kPage;
      for (int pg = page_lo; pg < page_hi; pg += kGroupWarps, ++K) {
        const int s = K % n_stages;
        if (K >= n_stages) {
          if (!mbar_wait(empty0 + 8 * s, ((K / n_stages) - 1) & 1, abort_flag)) { ok = false; break; }
        }
        const int n_pg = min(kGroupWarps, page_hi - pg);
        if (lane == 0) mbar_arrive_expect_tx(full0 + 8 * s, n_pg * kBlkBytes);
        __syncwarp();
        if (lane < n_pg) {
          const int64_t phys = tbl ? (int64_t)tbl[pg + lane] : ring_page0 + pg + lane;
          const char* src = p.pool + phys * ge.page_bytes + (int64_t)x.g * kBlkBytes;
          bulk_g2s(smem_u32(stages + (size_t)s * kStageBytes + lane * kBlkBytes), src, kBlkBytes,
                   full0 + 8 * s);
        }
      }
    }
    if (!ok && lane == 0) {
      // leave only after the copies already issued have landed (bounded)
      atomicExch(p.status, kDevWaitTimeout);
      for (int back = 1; back <= n_stages && K - back >= 0; ++back) {
        const int Kb = K - back;
        mbar_wait(full0 + 8 * (Kb % n_stages), (Kb / n_stages) & 1, abort_flag + 1);
      }
    }
    return;
  }

  // -------------------------------- consumers --------------------------------
  const int grp = warp / kGroupWarps;   // which stages this warp consumes
  const int wig = warp % kGroupWarps;   // page of the stage
  const int qrow = lane >> 2;           // fragment row (and row + 8)
  const int qcol = (lane & 3) * 2;
  // ldmatrix.x4 lane addressing inside a (page, head) block: lane -> (matrix lm, row lr)
  const int lm = lane >> 3, lr = lane & 7;
  const int k_tok = (lm >> 1) * 8 + lr, k_chk = lm & 1;   // K: (keys 0-7 | 8-15) x (chunk 2ks | 2ks+1)
  const int v_tok = (lm & 1) * 8 + lr, v_chk = lm >> 1;   // V: (keys 0-7 | 8-15) x (chunk 2jj | 2jj+1)

  int K = 0;
  for (int it = blockIdx.x; it < p.total_items; it += gridDim.x) {
    const Item x = decode_item(p, it);
    const int rows = min(kMaxGroupRows, p.group - x.hc * kMaxGroupRows);
    const int h0 = x.g * p.group + x.hc * kMaxGroupRows;

    // Q fragments (A operand), rows = query heads of the group
    uint32_t qa[kKSteps][4];
    {
      const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(p.q) +
                                ((int64_t)x.i * p.n_q_heads + h0) * D;
#pragma unroll
      for (int ks = 0; ks < kKSteps; ++ks) {
        const int d = ks * 16 + qcol;
        qa[ks][0] = qrow < rows ? *reinterpret_cast<const uint32_t*>(qb + qrow * D + d) : 0u;
        qa[ks][1] = qrow + 8 < rows ? *reinterpret_cast<const uint32_t*>(qb + (qrow + 8) * D + d) : 0u;
        qa[ks][2] = qrow < rows ? *reinterpret_cast<const uint32_t*>(qb + qrow * D + d + 8) : 0u;
        qa[ks][3] = qrow + 8 < rows ? *reinterpret_cast<const uint32_t*>(qb + (qrow + 8) * D + d + 8) : 0u;
      }
    }
    float m[2] = {-INFINITY, -INFINITY};
    float l[2] = {0.f, 0.f};
    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

    const int n_tiles = ((x.t1 + kPage - 1) / kPage - x.t0 / kPage + kGroupWarps - 1) / kGroupWarps;
    for (int k = 0; k < n_tiles; ++k) {
      const int Kg = K + k;
      if ((Kg & 1) != grp) continue;
      const int s = Kg % n_stages;
      if (!mbar_wait(full0 + 8 * s, (Kg / n_stages) & 1, abort_flag)) break;  // abort_flag is set
      const int tok_base = x.t0 + k * kTileKeys + wig * kPage;
      if (tok_base < x.t1) {
        const uint32_t kb = smem_u32(stages + (size_t)s * kStageBytes + wig * kBlkBytes);
        const uint32_t vb = kb + kPage * kRowBytes;
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kb + k_tok * kRowBytes + (((2 * ks + k_chk) ^ (k_tok & 7)) << 4), b0, b1, b2, b3);
          mma_bf16(s0, qa[ks], b0, b1);
          mma_bf16(s1, qa[ks], b2, b3);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s0[e] *= p.scale_log2e;
          s1[e] *= p.scale_log2e;
        }
        if (tok_base + kPage > x.t1) {  // ragged end of the split
          const int lim = x.t1 - tok_base;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (qcol + (e & 1) >= lim) s0[e] = -INFINITY;
            if (8 + qcol + (e & 1) >= lim) s1[e] = -INFINITY;
          }
        }
        // online softmax: rows qrow (elements 0,1) and qrow + 8 (elements 2,3)
        float mx0 = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
        float mx1 = fmaxf(fmaxf(s0[2], s0[3]), fmaxf(s1[2], s1[3]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m[0], mx0), mn1 = fmaxf(m[1], mx1);
        const float a0 = exp2f(m[0] - mn0), a1 = exp2f(m[1] - mn1);
        m[0] = mn0;
        m[1] = mn1;
        s0[0] = exp2f(s0[0] - mn0); s0[1] = exp2f(s0[1] - mn0);
        s1[0] = exp2f(s1[0] - mn0); s1[1] = exp2f(s1[1] - mn0);
        s0[2] = exp2f(s0[2] - mn1); s0[3] = exp2f(s0[3] - mn1);
        s1[2] = exp2f(s1[2] - mn1); s1[3] = exp2f(s1[3] - mn1);
        l[0] = l[0] * a0 + (s0[0] + s0[1] + s1[0] + s1[1]);
        l[1] = l[1] * a1 + (s0[2] + s0[3] + s1[2] + s1[3]);
        // P as two bf16 terms (hi + residual): the HBM stream leaves tensor-core time
        // to spare, so P keeps ~16 significant bits instead of 8
        uint32_t pa[4], pr[4];
        split_bf16(s0[0], s0[1], pa[0], pr[0]);
        split_bf16(s0[2], s0[3], pa[1], pr[1]);
        split_bf16(s1[0], s1[1], pa[2], pr[2]);
        split_bf16(s1[2], s1[3], pa[3], pr[3]);
#pragma unroll
        for (int j = 0; j < D / 8; ++j) {
          o[j][0] *= a0; o[j][1] *= a0;
          o[j][2] *= a1; o[j][3] *= a1;
        }
#pragma unroll
        for (int jj = 0; jj < D / 16; ++jj) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(vb + v_tok * kRowBytes + (((2 * jj + v_chk) ^ (v_tok & 7)) << 4), b0, b1, b2, b3);
          mma_bf16(o[2 * jj], pa, b0, b1);
          mma_bf16(o[2 * jj + 1], pa, b2, b3);
          mma_bf16(o[2 * jj], pr, b0, b1);
          mma_bf16(o[2 * jj + 1], pr, b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
    K += n_tiles;

    // ---- merge the eight warps' (max, sum, O) and write the item's result ----
    l[0] += __shfl_xor_sync(0xffffffffu, l[0], 1);
    l[0] += __shfl_xor_sync(0xffffffffu, l[0], 2);
    l[1] += __shfl_xor_sync(0xffffffffu, l[1], 1);
    l[1] += __shfl_xor_sync(0xffffffffu, l[1], 2);
    float* mo = merge + (size_t)warp * rows_cap * D;
    float* mml = merge_ml + (size_t)warp * rows_cap * 2;
    if (qrow < rows) {
#pragma unroll
      for (int j = 0; j < D / 8; ++j)
        *reinterpret_cast<float2*>(mo + qrow * D + j * 8 + qcol) = make_float2(o[j][0], o[j][1]);
      if ((lane & 3) == 0) { mml[qrow * 2] = m[0]; mml[qrow * 2 + 1] = l[0]; }
    }
    if (qrow + 8 < rows) {
#pragma unroll
      for (int j = 0; j < D / 8; ++j)
        *reinterpret_cast<float2*>(mo + (qrow + 8) * D + j * 8 + qcol) = make_float2(o[j][2], o[j][3]);
      if ((lane & 3) == 0) { mml[(qrow + 8) * 2] = m[1]; mml[(qrow + 8) * 2 + 1] = l[1]; }
    }
    consumer_bar();
    if (*abort_flag) {  // uniform: set before the barrier by whichever role gave up
      if (threadIdx.x == 0) atomicExch(p.status, kDevWaitTimeout);
      return;
    }
    for (int e = threadIdx.x; e < rows * D; e += kConsumerWarps * 32) {
      const int r = e / D, d = e - r * D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, merge_ml[(w * rows_cap + r) * 2]);
      float L = 0.f, acc = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float sc = exp2f(merge_ml[(w * rows_cap + r) * 2] - M);
        L += merge_ml[(w * rows_cap + r) * 2 + 1] * sc;
        acc += merge[((size_t)w * rows_cap + r) * D + d] * sc;
      }
      const int h = h0 + r;
      if (x.n_splits == 1) {
        reinterpret_cast<__nv_bfloat16*>(p.out)[((int64_t)x.i * p.n_q_heads + h) * D + d] =
            __float2bfloat16_rn(acc / L);
      } else {
        const int64_t slot = (int64_t)(p.chunk_base[x.i] + x.c) * p.n_q_heads + h;
        p.part_o[slot * D + d] = acc;
        if (d == 0) p.part_ml[slot] = make_float2(M, L);
      }
    }
    consumer_bar();
  }
}

size_t smem_bytes(int D, int group, int n_stages) {
  const int rows_cap = group < kMaxGroupRows ? group : kMaxGroupRows;
  size_t stage = (size_t)kGroupWarps * 2 * kPage * D * 2;
  return n_stages * stage + (size_t)kConsumerWarps * rows_cap * (D + 2) * 4 + 2 * kMaxStages * 8 + 16;
}

}  // namespace

cudaError_t prepare_decode_bf16() {
  cudaError_t e = cudaFuncSetAttribute(decode_split_bf16_kernel<128>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(decode_split_bf16_kernel<64>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_decode_split_bf16(const DecodeParams& p, int sm_count, cudaStream_t st) {
  const int D = p.geom.head_dim;
  int n_stages = kMaxStages;
  while (n_stages > 2 && smem_bytes(D, p.group, n_stages) > 220 * 1024) --n_stages;
  const size_t smem = smem_bytes(D, p.group, n_stages);
  const int grid = p.total_items < sm_count ? p.total_items : sm_count;
  if (grid <= 0) return cudaSuccess;
  if (D == 128)
    decode_split_bf16_kernel<128><<<grid, kThreads, smem, st>>>(p, n_stages);
  else
    decode_split_bf16_kernel<64><<<grid, kThreads, smem, st>>>(p, n_stages);
  return cudaGetLastError();
}

}  // namespace mixattn

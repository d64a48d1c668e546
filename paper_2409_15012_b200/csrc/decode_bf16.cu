// Split-KV flash decoding, bf16 cache, fp32 softmax and accumulation (sm_100a).
//
// Paper, Section 3: a decode query attends to all cached keys (standard layer) or to the
// last `window` keys (sliding-window layer); Section 1: the cost is moving the KV cache
// from HBM to shared memory, so this kernel is built around that stream:
//
//   * persistent CTAs (one per SM) walk a static list of work items
//     (sequence, split of its keys, KV head); the GQA query heads of that KV head
//     (up to 16) are the rows of one tensor-core tile, so K/V is read once per group;
//   * producer warps stream (page, head) blocks -- 16 keys of K and V, contiguous in
//     HBM, already in the swizzled shared-memory image -- with one bulk async copy each
//     into a ring of 64-key stages guarded by full/empty mbarriers; the ring keeps
//     running across work items, so the next item's keys arrive during this item's
//     epilogue.  One producer warp needs about 850 cycles per stage (four copy issues, two
//     barrier operations, the table lookup): enough for 32 KB stages, but the 16 KB stages
//     of the quantised cache are streamed by four producer warps that take the stages in
//     turn;
//   * eight consumer warps, two groups alternating stages, one 16-key page per warp:
//     S^T = K Q^T and O^T += V^T P^T on mma.sync m16n8k16 (bf16 in, fp32 out) with the
//     keys as the M dimension and the heads as N = 8, online softmax in base 2, private
//     running (max, sum, O) per warp;
//   * per item the warps merge through shared memory and write either the final output
//     (sequence not split) or an unnormalised partial + (max, sum) for the combine pass.
//     (Combining inside this kernel -- last split to finish, ticket counter -- was
//     measured slower: the fence before the ticket stalls the consumers per item.)
//   * a launch with at most one item per two SMs gives each item a cluster of two CTAs,
//     which stream halves of its keys and merge through distributed shared memory: one
//     CTA ingests K/V at a bounded rate, so idle SMs are better used than a second launch.
//
// Quantised cache (paper, Section 2, "KV Quantization"; KV8 instantiations): a (page, head)
// block holds FP8 E4M3 elements and one shared power-of-two exponent per head vector, half
// the bytes per key, so the arithmetic per byte doubles and the instruction count per page is
// what has to stay small.  The same stream and tile shapes; the elements are widened exactly
// to fp16 right after ldmatrix (two conversions per 32-bit fragment register, nothing else)
// and the products run on the fp16 tensor-core path.  A fragment register holds four
// consecutive bytes: four channels of a key for K, four keys of a channel for V, which is
// stored transposed.  Q is therefore loaded in the matching channel order, and the 16 keys of
// a page take the tile rows in the order 0 1 4 5 8 9 12 13 | 2 3 6 7 10 11 14 15, which is
// the key order the transposed weights then have in the second product.  A K row's exponent
// multiplies its scores; a V row's exponent is folded into its weight.
//
// Every mbarrier wait is bounded: on time-out the kernel raises a status word and all
// roles leave.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kGroupWarps = 4;                      // warps (= pages) per stage
constexpr int kTileKeys = kGroupWarps * kPage;      // 64 keys per stage
constexpr int kMaxStages = 12;
constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds of SM clock

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
// Bounded wait.  Returns false after kWaitLimitCycles or when another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();   // (the SM clock is cheap to read; the global timer is not)
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                         uint64_t l2_policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(l2_policy)
      : "memory");
}
// L2 eviction policy of a launch's K/V stream.  A ring shared by several layers is read again
// by the next launch, but a plain LRU keeps nothing of a cyclic scan larger than the cache: the
// leading part of the ring storage (as much as fits the L2) is cached normally and the rest,
// like a paged cache that is read once per step, is marked evict-first so that it passes through.
__device__ __forceinline__ uint64_t l2_policy_of(const char* pool, uint32_t keep_bytes, uint32_t pool_bytes) {
  uint64_t pol;
  if (keep_bytes > 0)
    asm volatile("createpolicy.range.global.L2::evict_normal.L2::evict_first.b64 %0, [%1], %2, %3;"
                 : "=l"(pol) : "l"(pool), "r"(keep_bytes), "r"(pool_bytes));
  else
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
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
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// four E4M3 codes -> two packed fp16 pairs (bytes 0, 1 and bytes 2, 3), exact
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t x, uint32_t& lo, uint32_t& hi) {
  asm("{\n\t.reg .b16 l, h;\n\t"
      "mov.b32 {l, h}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, l;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, h;\n\t}"
      : "=r"(lo), "=r"(hi) : "r"(x));
}
__device__ __forceinline__ float ex2_ftz(float x) {   // 2^x, one MUFU op; 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  const __half2 t = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}
// 2^X from the stored exponent byte X + 127.  Byte 0 (X = -127: a zero vector, or one whose
// largest element is below 2^-118) reads as 0 instead of 2^-127.
__device__ __forceinline__ float exp_byte_to_float(uint32_t b) { return __int_as_float((int)(b << 23)); }
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
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {  // transpose an 8x8 b16 fragment
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
// distributed shared memory: the address of the same variable in the first CTA of the cluster
__device__ __forceinline__ uint32_t map_to_cta0(uint32_t local) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(remote) : "r"(local));
  return remote;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// all threads of the cluster that have not exited (the producer warps exit on their own)
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
template <int NCW>
__device__ __forceinline__ void consumer_bar() {  // the consumer threads only
  asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
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
  // last i with chunk_base[i] <= cg: proportional guess, then a short walk (batches of equal
  // lengths hit at once; each probe is a dependent parameter load, so few probes matter)
  int lo = (int)(((long long)cg * p.n_seqs) / p.chunk_base[p.n_seqs]);
  while (p.chunk_base[lo] > cg) --lo;
  while (p.chunk_base[lo + 1] <= cg) ++lo;
  x.i = lo;
  x.c = cg - p.chunk_base[lo];
  x.n_splits = p.chunk_base[lo + 1] - p.chunk_base[lo];
  x.t0 = x.c * p.chunk_len[lo];
  x.t1 = min(p.n_eff[lo], x.t0 + p.chunk_len[lo]);
  return x;
}

// The part of an item's keys that CTA `crank` of a two-CTA cluster takes: whole stages of
// kTileKeys keys, the first CTA the larger half (never empty); the second may get none.
__device__ __forceinline__ void cluster_share(Item& x, int crank) {
  const int tiles = (x.t1 - x.t0 + kTileKeys - 1) / kTileKeys;   // x.t0 is a multiple of the page size
  const int mid = min(x.t1, x.t0 + ((tiles + 1) / 2) * kTileKeys);
  if (crank == 0) x.t1 = mid;
  else if (mid < x.t1) x.t0 = mid;
  else x.t0 = x.t1 = 0;   // nothing left for the second CTA: no stage is streamed
}

// NCW consumer warps: 8 (two groups alternating stages; one CTA per SM with a deep ring, for
// long key streams) or 4 (one group; two CTAs per SM with short rings, so that a launch with
// few, short work items keeps every item in flight at once instead of queueing two per SM).
// CL = 2: a launch of few items runs each item on a thread-block cluster of two CTAs (two SMs),
// which take halves of the item's keys and merge through distributed shared memory: one CTA
// ingests K/V at a fixed rate, so a short launch that leaves SMs idle is halved this way
// without a second launch.  The grid then holds exactly one cluster per item.
// KV8 = 1: the cache holds FP8 E4M3 rows with shared exponents (see the top of the file).
// Producer warps of a variant.  With more than one, the ring length must be a multiple of their
// number (checked by the launcher): a stage then always belongs to the same producer, whose
// program order keeps its waits on that stage's barriers one phase apart.  (A producer that
// waited for a phase two ahead of the barrier's would be answered "complete" by the parity test.)
__host__ __device__ constexpr int producer_warps(int ncw, int kv8) { return (kv8 && ncw == 8) ? 4 : 1; }

template <int D, int NCW, int CL, int KV8>
__global__ void __launch_bounds__((NCW + producer_warps(NCW, KV8)) * 32, NCW == 4 ? 2 : 1)
decode_split_bf16_kernel(const __grid_constant__ DecodeParams p, const int n_stages) {
  constexpr int kConsumerWarps = NCW;
  constexpr int kProducerWarps = producer_warps(NCW, KV8);
  constexpr int kGroups = NCW / kGroupWarps;
  constexpr int kRowBytes = KV8 ? D : D * 2;
  constexpr int kBlkBytes = 2 * kPage * kRowBytes + (KV8 ? 2 * kPage : 0);   // K+V (+ exponents) of one (page, head)
  constexpr int kStageBytes = kGroupWarps * kBlkBytes;
  constexpr int kKSteps = D / 16;

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stages = smem;
  float* merge = reinterpret_cast<float*>(smem + (size_t)n_stages * kStageBytes);
  const int rows_cap = min(p.group, kMaxGroupRows);
  float* merge_ml = merge + kConsumerWarps * rows_cap * D;            // [warp][row][2]
  uint64_t* bars = reinterpret_cast<uint64_t*>(merge_ml + kConsumerWarps * rows_cap * 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kMaxStages);
  // cluster exchange (CL > 1), in the first CTA of the cluster: [CTA][row][D] partial O, then [CTA][row] (max, sum)
  float* xch = reinterpret_cast<float*>(bars + 2 * kMaxStages + 2);
  int crank = 0;
  if constexpr (CL > 1) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
  const int item0 = CL > 1 ? (int)blockIdx.x / CL : (int)blockIdx.x;
  const int item_stride = CL > 1 ? (int)gridDim.x / CL : (int)gridDim.x;
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = smem_u32(bars + kMaxStages);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // Programmatic dependent launch: let the next kernel of the stream begin its launch and
  // set-up as soon as every CTA of this one is running ...
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
  // every thread of the cluster checks in once; the consumers wait for this phase before their
  // first access to the other CTA's shared memory, which must be running by then
  if constexpr (CL > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  // ... and do not touch global memory before the kernels ahead in the stream have
  // completed and flushed (a no-op when this kernel was launched the ordinary way)
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const KvGeom& ge = p.geom;

  if (warp >= kConsumerWarps) {
    // ------------------------------ producers ------------------------------
    // every producer warp walks the whole tile sequence and issues the tiles K with
    // K % kProducerWarps == pw
    const int pw = warp - kConsumerWarps;
    int K = 0;  // tiles of this CTA so far (all producers)
    // stage of this producer's next tile and how often it has been round the ring (kept by
    // addition: the ring length is a run-time value, and a division per stage sits on the
    // issue path)
    int ps = pw, pround = 0;
    bool ok = true;
    const uint64_t l2_policy = l2_policy_of(p.pool, p.l2_keep_bytes, p.l2_pool_bytes);
    for (int it = item0; ok && it < p.total_items; it += item_stride) {
      Item x = decode_item(p, it);
      if constexpr (CL > 1) cluster_share(x, crank);
      const int seq = p.seq_id[x.i];
      const int32_t* tbl = p.table ? p.table + (int64_t)seq * p.table_stride : nullptr;
      const int64_t ring_page0 = (int64_t)seq * p.ring_pages;
      const int page_lo = x.t0 / kPage;
      const int page_hi = (x.t1 + kPage - 1) / kPage;
      // page ids are fetched 32 at a time (one per lane), one batch ahead of their use,
      // so the table lookup is off the issue path of the copies
      int ids_next = 0;
      if (tbl && page_lo + lane < page_hi) ids_next = tbl[page_lo + lane];
      int ids = 0;
      for (int pg = page_lo; pg < page_hi; pg += kGroupWarps, ++K) {
        const int rel = pg - page_lo;
        if ((rel & 31) == 0) {
          ids = ids_next;
          if (tbl && pg + 32 + lane < page_hi) ids_next = tbl[pg + 32 + lane];
        }
        if (kProducerWarps > 1 && K % kProducerWarps != pw) continue;
        const int s = ps;
        if (pround > 0) {  // lane 0 waits; the verdict is made warp-uniform
          int w = 1;
          if (lane == 0) w = mbar_wait(empty0 + 8 * s, (pround - 1) & 1, abort_flag);
          if (!__shfl_sync(0xffffffffu, w, 0)) { ok = false; break; }
        }
        ps += kProducerWarps;
        if (ps >= n_stages) { ps -= n_stages; ++pround; }
        const int n_pg = min(kGroupWarps, page_hi - pg);
        if (lane == 0) mbar_arrive_expect_tx(full0 + 8 * s, n_pg * kBlkBytes);
        const int my_id = __shfl_sync(0xffffffffu, ids, (rel & 31) + (lane & (kGroupWarps - 1)));
        if (lane < n_pg) {
          const int64_t phys = tbl ? (int64_t)my_id : ring_page0 + pg + lane;
          const char* src = p.pool + phys * ge.page_bytes + (int64_t)x.g * kBlkBytes;
          bulk_g2s(smem_u32(stages + (size_t)s * kStageBytes + lane * kBlkBytes), src, kBlkBytes,
                   full0 + 8 * s, l2_policy);
        }
      }
    }
    if (!ok && lane == 0) {
      // leave only after the copies already issued have landed (bounded)
      atomicExch(p.status, kDevWaitTimeout);
      for (int back = 1; back <= n_stages && K - back >= 0; ++back) {
        const int Kb = K - back;
        if (Kb % kProducerWarps == pw) mbar_wait(full0 + 8 * (Kb % n_stages), (Kb / n_stages) & 1, abort_flag + 1);
      }
    }
    if constexpr (CL > 1) {
      // the producer takes no part in the merge, but the consumers' cluster barrier counts every
      // thread: check in for it before leaving (after the start-up phase, which is complete as soon
      // as both CTAs run)
      __syncwarp();
      asm volatile("barrier.cluster.wait.acquire.aligned;\n\tbarrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    return;
  }

  // -------------------------------- consumers --------------------------------
  // Transposed formulation: keys are the M dimension, the (up to 8) query heads of the
  // group the N dimension.  S^T = K Q^T (one m16n8 tile per 16 keys), P^T is transposed
  // in registers (movmatrix) into the B operand of O^T += V^T P^T.  Each thread owns two
  // heads (columns 2*(lane&3), +1) of every accumulator, so the online-softmax state is
  // thread-local apart from the column max / sum over the eight row groups.
  const int grp = warp / kGroupWarps;   // which stages this warp consumes
  const int wig = warp % kGroupWarps;   // page of the stage
  const int frow = lane >> 2;           // fragment row (and row + 8)
  const int fcol = (lane & 3) * 2;      // fragment column pair = the two heads of this thread
  // ldmatrix.x4 lane addressing inside a (page, head) block: lane -> (matrix lm, row lr)
  const int lm = lane >> 3, lr = lane & 7;
  const int k_tok = (lm & 1) * 8 + lr, k_chk = lm >> 1;   // K as A: (keys 0-7|8-15) x (chunk 2ks|2ks+1)
  const int v_tok = (lm >> 1) * 8 + lr, v_chk = lm & 1;   // V^T as A (.trans): (chunk 2jt|2jt+1) x (keys 0-7|8-15)
  // quantised cache: tile row r of a page is key 4 (r >> 1) + (r & 1) for r < 8 and that + 2 for r - 8
  const int k8_tok = 4 * (lr >> 1) + (lr & 1) + 2 * (lm & 1);   // key whose K row this lane addresses
  const int key0 = 4 * (frow >> 1) + (frow & 1);                // this thread's score rows: keys key0 and key0 + 2

  int K = 0;
  int cs = grp, cround = 0;   // stage of this group's next tile, passes over the ring (see the producers)
  for (int it = item0; it < p.total_items; it += item_stride) {
    Item x = decode_item(p, it);
    if constexpr (CL > 1) cluster_share(x, crank);
    const int rows = min(kMaxGroupRows, p.group - x.hc * kMaxGroupRows);
    const int h0 = x.g * p.group + x.hc * kMaxGroupRows;

    // Q^T fragments (B operand): thread holds head (lane >> 2), channels 16 ks + fcol (+8)
    uint32_t qb[kKSteps][2];
    if constexpr (!KV8) {
      const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q) +
                                ((int64_t)x.i * p.n_q_heads + h0 + frow) * D + fcol;
#pragma unroll
      for (int ks = 0; ks < kKSteps; ++ks) {
        qb[ks][0] = frow < rows ? *reinterpret_cast<const uint32_t*>(qp + ks * 16) : 0u;
        qb[ks][1] = frow < rows ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8) : 0u;
      }
    } else {
      // A K fragment register holds four consecutive channels of a key (two go to the k index
      // pair 2t, 2t+1 and two to 2t+8, 2t+9), so this thread's Q values of a 16-channel step
      // are the four channels 4t .. 4t+3, as fp16
      const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q) +
                                ((int64_t)x.i * p.n_q_heads + h0 + frow) * D + 2 * fcol;
#pragma unroll
      for (int ks = 0; ks < kKSteps; ++ks) {
        uint2 w = make_uint2(0u, 0u);
        if (frow < rows) w = *reinterpret_cast<const uint2*>(qp + ks * 16);
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&w.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
        qb[ks][0] = pack_f16(__low2float(a), __high2float(a));
        qb[ks][1] = pack_f16(__low2float(b), __high2float(b));
      }
    }
    float m[2] = {-INFINITY, -INFINITY};
    float l[2] = {0.f, 0.f};
    float o[D / 16][4];   // O^T: rows = channels 16 jt + frow (+8), cols = the thread's two heads
#pragma unroll
    for (int j = 0; j < D / 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

    const int n_tiles = ((x.t1 + kPage - 1) / kPage - x.t0 / kPage + kGroupWarps - 1) / kGroupWarps;
    // this group's tiles of the item: every kGroups-th, starting where the count left off
    for (int k = (grp + kGroups - K % kGroups) % kGroups; k < n_tiles; k += kGroups) {
      const int s = cs;
      // every lane waits (each needs to observe the copy), the verdict is warp-uniform
      if (!__all_sync(0xffffffffu, mbar_wait(full0 + 8 * s, cround & 1, abort_flag))) break;
      cs += kGroups;
      if (cs >= n_stages) { cs -= n_stages; ++cround; }
      const int tok_base = x.t0 + k * kTileKeys + wig * kPage;
      if (tok_base < x.t1) {
        const uint32_t kb = smem_u32(stages + (size_t)s * kStageBytes + wig * kBlkBytes);
        const uint32_t vb = kb + kPage * kRowBytes;
        float st[4] = {0.f, 0.f, 0.f, 0.f}, st2[4] = {0.f, 0.f, 0.f, 0.f};  // two chains: shorter latency
        float vscale0 = 1.f, vscale1 = 1.f;   // quantised cache: 2^X of the V rows of keys frow, frow + 8
        if constexpr (!KV8) {
#pragma unroll
          for (int ks = 0; ks < kKSteps; ks += 2) {
            uint32_t a[4], b[4];
            ldsm_x4(kb + k_tok * kRowBytes + (((2 * ks + k_chk) ^ (k_tok & 7)) << 4), a[0], a[1], a[2], a[3]);
            ldsm_x4(kb + k_tok * kRowBytes + (((2 * ks + 2 + k_chk) ^ (k_tok & 7)) << 4), b[0], b[1], b[2], b[3]);
            mma_bf16(st, a, qb[ks][0], qb[ks][1]);
            mma_bf16(st2, b, qb[ks + 1][0], qb[ks + 1][1]);
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) st[e] = (st[e] + st2[e]) * p.scale_log2e;
        } else {
          // one ldmatrix.x4 = (tile rows 0-7 | 8-15) x (16-byte chunk 2j | 2j+1) = two 16-channel steps
#pragma unroll
          for (int j = 0; j < kKSteps / 2; ++j) {
            uint32_t r[4], a[4], b[4];
            ldsm_x4(kb + k8_tok * kRowBytes + (((2 * j + k_chk) ^ fp8_k_swizzle(k8_tok)) << 4), r[0], r[1], r[2], r[3]);
            e4m3x4_to_f16x2x2(r[0], a[0], a[2]);
            e4m3x4_to_f16x2x2(r[1], a[1], a[3]);
            e4m3x4_to_f16x2x2(r[2], b[0], b[2]);
            e4m3x4_to_f16x2x2(r[3], b[1], b[3]);
            mma_f16(st, a, qb[2 * j][0], qb[2 * j][1]);
            mma_f16(st2, b, qb[2 * j + 1][0], qb[2 * j + 1][1]);
          }
          // the shared exponents of the page's rows sit behind its K and V elements
          const unsigned char* xs = stages + (size_t)s * kStageBytes + wig * kBlkBytes + 2 * kPage * kRowBytes;
          const float ks0 = exp_byte_to_float(xs[key0]) * p.scale_log2e;
          const float ks1 = exp_byte_to_float(xs[key0 + 2]) * p.scale_log2e;
          vscale0 = exp_byte_to_float(xs[kPage + key0]);
          vscale1 = exp_byte_to_float(xs[kPage + key0 + 2]);
          st[0] = (st[0] + st2[0]) * ks0; st[1] = (st[1] + st2[1]) * ks0;
          st[2] = (st[2] + st2[2]) * ks1; st[3] = (st[3] + st2[3]) * ks1;
        }
        if (tok_base + kPage > x.t1) {  // ragged end of the split: this thread's two keys (tile rows frow, frow + 8)
          const int lim = x.t1 - tok_base;
          if ((KV8 ? key0 : frow) >= lim) st[0] = st[1] = -INFINITY;
          if ((KV8 ? key0 + 2 : frow + 8) >= lim) st[2] = st[3] = -INFINITY;
        }
        // column (head) max over the 16 keys: two rows here, eight row groups across lanes
        float mx0 = fmaxf(st[0], st[2]), mx1 = fmaxf(st[1], st[3]);
#pragma unroll
        for (int sh = 4; sh < 32; sh <<= 1) {
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
        }
        const float mn0 = fmaxf(m[0], mx0), mn1 = fmaxf(m[1], mx1);
        float a0, a1;
        if constexpr (!KV8) {
          a0 = exp2f(m[0] - mn0); a1 = exp2f(m[1] - mn1);
          st[0] = exp2f(st[0] - mn0); st[1] = exp2f(st[1] - mn1);
          st[2] = exp2f(st[2] - mn0); st[3] = exp2f(st[3] - mn1);
        } else {   // (arguments are <= 0: a single MUFU op each, tiny results flushed to zero)
          a0 = ex2_ftz(m[0] - mn0); a1 = ex2_ftz(m[1] - mn1);
          st[0] = ex2_ftz(st[0] - mn0); st[1] = ex2_ftz(st[1] - mn1);
          st[2] = ex2_ftz(st[2] - mn0); st[3] = ex2_ftz(st[3] - mn1);
        }
        m[0] = mn0;
        m[1] = mn1;
        l[0] = l[0] * a0 + (st[0] + st[2]);
        l[1] = l[1] * a1 + (st[1] + st[3]);
        // P^T as two bf16 terms (value + rounding residual): the stream leaves tensor
        // time to spare, so P keeps ~16 significant bits; then transpose 8x8 blocks so
        // that keys become the k index of the B operand
        if constexpr (!KV8) {
          uint32_t ph0, pl0, ph1, pl1;
          split_bf16(st[0], st[1], ph0, pl0);   // keys 0-7
          split_bf16(st[2], st[3], ph1, pl1);   // keys 8-15
          ph0 = movmatrix_t(ph0); ph1 = movmatrix_t(ph1);
          pl0 = movmatrix_t(pl0); pl1 = movmatrix_t(pl1);
          uint32_t va[D / 16][4];
#pragma unroll
          for (int jt = 0; jt < D / 16; ++jt) {
            ldsm_x4_t(vb + v_tok * kRowBytes + (((2 * jt + v_chk) ^ (v_tok & 7)) << 4), va[jt][0], va[jt][1],
                      va[jt][2], va[jt][3]);
            o[jt][0] *= a0; o[jt][1] *= a1;
            o[jt][2] *= a0; o[jt][3] *= a1;
          }
#pragma unroll
          for (int jt = 0; jt < D / 16; ++jt) mma_bf16(o[jt], va[jt], ph0, ph1);
#pragma unroll
          for (int jt = 0; jt < D / 16; ++jt) mma_bf16(o[jt], va[jt], pl0, pl1);
        } else {
          // P^T as one fp16 term (11 significant bits against the 4 of the stored V), each
          // weight already multiplied by its V row's 2^X
          const uint32_t ph0 = movmatrix_t(pack_f16(st[0] * vscale0, st[1] * vscale0));   // tile rows 0-7
          const uint32_t ph1 = movmatrix_t(pack_f16(st[2] * vscale1, st[3] * vscale1));   // tile rows 8-15
          // once the running maxima have settled, most pages leave them alone (a0 = a1 = 1)
          if (__any_sync(0xffffffffu, a0 != 1.f || a1 != 1.f)) {
#pragma unroll
            for (int jt = 0; jt < D / 16; ++jt) {
              o[jt][0] *= a0; o[jt][1] *= a1;
              o[jt][2] *= a0; o[jt][3] *= a1;
            }
          }
          // V^T rows are channels, 16 key bytes each: one ldmatrix.x4 = 32 channels; a register
          // holds keys 4t .. 4t+3 of a channel, which are the contraction indices 2t, 2t+1 and
          // 2t+8, 2t+9 in the key order of the tile rows above
#pragma unroll
          for (int j = 0; j < D / 32; ++j) {
            uint32_t r[4], a[4], b[4];
            ldsm_x4(vb + (32 * j + lane) * kPage, r[0], r[1], r[2], r[3]);
            e4m3x4_to_f16x2x2(r[0], a[0], a[2]);
            e4m3x4_to_f16x2x2(r[1], a[1], a[3]);
            e4m3x4_to_f16x2x2(r[2], b[0], b[2]);
            e4m3x4_to_f16x2x2(r[3], b[1], b[3]);
            mma_f16(o[2 * j], a, ph0, ph1);
            mma_f16(o[2 * j + 1], b, ph0, ph1);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
    K += n_tiles;

    // ---- merge the eight warps' (max, sum, O) and write the item's result ----
#pragma unroll
    for (int sh = 4; sh < 32; sh <<= 1) {
      l[0] += __shfl_xor_sync(0xffffffffu, l[0], sh);
      l[1] += __shfl_xor_sync(0xffffffffu, l[1], sh);
    }
    float* mo = merge + (size_t)warp * rows_cap * D;
    float* mml = merge_ml + (size_t)warp * rows_cap * 2;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int r = fcol + e;
      if (r < rows) {
#pragma unroll
        for (int jt = 0; jt < D / 16; ++jt) {
          mo[r * D + jt * 16 + frow] = o[jt][e];
          mo[r * D + jt * 16 + frow + 8] = o[jt][2 + e];
        }
        if (frow == 0) { mml[r * 2] = m[e]; mml[r * 2 + 1] = l[e]; }
      }
    }
    consumer_bar<NCW>();
    const bool gave_up = *abort_flag != 0;  // uniform: set before the barrier by whichever role gave up
    if (gave_up && threadIdx.x == 0) atomicExch(p.status, kDevWaitTimeout);
    if (CL == 1 && gave_up) return;
    // (in a cluster every consumer thread goes on to the cluster barrier below, which has no
    // time-out of its own: the other CTA's threads reach it after at most their own bounded waits)
    if constexpr (CL > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    float* xo = xch;                                   // [CL][rows_cap][D]
    float* xml = xch + CL * rows_cap * D;              // [CL][rows_cap][2]
    for (int e = threadIdx.x; e < rows * D && !gave_up; e += kConsumerWarps * 32) {
      const int r = e / D, d = e - r * D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, merge_ml[(w * rows_cap + r) * 2]);
      float L = 0.f, acc = 0.f;
      if (M > -INFINITY) {   // (a CTA of a cluster may have had no key at all)
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
          const float sc = exp2f(merge_ml[(w * rows_cap + r) * 2] - M);
          L += merge_ml[(w * rows_cap + r) * 2 + 1] * sc;
          acc += merge[((size_t)w * rows_cap + r) * D + d] * sc;
        }
      }
      if constexpr (CL > 1) {
        // hand (M, L, acc) to the first CTA of the cluster through its shared memory
        st_cluster_f32(map_to_cta0(smem_u32(xo + ((size_t)crank * rows_cap + r) * D + d)), acc);
        if (d == 0) {
          st_cluster_f32(map_to_cta0(smem_u32(xml + ((size_t)crank * rows_cap + r) * 2)), M);
          st_cluster_f32(map_to_cta0(smem_u32(xml + ((size_t)crank * rows_cap + r) * 2 + 1)), L);
        }
        continue;
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
    if constexpr (CL > 1) {
      cluster_sync_all();   // both CTAs' partials are in the first CTA's shared memory
      if (gave_up) return;
      if (crank == 0) {
        for (int e = threadIdx.x; e < rows * D; e += kConsumerWarps * 32) {
          const int r = e / D, d = e - r * D;
          const float M0 = xml[r * 2], M1 = xml[(rows_cap + r) * 2];
          const float M = fmaxf(M0, M1);
          const float s0 = exp2f(M0 - M), s1 = exp2f(M1 - M);   // 2^-inf = 0 for a CTA without keys
          const float L = xml[r * 2 + 1] * s0 + xml[(rows_cap + r) * 2 + 1] * s1;
          const float acc = xo[(size_t)r * D + d] * s0 + xo[((size_t)rows_cap + r) * D + d] * s1;
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
      }
    }
    consumer_bar<NCW>();
  }
}

size_t smem_bytes(int D, int group, int n_stages, int ncw, int cl, int kv8) {
  const int rows_cap = group < kMaxGroupRows ? group : kMaxGroupRows;
  size_t stage = (size_t)kGroupWarps * (kv8 ? 2 * kPage * D + 2 * kPage : 2 * kPage * D * 2);
  const size_t exchange = cl > 1 ? (size_t)cl * rows_cap * (D + 2) * 4 : 0;
  return n_stages * stage + (size_t)ncw * rows_cap * (D + 2) * 4 + 2 * kMaxStages * 8 + 32 + exchange;
}

}  // namespace

cudaError_t prepare_decode_bf16() {
  cudaError_t e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 8, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<64, 8, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 4, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<64, 4, 1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 8, 2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<64, 8, 2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  // quantised cache: head_dim 128 only
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 8, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 4, 1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_split_bf16_kernel<128, 8, 2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  return e;
}

cudaError_t launch_decode_split_bf16(const DecodeParams& p, int sm_count, cudaStream_t st) {
  const int D = p.geom.head_dim;
  if (p.total_items <= 0) return cudaSuccess;
  // Few, short items (more than one but at most two per SM, e.g. one 1024-key window per
  // (sequence, KV head)): two small CTAs per SM keep all of them streaming at once, and the
  // launch is bound by HBM instead of by the SM that drew two items.
  int64_t max_keys = 0;
  for (int i = 0; i < p.n_seqs; ++i) max_keys = p.chunk_len[i] > max_keys ? p.chunk_len[i] : max_keys;
  const bool small = p.total_items > sm_count && p.total_items <= 2 * sm_count && max_keys <= 2048;
  // At most one item per two SMs, and items of several stages: a cluster of two CTAs per item.
  const bool paired = 2 * p.total_items <= sm_count && max_keys >= 4 * kTileKeys;
  const int cl = paired ? 2 : 1;
  const int kv8 = p.geom.fp8;
  const int ncw = small ? 4 : 8;
  const size_t budget = small ? 110 * 1024 : 220 * 1024;
  if (kv8 && D != 128) return cudaErrorInvalidValue;
  int n_stages = kv8 ? kMaxStages : 8;
  while (n_stages > 2 && smem_bytes(D, p.group, n_stages, ncw, cl, kv8) > budget) --n_stages;
  // The consumer groups take tiles in turn: with a ring that is a multiple of the number of groups
  // every stage always belongs to the same group, which then waits for its phases one after the
  // other (a parity wait is only valid for the phase right after the last one known complete).
  // With several producer warps a stage must also always belong to the same producer.
  const int groups = ncw / kGroupWarps, producers = producer_warps(ncw, kv8);
  const int unit = groups > producers ? groups : producers;   // (1, 2 or 4: the larger is a multiple of the smaller)
  n_stages -= n_stages % unit;
  if (n_stages < unit) return cudaErrorInvalidConfiguration;
  const size_t smem = smem_bytes(D, p.group, n_stages, ncw, cl, kv8);
  const int slots = small ? 2 * sm_count : sm_count;
  const int grid = paired ? 2 * p.total_items : (p.total_items < slots ? p.total_items : slots);
  // launched with programmatic stream serialization: the kernel's set-up may overlap the
  // tail of the previous kernel in the stream; it waits (griddepcontrol.wait) before its
  // first global access
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3((ncw + producer_warps(ncw, kv8)) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = paired ? 2 : 1;
  if (kv8) {
    if (paired) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 8, 2, 1>, p, n_stages);
    if (small) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 4, 1, 1>, p, n_stages);
    return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 8, 1, 1>, p, n_stages);
  }
  if (D == 128) {
    if (paired) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 8, 2, 0>, p, n_stages);
    if (small) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 4, 1, 0>, p, n_stages);
    return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<128, 8, 1, 0>, p, n_stages);
  }
  if (paired) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<64, 8, 2, 0>, p, n_stages);
  if (small) return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<64, 4, 1, 0>, p, n_stages);
  return cudaLaunchKernelEx(&cfg, decode_split_bf16_kernel<64, 8, 1, 0>, p, n_stages);
}

}  // namespace mixattn

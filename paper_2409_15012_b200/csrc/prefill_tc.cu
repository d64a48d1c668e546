// Prompt attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16, head_dim 128 or 64
// (described for 128; the 64-channel form is noted at the kernel).
//
// Paper, Section 3 with the causal order of Section 1: query i attends to keys j <= i
// (standard layer) or i - window < j <= i (sliding window).  Flash-attention forward:
// one CTA owns a 128-query tile of one (sequence, head) and walks the 128-key tiles that
// intersect its band; tiles wholly outside the band are never loaded.  A sequence's queries
// may sit behind a prefix of keys cached by earlier calls (k / v then hold prefix + S rows):
// query row r has position prefix + r.
//
//   warp 0     TMA producer: Q once, then K and V tiles (3 / 2 stages) as 128B-swizzled
//              [128 x 64] boxes straight from the caller's tensors
//   warp 1     one elected thread issues the tcgen05.mma (K16 steps, bf16 -> fp32 in TMEM) of
//              S = Q K^T (M128 N128, both operands from shared memory) into one of two S
//              buffers, two tiles ahead of the softmax
//   warps 2-3  one elected thread per stream issues O_h += P_h V_h with P_h read from
//              tensor memory and V MN-major from its row-major tile
//   warps 4-7  softmax stream "lo": key columns 0-63 of every tile; warps 8-11 stream "hi":
//              columns 64-127.  The two streams are independent flash-attention passes
//              over interleaved halves of the keys (own exponent reference, own row sum,
//              own O accumulator in TMEM), merged exactly at the end like split-KV partials.
//              Thread r of a stream owns query row r (TMEM lane r): tcgen05.ld of its half
//              of the S row, band masks on edge tiles only, base-2 softmax weights with one
//              MUFU ex2 per score, P written back as bf16 pairs over its own columns of the
//              S buffer (tcgen05.st).  The exponent reference of a row is the maximum of the
//              first tile in which the row saw a key and is only moved (accumulators
//              rescaled, weights recomputed) when a later score leads it by more than 2^64,
//              which is noticed from the sum of the tile's weights: the exponentials of a
//              tile neither wait for the tile maximum nor compute it.
//   warps 12-15  epilogue: thread r merges the two accumulators of row r, normalises and
//              writes the row while the softmax warps are already on the next work item.
//
// Registers are moved between the roles with setmaxnreg (48 for the single-thread roles,
// 168 for the softmax warps, 128 for the epilogue).  Two softmax warps per scheduler work on
// independent data, the scores of the next two tiles are always ready, and the P V products
// are issued in whichever order the streams finish.
// TMEM: S0, S1, O_lo, O_hi = 4 x 128 columns.  All mbarrier waits are bounded; on
// time-out a status word is raised, every role leaves its loop, and TMEM is released at
// the common exit.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "internal.h"

namespace mixattn {

namespace {

constexpr int kBM = 128;                       // queries per work item
constexpr int kBN = 128;                       // keys per tile
constexpr int kHalfBytes = 128 * 128;          // one [128 rows x 64 bf16] swizzled block
constexpr int kTileBytes = 2 * kHalfBytes;     // a 128 x 128 bf16 operand tile
constexpr int kThreads = 512;                  // 4 single-thread roles, 2 x 4 softmax warps, 4 epilogue warps
constexpr int kKStages = 3, kVStages = 2;
constexpr int kSmQ = 0;                        // two Q buffers (this item / next item)
constexpr int kSmK = kSmQ + 2 * kTileBytes;
constexpr int kSmV = kSmK + kKStages * kTileBytes;
constexpr int kSmBar = kSmV + kVStages * kTileBytes;   // barriers, TMEM pointer, abort flag
constexpr int kSmXchg = kSmBar + 256;                  // [2 streams][128 rows] (max, sum)
constexpr int kSmemBytes = kSmXchg + 2 * 128 * 8 + 768;  // + slack to align a 256-B aligned base to 1024 B
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds of SM clock
constexpr uint32_t kColS = 0, kColO = 256;     // TMEM columns: S buffer b at 128 b, O of stream h at 256 + 128 h

// barrier indices
enum {
  B_QF = 0, B_QE = 2,            // Q buffer full / free (per buffer)
  B_KF = 4, B_KE = 7,            // K stage full / free
  B_VF = 10, B_VE = 12,          // V stage full / free
  B_SF = 14, B_SR = 16,          // S buffer: scores ready / buffer (with the P in it) consumed by both P V
  B_PF = 18,                     // per stream and S buffer (18 + 2 stream + buffer): P announced
  B_OF = 22,                     // per stream: the item's last P V done (one phase per item: a parity wait
                                 // is only valid for the phase right after the last one known complete)
  B_XC = 24, B_OR = 25,          // per item: streams published (reference, sum) / epilogue has read the O accumulators
  B_N = 26
};

struct TcParams {
  int32_t n_q_heads, group, window, n_seqs;
  int32_t max_qt;        // query tiles of the longest sequence
  float scale_log2e;
  int32_t* status;
  __nv_bfloat16* out;
  int32_t row0[kMaxCallSeqs + 1];   // first q / out row of each sequence
  int32_t krow0[kMaxCallSeqs];      // first k / v row of each sequence
  int32_t prefix[kMaxCallSeqs];     // keys before the sequence's first query
  int32_t cached[kMaxCallSeqs];     // the first so many of them live in a ring cache, not in k / v
  int32_t ring_page0[kMaxCallSeqs]; // first page of the sequence's ring
  int32_t ring_pages;               // pages per sequence in the ring (a multiple of 8)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {   // one look, never suspends
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();   // (the SM clock is cheap to read; the global timer is not)
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 format (version 1).
// lbo / sbo in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// D = A * B (+ D when accumulate != 0); one thread issues for the CTA.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Same with the A operand in tensor memory (rows = lanes, two bf16 per 32-bit column).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, single MUFU op; 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {   // three-input maximum, one instruction
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Waits for the tensor-memory loads in flight; the registers they fill are named as operands
// so that no use of them can be scheduled before the wait.
__device__ __forceinline__ void tmem_wait_ld_pin(uint32_t (&a)[32], uint32_t (&b)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
        "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
        "+r"(a[16]), "+r"(a[17]), "+r"(a[18]), "+r"(a[19]), "+r"(a[20]), "+r"(a[21]), "+r"(a[22]), "+r"(a[23]),
        "+r"(a[24]), "+r"(a[25]), "+r"(a[26]), "+r"(a[27]), "+r"(a[28]), "+r"(a[29]), "+r"(a[30]), "+r"(a[31])
      :: "memory");
  asm volatile(""
      : "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
        "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15]),
        "+r"(b[16]), "+r"(b[17]), "+r"(b[18]), "+r"(b[19]), "+r"(b[20]), "+r"(b[21]), "+r"(b[22]), "+r"(b[23]),
        "+r"(b[24]), "+r"(b[25]), "+r"(b[26]), "+r"(b[27]), "+r"(b[28]), "+r"(b[29]), "+r"(b[30]), "+r"(b[31])
      :: "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// (x, y) -> packed bf16 pair `hi` and the packed bf16 pair `lo` of the rounding residuals
__device__ __forceinline__ void split_bf16(float x, float y, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16(x, y);
  lo = pack_bf16(x - __uint_as_float(hi << 16), y - __uint_as_float(hi & 0xffff0000u));
}

// instruction descriptor: D fp32, A/B bf16, M = 128, N = n; b_mn = 1 for an MN-major B
__host__ __device__ constexpr uint32_t idesc_bf16(int b_mn, uint32_t n = 128) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// One work item: query tile qt of head h of sequence b.  Ids enumerate (sequence, reverse
// tile index, head): the CTAs of the grid work on one sequence at a time, whose K/V stays
// in L2 (a pass over all sequences at once re-read K/V from HBM 5x), heaviest tiles first,
// and the heads of a KV group, which read the same K/V tiles, run at the same time.
constexpr int kNoDup = 1 << 30;
struct WorkItem {
  int h, g, row_base, krow_base, S, i0, pos0, jt_lo, n_tiles;   // pos0 = position of query row i0 among the keys
  // Keys cached in a ring are read from the ring, the others from k / v.  When the cached keys
  // end inside a tile, that tile is visited twice: entry dup - 1 of the item's tile list takes
  // its cached keys from the ring, entry dup the rest from k / v (each masks the other's keys).
  int cached, ring_page0, dup;                                  // dup = kNoDup when no tile is visited twice
  bool valid;
  bool lo;   // rows of this tile may see fewer than a tile of keys: P enters P V as two bf16 terms
};
template <bool kRing>
__device__ __forceinline__ WorkItem get_item(const TcParams& p, int id) {
  WorkItem w;
  const int per_seq = p.max_qt * p.n_q_heads;
  const int b = id / per_seq;
  const int rem = id - b * per_seq;
  const int qt_rev = rem / p.n_q_heads;
  w.h = rem - qt_rev * p.n_q_heads;
  w.g = w.h / p.group;
  w.row_base = p.row0[b];
  w.krow_base = p.krow0[b];
  w.S = p.row0[b + 1] - p.row0[b];
  const int qt = (w.S + kBM - 1) / kBM - 1 - qt_rev;
  w.valid = qt >= 0;
  w.i0 = qt * kBM;
  w.pos0 = p.prefix[b] + w.i0;
  const int key_hi = p.prefix[b] + min(w.i0 + kBM - 1, w.S - 1);
  const int key_lo = p.window > 0 ? max(0, w.pos0 - p.window + 1) : 0;
  w.jt_lo = key_lo / kBN;
  w.n_tiles = key_hi / kBN - w.jt_lo + 1;
  w.cached = kRing ? p.cached[b] : 0;
  w.ring_page0 = kRing ? p.ring_page0[b] : 0;
  w.dup = kNoDup;
  if (kRing && w.cached % kBN != 0 && w.cached / kBN >= w.jt_lo) {   // (the queries sit behind the cached keys, so that tile is not past the last)
    w.dup = w.cached / kBN - w.jt_lo + 1;
    ++w.n_tiles;
  }
  // A row that sees only a few keys is a mix of a few V rows: its weights' bf16 rounding (2^-9
  // each) does not average out and, on outputs of magnitude 2..4, would add to the output's own
  // bf16 rounding.  Such rows (the first query tile of a sequence, or a window shorter than a
  // tile) carry the rounding residual of P as a second bf16 term, like the decode kernel; all
  // other tiles, whose rows average over at least a tile of keys, keep the single term.
  w.lo = w.pos0 < kBM || (p.window > 0 && p.window < kBN);
  return w;
}

// key tile (index along the sequence's keys) of entry j of an item's tile list
template <bool kRing>
__device__ __forceinline__ int tile_of(const WorkItem& w, int j) {
  return kRing ? w.jt_lo + j - (j >= w.dup ? 1 : 0) : w.jt_lo + j;
}

// kRing: some sequences have cached keys in a ring (a separate instantiation, so that the
// ordinary launches carry none of its code)
// kD: head_dim, 128 or 64.  With 64 channels an operand tile is one [128 x 64] block instead of
// two (the buffers keep their size), the score product takes four steps of 16 channels, the
// P V products write 64 accumulator columns, and the softmax warps do exactly the same work.
template <bool kRing, int kD>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_ring,
                  const __grid_constant__ TcParams p) {
  static_assert(kD == 128 || kD == 64, "head_dim");
  constexpr uint32_t kOpBytes = kD == 128 ? kTileBytes : kHalfBytes;   // bytes of one Q / K / V tile
  constexpr int kSteps = kD / 16;                                        // 16-channel steps of the score product
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar0 = base + kSmBar;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + kSmBar + B_N * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + kSmBar + B_N * 8 + 8);
#define BAR(i) (bar0 + 8u * (i))

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ids = p.max_qt * p.n_seqs * p.n_q_heads;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(BAR(B_QF + s), 1);
      mbar_init(BAR(B_QE + s), 1);
      mbar_init(BAR(B_VF + s), 1);
      mbar_init(BAR(B_VE + s), 2);   // both P V issuers
      mbar_init(BAR(B_SF + s), 1);
      mbar_init(BAR(B_SR + s), 2);   // both P V issuers
      mbar_init(BAR(B_PF + s), 4);
      mbar_init(BAR(B_PF + 2 + s), 4);
      mbar_init(BAR(B_OF + s), 1);
    }
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(BAR(B_KF + s), 1);
      mbar_init(BAR(B_KE + s), 1);
    }
    mbar_init(BAR(B_XC), 8);
    mbar_init(BAR(B_OR), 4);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // TMEM: all 512 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Every role walks the same item list and keeps the same counters: G = key tiles
  // processed so far by this CTA (all items), it = items processed so far.  Per-tile
  // barriers are indexed by G, per-item barriers by it, so phases carry over.
  if (warp < 4) {
    // single-thread roles: give registers back to the pool
    asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
    if (warp == 0) {
      // ------------------------------ TMA producer ------------------------------
      if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_ring) : "memory");
        bool ok = true;
        int G = 0, it = 0, q_issued = 0, k_issued = 0, v_issued = 0;
        for (int id = blockIdx.x; id < n_ids && ok; id += gridDim.x) {
          const WorkItem w = get_item<kRing>(p, id);
          if (!w.valid) continue;
          const int qb = it & 1;
          if (it >= 2) ok = mbar_wait(BAR(B_QE + qb), ((it >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(BAR(B_QF + qb), kOpBytes);
          tma_load_3d(base + kSmQ + qb * kTileBytes, &tm_q, 0, w.h, w.row_base + w.i0, BAR(B_QF + qb));
          if (kD == 128) tma_load_3d(base + kSmQ + qb * kTileBytes + kHalfBytes, &tm_q, 64, w.h, w.row_base + w.i0, BAR(B_QF + qb));
          ++q_issued;
          for (int j = 0; j < w.n_tiles && ok; ++j) {
            const int Gj = G + j;
            const int jt = tile_of<kRing>(w, j);
            // A tile of cached keys is eight whole pages of the sequence's ring: the page rows are
            // stored with the 16-byte chunks already permuted the way the MMA expects a
            // 128-byte-swizzled tile, so an unswizzled copy of (8 pages x 16 tokens x 128 bytes)
            // is that tile.  All other tiles come from k / v, whose row 0 is key w.cached.
            const bool from_ring = kRing && jt * kBN < w.cached && j != w.dup;
            const int row = w.krow_base + jt * kBN - w.cached;   // (negative rows of the tile shared with the ring read as zeros)
            const int page = w.ring_page0 + (jt * (kBN / kPage)) % p.ring_pages;
            const int ks = Gj % kKStages, ku = Gj / kKStages;
            if (ku > 0) ok = mbar_wait(BAR(B_KE + ks), (ku - 1) & 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(BAR(B_KF + ks), kOpBytes);
            if (from_ring) {
              tma_load_5d(base + kSmK + ks * kTileBytes, &tm_ring, 0, 0, 0, w.g, page, BAR(B_KF + ks));
              if (kD == 128) tma_load_5d(base + kSmK + ks * kTileBytes + kHalfBytes, &tm_ring, 64, 0, 0, w.g, page, BAR(B_KF + ks));
            } else {
              tma_load_3d(base + kSmK + ks * kTileBytes, &tm_k, 0, w.g, row, BAR(B_KF + ks));
              if (kD == 128) tma_load_3d(base + kSmK + ks * kTileBytes + kHalfBytes, &tm_k, 64, w.g, row, BAR(B_KF + ks));
            }
            ++k_issued;
            const int vs = Gj % kVStages, vu = Gj / kVStages;
            if (vu > 0) ok = mbar_wait(BAR(B_VE + vs), (vu - 1) & 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(BAR(B_VF + vs), kOpBytes);
            if (from_ring) {
              tma_load_5d(base + kSmV + vs * kTileBytes, &tm_ring, 0, 0, 1, w.g, page, BAR(B_VF + vs));
              if (kD == 128) tma_load_5d(base + kSmV + vs * kTileBytes + kHalfBytes, &tm_ring, 64, 0, 1, w.g, page, BAR(B_VF + vs));
            } else {
              tma_load_3d(base + kSmV + vs * kTileBytes, &tm_v, 0, w.g, row, BAR(B_VF + vs));
              if (kD == 128) tma_load_3d(base + kSmV + vs * kTileBytes + kHalfBytes, &tm_v, 64, w.g, row, BAR(B_VF + vs));
            }
            ++v_issued;
          }
          G += w.n_tiles;
          ++it;
        }
        if (!ok) {  // leave only after the copies already issued have landed (bounded)
          atomicExch(p.status, kDevWaitTimeout);
          for (int back = 1; back <= 2 && q_issued - back >= 0; ++back)
            mbar_wait(BAR(B_QF + ((q_issued - back) & 1)), ((q_issued - back) >> 1) & 1, abort_flag + 1);
          for (int back = 1; back <= kKStages && k_issued - back >= 0; ++back)
            mbar_wait(BAR(B_KF + (k_issued - back) % kKStages), ((k_issued - back) / kKStages) & 1, abort_flag + 1);
          for (int back = 1; back <= kVStages && v_issued - back >= 0; ++back)
            mbar_wait(BAR(B_VF + (v_issued - back) % kVStages), ((v_issued - back) / kVStages) & 1, abort_flag + 1);
        }
      }
    } else if (warp == 1) {
      // ------------------------------ MMA issuer, scores ------------------------------
      // Three threads issue MMAs (this one S = Q K^T, warps 2 and 3 the P V products of the
      // two streams): issuing is a serial, latency-bound instruction stream, and one thread
      // alone was the bottleneck.
      if (lane == 0) {
        constexpr uint32_t kIdescS = idesc_bf16(0);
        bool ok = true;
        int G = 0, it = 0;
        for (int id = blockIdx.x; id < n_ids && ok; id += gridDim.x) {
          const WorkItem w = get_item<kRing>(p, id);
          if (!w.valid) continue;
          const int qb = it & 1;
          ok = mbar_wait(BAR(B_QF + qb), (it >> 1) & 1, abort_flag);
          uint64_t qdesc[kSteps];
  #pragma unroll
          for (int ks = 0; ks < kSteps; ++ks)   // head_dim = kSteps steps of 16 channels
            qdesc[ks] = smem_desc(base + kSmQ + qb * kTileBytes + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024);
          for (int j = 0; j < w.n_tiles && ok; ++j) {
            // S(G) = Q K^T into S buffer G & 1, which held S(G-2) / P(G-2): wait until both
            // P V(G-2) have consumed it (they are issued by another thread)
            const int Gj = G + j, sb = Gj & 1, ks_ = Gj % kKStages;
            ok = mbar_wait(BAR(B_KF + ks_), (Gj / kKStages) & 1, abort_flag);   // (long there as a rule)
            if (ok && Gj >= 2) ok = mbar_wait(BAR(B_SR + sb), ((Gj >> 1) - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint64_t kdesc = smem_desc(base + kSmK + ks_ * kTileBytes, 16, 1024);
  #pragma unroll
            for (int ks = 0; ks < kSteps; ++ks)
              umma_bf16(tmem + kColS + sb * 128, qdesc[ks],
                        kdesc + (uint64_t)((ks >> 2) * (kHalfBytes >> 4) + (ks & 3) * 2), kIdescS, ks > 0);
            umma_commit(BAR(B_SF + sb));    // scores ready
            umma_commit(BAR(B_KE + ks_));   // K stage free
          }
          if (ok) umma_commit(BAR(B_QE + qb));   // Q buffer free once this item's S products are done
          G += w.n_tiles;
          ++it;
        }
        if (!ok) atomicExch(p.status, kDevWaitTimeout);
      }
    } else {
      // ------------------------------ MMA issuers, P V (one per stream) ------------------------------
      if (lane == 0) {
        constexpr uint32_t kIdescPV = idesc_bf16(1, kD);
        const int hs = warp - 2;
        bool ok = true;
        int G = 0, it = 0;
        for (int id = blockIdx.x; id < n_ids && ok; id += gridDim.x) {
          const WorkItem w = get_item<kRing>(p, id);
          if (!w.valid) continue;
          // the first P V of an item overwrites the O accumulator: the streams must have
          // read the previous item's result
          if (it >= 1) ok = mbar_wait(BAR(B_OR), (it - 1) & 1, abort_flag);
          for (int j = 0; j < w.n_tiles && ok; ++j) {
            const int Gj = G + j, sb = Gj & 1, vs = Gj % kVStages;
            ok = mbar_wait(BAR(B_VF + vs), (Gj / kVStages) & 1, abort_flag);
            if (ok) ok = mbar_wait(BAR(B_PF + 2 * hs + sb), (Gj >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // O_h += P_h V[64 h .. 64 h + 63]: A = P from tensor memory (two bf16 per column),
            // B = V MN-major (channels contiguous, keys strided by 128 B)
            const uint64_t vdesc = smem_desc(base + kSmV + vs * kTileBytes + hs * 4 * 2048, kHalfBytes, 1024);
  #pragma unroll
            for (int ks = 0; ks < 4; ++ks)   // 64 keys = 4 steps of 16
              umma_bf16_ts(tmem + kColO + hs * 128, tmem + kColS + sb * 128 + hs * 64 + ks * 8,
                           vdesc + (uint64_t)(ks * (2048 >> 4)), kIdescPV, (j > 0 || ks > 0) ? 1u : 0u);
            if (w.lo) {   // the residual term of P sits in the other 32 of the stream's 64 columns
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                umma_bf16_ts(tmem + kColO + hs * 128, tmem + kColS + sb * 128 + hs * 64 + 32 + ks * 8,
                             vdesc + (uint64_t)(ks * (2048 >> 4)), kIdescPV, 1u);
            }
            if (j == w.n_tiles - 1) umma_commit(BAR(B_OF + hs));   // this stream's accumulator is complete
            umma_commit(BAR(B_VE + vs));   // V stage free once both streams' P V are done (count 2)
            umma_commit(BAR(B_SR + sb));   // and so is the S buffer
          }
          G += w.n_tiles;
          ++it;
        }
        if (!ok) atomicExch(p.status, kDevWaitTimeout);
      }
    }
  } else if (warp >= 12) {
    // ------------------------------ epilogue warps ------------------------------
    // Thread r merges the two streams' accumulators of query row r like split-KV partials
    // and writes the row, while the softmax warps already work on the next item.
    const int qd = warp & 3;
    const int r = qd * 32 + lane;
    const uint32_t lane_base = tmem + ((uint32_t)(qd * 32) << 16);
    const float2* xchg = reinterpret_cast<const float2*>(gbase + kSmXchg);
    bool ok = true;
    int it = 0;
    for (int id = blockIdx.x; id < n_ids && ok; id += gridDim.x) {
      const WorkItem w = get_item<kRing>(p, id);
      if (!w.valid) continue;
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_XC), it & 1, abort_flag));
      if (!ok) break;
      const float2 lo = xchg[r], hi = xchg[128 + r];
      // both streams' last P V of the item have landed
      ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_OF + 0), it & 1, abort_flag) &&
                                   mbar_wait(BAR(B_OF + 1), it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const float m_all = fmaxf(lo.x, hi.x);              // finite for every valid row (key i is visible)
      const float e_lo = ex2_approx(lo.x - m_all), e_hi = ex2_approx(hi.x - m_all);   // 2^-inf = 0
      const float inv = 1.f / (lo.y * e_lo + hi.y * e_hi);
      const float w_lo = e_lo * inv, w_hi = e_hi * inv;
      const int i = w.i0 + r;
      __nv_bfloat16* orow = p.out + ((int64_t)(w.row_base + i) * p.n_q_heads + w.h) * kD;
#pragma unroll
      for (int c = 0; c < kD / 32; ++c) {
        uint32_t olo[32], ohi[32];
        tmem_ld32(lane_base + kColO + c * 32, olo);
        tmem_ld32(lane_base + kColO + 128 + c * 32, ohi);
        tmem_wait_ld();
        if (c == kD / 32 - 1) {   // the accumulators may be overwritten by the next item
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(B_OR));
        }
        if (i < w.S) {
#pragma unroll
          for (int q8 = 0; q8 < 4; ++q8) {
            uint32_t o4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int d = q8 * 8 + e * 2;
              o4[e] = pack_bf16(__uint_as_float(olo[d]) * w_lo + __uint_as_float(ohi[d]) * w_hi,
                                __uint_as_float(olo[d + 1]) * w_lo + __uint_as_float(ohi[d + 1]) * w_hi);
            }
            *reinterpret_cast<uint4*>(orow + c * 32 + q8 * 8) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
          }
        }
      }
      ++it;
    }
    if (!ok && lane == 0) atomicExch(p.status, kDevWaitTimeout);
  } else {
    // ------------------------------ softmax warps ------------------------------
    asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
    const int hs = (warp - 4) >> 2;       // stream: key columns [64 hs, 64 hs + 64) of every tile
    const int qd = warp & 3;              // TMEM lane quarter this warp may access
    const int r = qd * 32 + lane;         // query row within the tile
    const uint32_t lane_base = tmem + ((uint32_t)(qd * 32) << 16);
    const uint32_t o_addr = lane_base + kColO + hs * 128;
    float2* xchg = reinterpret_cast<float2*>(gbase + kSmXchg);
    // The exponent reference of a row is the maximum of the first tile in which the row saw a
    // key; it is only moved (and the accumulators rescaled) when a later score leads it by
    // more than 2^kMaxLead, so the exponentials of a tile do not wait for the tile maximum.
    constexpr float kMaxLead = 64.f;
    bool ok = true;
    int G = 0, it = 0;
    for (int id = blockIdx.x; id < n_ids && ok; id += gridDim.x) {
      const WorkItem w = get_item<kRing>(p, id);
      if (!w.valid) continue;
      const int i = w.pos0 + r;           // query position among the sequence's keys
      float m_ref = -INFINITY, l = 0.f;
      uint32_t sv[64];
      {
        if (!__all_sync(0xffffffffu, mbar_wait(BAR(B_SF + (G & 1)), (G >> 1) & 1, abort_flag))) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = lane_base + kColS + (G & 1) * 128 + hs * 64;
        tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_wait_ld_pin(*reinterpret_cast<uint32_t(*)[32]>(&sv[0]), *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
      }
      // The tile loop exists twice: for ordinary items (one bf16 term of P) and for the few items
      // whose rows see fewer than a tile of keys (two terms).  Keeping the second form out of the
      // first one's code matters: with both in one loop body the ordinary tiles ran 3-5 % slower.
      auto run_tiles = [&](auto lo_tag) {
        constexpr bool kLo = decltype(lo_tag)::value;
        for (int j = 0; j < w.n_tiles; ++j) {
          const int Gj = G + j, sb = Gj & 1;
          const int j0 = tile_of<kRing>(w, j) * kBN + hs * 64;   // first key of this stream's columns
          const uint32_t s_addr = lane_base + kColS + sb * 128 + hs * 64;
          // band edges: causal (keys after the query) and window (keys older than i - window); and
          // the two visits of the tile in which the cached keys end
          const bool edge = (j0 + 63 > w.pos0) || (p.window > 0 && j0 <= w.pos0 + kBM - 1 - p.window) ||
                            (kRing && (j + 1 == w.dup || j == w.dup));
          auto mask_edges = [&]() {
            int k_max = i - j0;                                      // columns <= k_max are causal-visible
            int k_min = p.window > 0 ? i - p.window + 1 - j0 : 0;    // columns >= k_min are inside the window
            if (kRing && j + 1 == w.dup) k_max = min(k_max, w.cached - 1 - j0);   // this visit: the cached keys only
            if (kRing && j == w.dup) k_min = max(k_min, w.cached - j0);           // this visit: the keys from k / v only
  #pragma unroll
            for (int e = 0; e < 64; ++e)
              if (e > k_max || e < k_min) sv[e] = 0xff800000u;             // -inf
          };
          if (edge) mask_edges();
          // a row that has not seen a key yet takes its reference from this tile
          const bool fresh = m_ref == -INFINITY;
          if (__any_sync(0xffffffffu, fresh)) {
            float mx0 = -INFINITY, mx1 = -INFINITY;
  #pragma unroll
            for (int e = 0; e < 64; e += 4) {
              mx0 = fmax3(mx0, __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
              mx1 = fmax3(mx1, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
            }
            if (fresh) m_ref = fmaxf(mx0, mx1) * p.scale_log2e;
          }
          float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;   // no visible key yet: weights 0, no NaN
          // probe the next tile's scores now; the answer is read after the exponentials
          const bool more = j + 1 < w.n_tiles;
          const bool next_ready = more && mbar_test_wait(BAR(B_SF + (sb ^ 1)), ((Gj + 1) >> 1) & 1);
          float sum0 = 0.f, sum1 = 0.f;
          uint32_t pk[32], pl[32];   // P as bf16 pairs; pl = rounding residuals (only on w.lo items)
          if constexpr (!kLo) {
  #pragma unroll
            for (int e = 0; e < 64; e += 4) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(sv[e]), p.scale_log2e, neg_m));
              const float p1 = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), p.scale_log2e, neg_m));
              const float p2 = ex2_approx(fmaf(__uint_as_float(sv[e + 2]), p.scale_log2e, neg_m));
              const float p3 = ex2_approx(fmaf(__uint_as_float(sv[e + 3]), p.scale_log2e, neg_m));
              sum0 += p0 + p2;
              sum1 += p1 + p3;
              pk[e >> 1] = pack_bf16(p0, p1);
              pk[(e >> 1) + 1] = pack_bf16(p2, p3);
            }
          } else {
  #pragma unroll
            for (int e = 0; e < 64; e += 2) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(sv[e]), p.scale_log2e, neg_m));
              const float p1 = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), p.scale_log2e, neg_m));
              sum0 += p0;
              sum1 += p1;
              split_bf16(p0, p1, pk[e >> 1], pl[e >> 1]);
            }
          }
          // A score that leads the reference by more than 2^kMaxLead shows in the sum of the tile's
          // weights (64 weights of at most 2^kMaxLead each stay below 2^(kMaxLead + 6); an overflow
          // gives inf or NaN, which fail the comparison too), so the loop above carries no maximum.
          const bool big = !(sum0 + sum1 <= 0x1p70f);
          static_assert(kMaxLead == 64.f, "the bound above is 2^(kMaxLead + 6)");
          if (__any_sync(0xffffffffu, big)) {
            // rare: take the tile maximum from the scores, which are still in the S buffer (P has
            // not been written yet), move the reference of the leading rows up to it, rescale what
            // they have accumulated, and recompute this tile's weights
            tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
            tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
            tmem_wait_ld_pin(*reinterpret_cast<uint32_t(*)[32]>(&sv[0]), *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
            if (edge) mask_edges();
            float mxa = -INFINITY, mxb = -INFINITY;
  #pragma unroll
            for (int e = 0; e < 64; e += 4) {
              mxa = fmax3(mxa, __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
              mxb = fmax3(mxb, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
            }
            const float mt = fmaxf(mxa, mxb) * p.scale_log2e;
            const bool far = mt > m_ref + kMaxLead;
            const float alpha = far ? ex2_approx(m_ref - mt) : 1.f;
            if (j > 0) {   // the O row holds earlier tiles: rescale it once this stream's previous P V has landed
              // (the S buffer of tile G - 1 is released when both streams' P V of that tile are done;
              // its previous phase is known complete because the scores of tile G - 1 existed)
              if (!__all_sync(0xffffffffu, mbar_wait(BAR(B_SR + (sb ^ 1)), ((Gj - 1) >> 1) & 1, abort_flag))) { ok = false; break; }
              tc_fence_after();
  #pragma unroll 1
              for (int c = 0; c < kD / 32; ++c) {
                uint32_t ov[32];
                tmem_ld32(o_addr + c * 32, ov);
                tmem_wait_ld();
  #pragma unroll
                for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * alpha);
                tmem_st32(o_addr + c * 32, ov);
              }
            }
            l *= alpha;
            if (far) m_ref = mt;
            neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
            sum0 = 0.f;
            sum1 = 0.f;
  #pragma unroll
            for (int e = 0; e < 64; e += 2) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(sv[e]), p.scale_log2e, neg_m));
              const float p1 = ex2_approx(fmaf(__uint_as_float(sv[e + 1]), p.scale_log2e, neg_m));
              sum0 += p0;
              sum1 += p1;
              if constexpr (kLo) split_bf16(p0, p1, pk[e >> 1], pl[e >> 1]);
              else pk[e >> 1] = pack_bf16(p0, p1);
            }
          }
          l += sum0 + sum1;
          // P (bf16 pairs) over the first 32 of this stream's 64 score columns, the residual
          // term, where the item carries one, over the other 32
          tmem_st32(s_addr, pk);
          if constexpr (kLo) tmem_st32(s_addr + 32, pl);
          tmem_wait_st();
          tc_fence_before();
          // (one announcement barrier per S buffer: its next phase cannot complete before the
          // scores of tile G + 2 exist, that is before the MMA thread has consumed this one)
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(B_PF + 2 * hs + sb));
          // the next tile's scores
          if (more) {
            if (!__all_sync(0xffffffffu, next_ready || mbar_wait(BAR(B_SF + (sb ^ 1)), ((Gj + 1) >> 1) & 1, abort_flag))) { ok = false; break; }
            tc_fence_after();
            const uint32_t n_addr = lane_base + kColS + (sb ^ 1) * 128 + hs * 64;
            tmem_ld32(n_addr, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
            tmem_ld32(n_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          }
          if (more) tmem_wait_ld_pin(*reinterpret_cast<uint32_t(*)[32]>(&sv[0]), *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        }
      };
      if (w.lo) run_tiles(std::true_type{});
      else run_tiles(std::false_type{});
      if (!ok) break;
      G += w.n_tiles;
      // hand (reference, sum) of the row to the epilogue warps; the slot is free once they
      // have read the previous item's pair
      if (it >= 1) ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_OR), (it - 1) & 1, abort_flag));
      if (!ok) break;
      xchg[hs * 128 + r] = make_float2(m_ref, l);
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_XC));
      ++it;
    }
    if (!ok && lane == 0) atomicExch(p.status, kDevWaitTimeout);
  }
  // common exit: everyone is past its last TMEM access
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
#undef BAR
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &ptr, 12000, cudaEnableDefault, &qres) ==
            cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// [rows, heads, D] bf16 tensor; box = 64 channels x 1 head x 128 rows, 128-byte swizzle
bool make_map(CUtensorMap* map, const void* ptr, int64_t rows, int heads, int D) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2};
  cuuint32_t box[3] = {64, 1, 128};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Ring storage of one owner layer, native bf16 format, seen as
// [pages][heads][K | V][16 tokens][head_dim channels]; box = 64 channels x 16 tokens x 8 pages of one
// head's K or V.  The stored rows carry the 128-byte-swizzle permutation already (internal.h),
// so the copy itself does not swizzle.
bool make_ring_map(CUtensorMap* map, const void* pool, const KvGeom& ge, int64_t pages) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[5] = {(cuuint64_t)ge.head_dim, (cuuint64_t)kPage, 2, (cuuint64_t)ge.n_kv_heads, (cuuint64_t)pages};
  cuuint64_t strides[4] = {(cuuint64_t)ge.row_bytes, (cuuint64_t)kPage * ge.row_bytes, (cuuint64_t)ge.blk_bytes,
                           (cuuint64_t)ge.page_bytes};
  cuuint32_t box[5] = {64, (cuuint32_t)kPage, 1, 1, kBN / kPage};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool prefill_tc_ring_direct_supported(const KvGeom& ge, int window) {
  return !ge.fp8 && ge.swizzle && (ge.head_dim == 128 || ge.head_dim == 64) && ge.elem_bytes == 2 && window > 0 && window % kBN == 0;
}

bool prefill_tc_supported(int dtype, int head_dim, const void* q, const void* k, const void* v) {
  auto aligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  return dtype == MIXATTN_BF16 && (head_dim == 128 || head_dim == 64) && aligned(q) && aligned(k) && aligned(v) && encode_fn() != nullptr;
}

cudaError_t prepare_prefill_tc() {
  cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(prefill_tc_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(prefill_tc_kernel<false, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(prefill_tc_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  return e;
}

cudaError_t launch_prefill_tc(const PrefillParams& pp, int max_len, int sm_count, cudaStream_t st) {
  if (pp.n_seqs <= 0 || max_len <= 0) return cudaSuccess;
  const int64_t rows = pp.row0[pp.n_seqs];
  int64_t k_rows = 0;   // k / v hold prefix - cached + S rows per sequence
  for (int i = 0; i < pp.n_seqs; ++i) {
    const int cached = pp.ring_pool != nullptr ? pp.cached[i] : 0;
    if (cached < 0 || cached > pp.prefix[i]) return cudaErrorInvalidValue;
    const int64_t end = (int64_t)pp.krow0[i] + pp.prefix[i] - cached + (pp.row0[i + 1] - pp.row0[i]);
    if (end > k_rows) k_rows = end;
  }
  CUtensorMap tq, tk, tv, tring;
  const int D = pp.head_dim;
  if (D != 128 && D != 64) return cudaErrorInvalidValue;
  if (!make_map(&tq, pp.q, rows, pp.n_q_heads, D) || !make_map(&tk, pp.k, k_rows, pp.n_kv_heads, D) ||
      !make_map(&tv, pp.v, k_rows, pp.n_kv_heads, D))
    return cudaErrorInvalidValue;
  if (pp.ring_pool != nullptr) {
    if (!prefill_tc_ring_direct_supported(pp.geom, pp.window) || pp.ring_pages * kPage != pp.window ||
        !make_ring_map(&tring, pp.ring_pool, pp.geom, pp.ring_total_pages))
      return cudaErrorInvalidValue;
  } else {
    tring = tk;   // never read
  }
  TcParams p;
  p.n_q_heads = pp.n_q_heads;
  p.group = pp.n_q_heads / pp.n_kv_heads;
  p.window = pp.window;
  p.n_seqs = pp.n_seqs;
  p.scale_log2e = pp.scale_log2e;
  p.status = pp.status;
  p.out = static_cast<__nv_bfloat16*>(pp.out);
  for (int i = 0; i <= pp.n_seqs; ++i) p.row0[i] = pp.row0[i];
  for (int i = 0; i < pp.n_seqs; ++i) {
    p.krow0[i] = pp.krow0[i];
    p.prefix[i] = pp.prefix[i];
    p.cached[i] = pp.ring_pool != nullptr ? pp.cached[i] : 0;
    p.ring_page0[i] = pp.ring_pool != nullptr ? pp.ring_page0[i] : 0;
  }
  p.ring_pages = pp.ring_pool != nullptr ? pp.ring_pages : kBN / kPage;
  p.max_qt = (max_len + kBM - 1) / kBM;
  const int64_t n_ids = (int64_t)p.max_qt * pp.n_seqs * pp.n_q_heads;
  const int grid = (int)(n_ids < sm_count ? n_ids : sm_count);   // persistent: one CTA per SM
  const bool ring = pp.ring_pool != nullptr;
  if (D == 128) {
    if (ring) prefill_tc_kernel<true, 128><<<grid, kThreads, kSmemBytes, st>>>(tq, tk, tv, tring, p);
    else prefill_tc_kernel<false, 128><<<grid, kThreads, kSmemBytes, st>>>(tq, tk, tv, tring, p);
  } else {
    if (ring) prefill_tc_kernel<true, 64><<<grid, kThreads, kSmemBytes, st>>>(tq, tk, tv, tring, p);
    else prefill_tc_kernel<false, 64><<<grid, kThreads, kSmemBytes, st>>>(tq, tk, tv, tring, p);
  }
  return cudaGetLastError();
}

}  // namespace mixattn

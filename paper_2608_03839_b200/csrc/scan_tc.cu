// K3: tensor-core scan for batched queries (many requests against one shared pool).
//
// Scoring line of Algorithm 1 (cosine of the query with every stored state) for nq queries at
// once: S[i, q] = <key_i, qn_q> is a [N x d] x [d x nq] contraction.  Keys are the M
// operand (tiles of 128 rows), the normalised queries the N operand (nq padded to a
// multiple of 16), d is walked in blocks of 64 elements.  Each CTA is persistent and
// warp-specialised:
//   warp 0      TMA producer: key tile + query tile per k-block into a 128B-swizzled
//               shared-memory ring (cp.async.bulk.tensor, mbarrier complete_tx)
//   warp 1      tcgen05.mma issuer (one elected lane), fp32 accumulators in TMEM, two
//               accumulator buffers so the next tile's MMAs overlap the epilogue
//   warps 2-5   epilogue: tcgen05.ld the 128 x nq scores, filter them against the
//               per-query running k-th best, and keep per-query top-k lists (Eq. 2) in
//               shared memory, or in L2 when they are large; scores never go to global
//               memory
// The key stream (N*d*2 bytes from HBM, once) bounds the kernel up to nq ~ 64-96; the
// epilogue warps then wait for accumulators 60-80 % of the time.  Beyond that:
//   - A CTA's first tile has no thresholds yet.  It is read twice: once for its best score
//     per query only, which the CTAs exchange to agree on a bound (the k-th largest of their
//     bests), then as every other tile, against that bound.  Without this every score of the
//     first one or two tiles went through the sorted lists (~2.5 tiles' worth of time at
//     nq = 128, with the accumulators full and the key stream stalled).
//   - From 129 queries on, two CTAs share each tile of 256 rows (template argument kPair;
//     described at the kernel), which halves the query bytes an SM pulls from L2 and writes
//     to its shared memory per key byte.
//   - Per k-block of a 128-row tile the tensor core reads the 16 KB of keys and the
//     n_pad x 128 bytes of queries from shared memory while TMA writes the next ones: at
//     n_pad = 256 that is 96 KB through the SM's shared memory per k-block, and cycle
//     counters in the MMA-issuing thread (not part of the build) show the four
//     128 x 256 x 16 MMAs of a k-block taking ~750 cycles where the tensor pipe alone would
//     need 512 and the SM's share of the HBM rate allows 720: at nq = 256 the scan is bound
//     on chip (and, in runs of more than a fraction of a second, by the power cap: the SM
//     clock settles at 1.0-1.3 GHz), not by HBM.  A pair of CTAs moves 64-80 KB per k-block
//     and gains 6-10 %.
// The MMA warp walks its loop as a whole and one elected lane issues, so that descriptors and
// addresses are computed in uniform control flow (with the loop inside `if (lane == 0)` a
// k-block's four MMAs and its commit took ~745 cycles to issue at n_pad = 256, now ~500).
// Small pools (a few tiles per SM): a query costs about 40 us plus the key bytes at HBM
// speed, against 12 us plus the same for the CUDA-core scan.  A tile's scores exist only
// after its whole K loop, so the first tile's latency chain is not overlapped.  Then come
// the query normalisation kernel and the merge.
// Measured and not kept:
//   - a variant with the roles swapped (queries as M = 128, one query per TMEM lane and per
//     epilogue thread; 256 key rows as N): passes the same tests, slower everywhere (0.90
//     instead of 1.03 of the measured HBM rate at nq = 16, 0.73 instead of 0.81 at nq = 128 on
//     the 8.6 GB pool, 2-3x slower on small pools);
//   - per-CTA row ranges at 32-row granularity, ring depths up to 12, seeding the first
//     tile's thresholds from per-warp 32-bit sorts: nothing gained;
//   - separate shared-memory rings for keys and query tiles (query tiles queue behind the key
//     requests, so they need the same lead; 5-8 % slower); a 32-deep candidate queue with
//     retry; ballot-packed per-warp queue segments instead of shared-memory atomics (drain
//     60 % slower); sorting every column of the first tile in registers without the queue; a
//     variant that transposes the scores through shared memory so that one warp owns a
//     query's 128 rows (15-30 % slower);
//   - per-query lists kept in shared memory as 6-byte slots (fp32 score + 16-bit local row)
//     to make 256 x 64 of them fit beside a two-stage ring: with the lists in global memory
//     (L2) the ring has four stages and the scan is a third faster;
//   - two CTAs on a tile with the other CTA's copies counted directly on the leader's
//     barrier after an arrival (with its byte count) from the other CTA's producer, or with
//     a warp of the other CTA relaying "stage landed" to the leader: an arrival on a barrier
//     of the other CTA with release semantics costs the arriving thread ~600 cycles, and
//     either form ran at 1,600 cycles per k-block;
//   - a single 128 x 256 x 16 MMA issued as two interleaved 128 x 128 x 16 ones (independent
//     accumulators): 8 instructions in ~950 cycles instead of 4 in ~750; the same two halves
//     issued by two warps at once: 857 cycles per k-block against 856 with one issuer, so
//     what bounds the loop is the operands' way through shared memory, not the issue;
//   - a suspend-time hint (2 or 20 us) on the mbarrier waits, to spin less under the power
//     cap: no change in sustained runs;
//   - asking for the keys of the next 8 or 24 k-blocks into L2 ahead of the ring
//     (cp.async.bulk.prefetch.tensor): 1.4x and 2x slower at every nq.
//
// Every mbarrier wait is bounded: after the pool's wait limit (two seconds by default) it
// raises the pool's `stalled` flag, the CTA drains what it has in flight, frees its TMEM and
// returns.  The two meetings of the CTAs in a first tile are short waits (0.1 ms) that give
// up silently, since they only serve a tighter filter.
#include <cuda.h>

#include <new>

#include "common.cuh"
#include "internal.h"

namespace oilbird {

constexpr int kTcThreads = 192;
constexpr int kConvWarps = 6;          // warps that turn codes into f16 (8-bit pools)
constexpr int kTcThreadsFp8 = kTcThreads + 32 * kConvWarps;
constexpr int kTileM = 128;            // key rows per tile = TMEM lanes
// bf16 elements per k-block = one 128-byte swizzle row.  (32-element blocks with the 64-byte
// swizzle were measured too: more, finer ring stages, but every 128-byte line is then
// requested twice and the scan runs 30-40 % slower at every nq.)
constexpr int kBlockK = 64;
constexpr int kATileBytes = kTileM * kBlockK * 2;   // 16 KB
constexpr int kCodeTileBytes = kTileM * kBlockK;    // the same tile as E4M3 codes: 8 KB
constexpr int kColsPerRound = 16;      // score columns read from TMEM and filtered at a time
constexpr int kQueueCap = kTileM * kColsPerRound;   // candidate slots, shared out among the queries
constexpr int kMaxStages = 8;

// Lists stay in shared memory if this many ring stages still fit beside them.
constexpr int kTcMinSmemStages = 4;

// ------------------------------------------------------------------ PTX wrappers ---
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// try_wait whose acquire reaches across the cluster: for a barrier that a thread of the other
// CTA arrives on after it has seen its own copies land
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if it gave up (or another role already did).
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStats* stats) {
  if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns(), limit = wait_limit_ns(stats);
  for (uint32_t spin = 0;; ++spin) {
    if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 63u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit) {
        *abort_flag = 1;
        atomicExch(&stats->stalled, 1);
        return false;
      }
    }
  }
}
// One lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
// mbar_wait by a whole converged warp, with one outcome for all its lanes
template <bool kCluster = false>
__device__ __forceinline__ bool warp_mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                               DeviceStats* stats) {
  const bool ok = mbar_wait<kCluster>(bar, parity, abort_flag, stats);
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
// ---- two CTAs on one tile (a cluster of two; rank 0 leads) ----
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// the address, in the cluster's shared window, of the same shared-memory object in CTA `rank`
__device__ __forceinline__ uint32_t smem_of_rank(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {      // every thread of both CTAs
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_at(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
               : "memory");
}
// TMA load into this CTA's shared memory whose completion is counted on a barrier that may
// live in the other CTA of the pair (no operand is shared between the CTAs: each loads its
// own rows)
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
// completion of the pair's MMAs so far, counted on one barrier given by its cluster address
__device__ __forceinline__ void tc_commit_pair_at(uint32_t bar_cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar_cluster_addr)
               : "memory");
}
// D[tmem of both CTAs] (+)= A * B over the pair: M = 256 (128 rows from each CTA's A tile),
// N from idesc (each CTA's B tile holds N/2 of the query rows), K = 16.  One thread of the
// leading CTA issues it.
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                 uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(smem_u32(bar))
               : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 x bf16 -> fp32, M=128, N from idesc, K=16
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32"
      " {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void epilogue_bar() {      // the 128 epilogue threads only
  asm volatile("bar.sync 1, 128;" ::: "memory");
}
// the same barrier, returning whether any of the 128 threads brought a true flag
__device__ __forceinline__ bool epilogue_bar_or(bool flag) {
  uint32_t any;
  asm volatile(
      "{\n\t.reg .pred p_in, p_out;\n\t"
      "setp.ne.u32 p_in, %1, 0;\n\t"
      "bar.red.or.pred p_out, 1, 128, p_in;\n\t"
      "selp.u32 %0, 1, 0, p_out;\n\t}"
      : "=r"(any) : "r"((uint32_t)flag) : "memory");
  return any != 0;
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes wide
// and 128B-swizzled (what the TMA box above produces): 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                              // leading byte offset (unused, 16 B)
  d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset: 8 rows of 128 B
  d |= (uint64_t)1 << 46;                              // descriptor version (Blackwell)
  d |= (uint64_t)2 << 61;                              // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A/B bf16, both K-major, M = m (128; 256 over a CTA pair), N = n.
__host__ __device__ inline uint32_t umma_idesc_bf16(int n, int m = kTileM) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

// The same with f16 operands (8-bit pools: an E4M3 code is an f16 number exactly).
__host__ __device__ inline uint32_t umma_idesc_f16(int n, int m = kTileM) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// four E4M3 codes (one word) -> two f16x2 (codes 0,1 and codes 2,3)
__device__ __forceinline__ void e4m3x4_to_f16x4(uint32_t w, uint32_t& h01, uint32_t& h23) {
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "mov.b32 {lo, hi}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, lo;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, hi;\n\t}"
      : "=r"(h01), "=r"(h23)
      : "r"(w));
}
// Order-preserving map float -> unsigned (and back), so that a warp-wide maximum of scores is
// one redux instruction; 0 is below every score.
__device__ __forceinline__ uint32_t score_to_ord(float s) {
  s += 0.0f;
  const uint32_t b = __float_as_uint(s);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_to_score(uint32_t b) {
  return __uint_as_float((b & 0x80000000u) ? (b & 0x7fffffffu) : ~b);
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Rendezvous of the grid's CTAs on an arrival counter, for a bound that only makes the
// filter tighter: a short wait that simply ends when its time is up (nothing is flagged; the
// caller goes on with whatever the other CTAs have published by then).
constexpr unsigned long long kRendezvousNs = 100000ull;
__device__ __forceinline__ void rendezvous_wait(const unsigned* counter, unsigned want) {
  if (ld_acquire_u32(counter) >= want) return;
  const unsigned long long t0 = global_ns();
  while (ld_acquire_u32(counter) < want && global_ns() - t0 < kRendezvousNs) __nanosleep(100);
}

// ------------------------------------------------------------- per-query lists ---
struct TcShared {
  uint64_t full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], drain;
  uint64_t cvt[kMaxStages];     // 8-bit pools: the stage's codes have been turned into f16
  uint32_t tmem_base;
  int abort_flag;
  int epi_go;
};

// Per-query candidate lists of one CTA: kk packed 64-bit keys per query, descending, empty
// slots 0.  They live in shared memory while that leaves the operand ring deep enough; for
// many queries and large k (256 x 64 slots are 128 KB) they live in global memory instead,
// directly in the CTA's slice of the scan's output, where they stay in L2: a list is read
// and written only by the warp that owns its query and, once the thresholds have settled,
// only a few times per tile, while the shared memory it would take is worth two or three
// ring stages of operands in flight (the key stream of one SM needs ~45 KB in flight to
// run at its share of the HBM rate).
struct ListStore {
  u64* slots;
  int kk;
  bool global;

  __device__ __forceinline__ u64 load(int q, int i) const {
    return global ? __ldcg(slots + (size_t)q * kk + i) : slots[(size_t)q * kk + i];
  }
  __device__ __forceinline__ void store(int q, int i, u64 key) const {
    if (global) __stcg(slots + (size_t)q * kk + i, key);
    else slots[(size_t)q * kk + i] = key;
  }
};

// Fold the candidates queued in one round into the descending lists of the (up to four)
// queries this warp owns in the round.  Lists live in shared memory (kk = 32*E slots, empty
// slots are 0) and are held in registers meanwhile; afterwards the filter threshold of
// each query, the score of its k-th entry once k entries exist, is refreshed.
// A crowd of candidates (a CTA's first tiles, while its thresholds are still low) is sorted
// 32*E at a time and merged; the usual handful is inserted one by one, the queries'
// independent insert chains interleaved so that they hide each other's shuffle latency.
constexpr int kDrainQ = kColsPerRound / 4;      // queries per warp and round
constexpr int kCrowd = 8;

template <int E>
__device__ __forceinline__ void drain_cols(const ListStore& lists, const u64* q_key, int q_cap,
                                           const int* q_cnt, const int (&cols)[kDrainQ], int k,
                                           float* thr_s, int lane, int col0) {
  u64 v[kDrainQ][E];
  u64 kth[kDrainQ];
  int n[kDrainQ];
  int n_max = 0, crowd_max = 0;
#pragma unroll
  for (int u = 0; u < kDrainQ; ++u) {
    const int q = cols[u];
    n[u] = q >= 0 ? q_cnt[q] : 0;
    n[u] = n[u] > q_cap ? q_cap : n[u];          // pushes beyond the queue's end were not stored
    if (n[u] > 0) {
#pragma unroll
      for (int r = 0; r < E; ++r) v[u][r] = lists.load(q, r * 32 + lane);
      kth[u] = warp_list_get<E>(v[u], k - 1);
    } else {
#pragma unroll
      for (int r = 0; r < E; ++r) v[u][r] = 0;
      kth[u] = 0;
    }
    if (n[u] >= kCrowd) crowd_max = n[u] > crowd_max ? n[u] : crowd_max;
    else n_max = n[u] > n_max ? n[u] : n_max;
  }
  // crowds: batches of 32*E candidates are sorted and merged, the four queries' networks
  // in one basic block so that they overlap (an uncrowded query rides along with zeros)
  for (int i0 = 0; i0 < crowd_max; i0 += 32 * E) {
    u64 b[kDrainQ][E];
#pragma unroll
    for (int u = 0; u < kDrainQ; ++u) {
#pragma unroll
      for (int r = 0; r < E; ++r) {
        const int i = i0 + r * 32 + lane;
        const u64 key = (n[u] >= kCrowd && i < n[u]) ? q_key[(size_t)(cols[u] - col0) * q_cap + i] : 0;
        b[u][r] = key > kth[u] ? key : 0;
      }
    }
    warp_sort_desc_batch<kDrainQ, E>(b, lane);
    warp_merge_desc_batch<kDrainQ, E>(v, b, lane);
#pragma unroll
    for (int u = 0; u < kDrainQ; ++u) kth[u] = warp_list_get<E>(v[u], k - 1);
  }
  for (int i = 0; i < n_max; ++i) {
#pragma unroll
    for (int u = 0; u < kDrainQ; ++u) {
      // every queued candidate beat the threshold it was filtered with; kth only settles
      // ties and is refreshed after the round (a worse key just falls off the end)
      u64 key = (n[u] < kCrowd && i < n[u]) ? q_key[(size_t)(cols[u] - col0) * q_cap + i] : 0;
      key = key > kth[u] ? key : 0;
      warp_sorted_insert<E>(v[u], key, lane);
    }
  }
#pragma unroll
  for (int u = 0; u < kDrainQ; ++u) {
    if (n[u] > 0) {
      const int q = cols[u];
#pragma unroll
      for (int r = 0; r < E; ++r) lists.store(q, r * 32 + lane, v[u][r]);
      const u64 nk = warp_list_get<E>(v[u], k - 1);
      // never below a bound adopted from the other CTAs
      if (lane == 0 && nk != 0) thr_s[q] = fmaxf(thr_s[q], candidate_score(nk));
    }
  }
}

// Warp ew folds everything queued for its queries (ew, ew + 4, ...) into their lists, four
// queries at a time, and empties those queues.  Candidates wait in per-query queues from the
// round that found them to the end of their tile (or until a queue is full): a list kept in
// global memory costs a round trip to L2 to fetch and one to put back, and draining after
// every round of sixteen columns paid that for the one or two queries of the round that had
// a candidate (256 queries, k = 64: 198 of 224 rounds drained, 3,650 cycles each, the
// epilogue busy for 840,000 of the kernel's 1,090,000 cycles and the MMAs waiting for it).
template <int E>
__device__ __forceinline__ void flush_queues(const ListStore& lists, const u64* q_key, int q_cap,
                                             int* q_cnt, int n_pad, int ew, int k, float* thr_s,
                                             int lane, int col0 = 0) {
  // col0: the queue of query q starts at slot (q - col0) * q_cap (the round-wide layout below)
  const int per_warp = n_pad >> 2;
  for (int base = 0; base < per_warp; base += 32) {
    const int i = base + lane;
    const int cnt = i < per_warp ? q_cnt[ew + 4 * i] : 0;
    unsigned m = __ballot_sync(0xffffffffu, cnt > 0);
    while (m) {
      int cols[kDrainQ];
#pragma unroll
      for (int u = 0; u < kDrainQ; ++u) {
        cols[u] = m ? ew + 4 * (base + __ffs(m) - 1) : -1;
        m &= m - 1;
      }
      drain_cols<E>(lists, q_key, q_cap, q_cnt, cols, k, thr_s, lane, col0);
      __syncwarp();
      int mine = -1;
#pragma unroll
      for (int u = 0; u < kDrainQ; ++u) mine = lane == u ? cols[u] : mine;
      if (mine >= 0) q_cnt[mine] = 0;
    }
  }
  __syncwarp();
}

// The k-th largest of the CTAs' published best scores for query q (one per CTA), by k rounds
// of warp-wide maximum extraction; -inf while fewer than k CTAs have published one.  Each is
// the score of a distinct row, so k rows of the pool reach the value returned.
__device__ __forceinline__ float kth_largest_best(const float* lmax, int q, int k, int lane) {
  float mine[kTcMaxCtas / 32];
#pragma unroll
  for (int i = 0; i < kTcMaxCtas / 32; ++i) {
    const int c = i * 32 + lane;
    mine[i] = c < (int)gridDim.x ? __ldcg(&lmax[(size_t)q * kTcMaxCtas + c]) : -INFINITY;
  }
  float kth_best = -INFINITY;
  for (int r = 0; r < k; ++r) {
    float m = mine[0];
#pragma unroll
    for (int i = 1; i < kTcMaxCtas / 32; ++i) m = fmaxf(m, mine[i]);
    float w = m;
#pragma unroll
    for (int o = 16; o; o >>= 1) w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, o));
    kth_best = w;
    if (w == -INFINITY) break;                                     // fewer than k bests yet
    const int owner = __ffs(__ballot_sync(0xffffffffu, m == w)) - 1;
    if (lane == owner) {                                           // remove one instance
      bool done = false;
#pragma unroll
      for (int i = 0; i < kTcMaxCtas / 32; ++i)
        if (!done && mine[i] == w) { mine[i] = -INFINITY; done = true; }
    }
  }
  return kth_best;
}

// ------------------------------------------------------------------- the kernel ---
// Queries [q0, q0+nq_c) of the call; n_pad = nq_c rounded up to 16 = MMA N.
// mt (1 or 2) key tiles of 128 rows share each query tile: with mt = 2 the query bytes
// pulled from L2 per key byte halve, which is what limits the kernel from nq ~ 64 up.
// n_bufs accumulator sets of mt*n_pad TMEM columns each (2 = the next macro tile's MMAs
// overlap the epilogue; 1 when 2*mt*n_pad would exceed the 512 columns).
//
// kPair: two CTAs (a cluster of two, on neighbouring SMs) work on one tile of 256 rows, for
// batches of more than 128 queries.  There the accumulators of 128 rows x n_pad queries take
// half of an SM's TMEM, so a lone CTA can share a query tile between no more than one key
// tile at a time: 2 bytes of query per byte of key through the SM's L2 port, which is then
// what bounds the kernel (~1,100 cycles per 16 KB of keys against ~720 at the HBM rate).  In
// a pair each CTA loads its own 128 key rows and HALF of the query rows, and one
// tcgen05.mma over both CTAs (M = 256) reads both halves: 1 byte of query per byte of key.
// No load is shared or broadcast between the CTAs: each CTA's copies land in its own shared
// memory.  The leading CTA (rank 0) issues the MMAs and owns the `full` and `tmem_empty`
// barriers, on which both CTAs' copies and both CTAs' epilogue warps are counted; `empty`
// and `tmem_full` exist in both CTAs and the leader's commits are counted on both.  With
// mt = 2 each CTA holds two key tiles per stage and the pair's macro tile is 512 rows:
// sub-tile `sub` of tile t is rows ((t*mt + sub)*2 + rank)*128 onward.
//
// kFp8 (lone CTAs only): the pool holds E4M3 codes and one fp32 scale per row.  The tensor
// core takes 16-bit operands, so a stage's codes (8 KB per tile, loaded by TMA without
// swizzle) are turned into the f16 tile the MMA reads by six more warps: 16 codes per
// 16-byte shared-memory load, `cvt.rn.f16x2.e4m3x2` (exact), two 16-byte stores into the
// 128-byte-swizzled layout a TMA load would have produced, a proxy fence, and an arrival on
// the stage's `cvt` barrier, which is what the MMA warp waits for in place of `full`.  The
// queries arrive as f16 scaled by 2^14 (see the query preparation); a row's scale and the
// 2^-14 are applied to its scores as they leave TMEM.  HBM carries half the bytes of a
// 16-bit pool; shared memory carries more (codes in and out, f16 in and out), which is what
// bounds this form (C4 as codes, nq = 16: 0.95 ms = 4.5 TB/s of codes where the stage's
// 100 KB through shared memory at 128 B/clock give 0.8).  Measured and dropped: making the
// f16 numbers with integer shifts and masks (the code's magnitude bits at f16's exponent and
// fraction read 2^-8 times its value, exactly, subnormal codes included) for all rows or
// for every other quarter of a tile: 1.30 and 1.11 ms against 0.95; four or eight
// converting warps in place of six: 1.02 and 0.95 against 0.97; a ring of code stages with
// two f16 slots of their own: 1.14; the converting warps fetching the codes from global
// memory themselves, two stages ahead in registers (no TMA, no codes in shared memory):
// 1.34 against 0.97.
template <bool kPair, bool kFp8 = false>
__global__ void __launch_bounds__(kFp8 ? kTcThreadsFp8 : kTcThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap key_map,
               const __grid_constant__ CUtensorMap q_map, PoolView pv, int q0, int nq_c,
               int nq_total, int n_pad, int k, int kk, int n_stages, int tmem_cols, int mt,
               int n_bufs, int global_lists, const uint64_t* __restrict__ exclude_tag,
               u64* __restrict__ partial, DeviceStats* stats, float* xchg,
               const float* __restrict__ scales) {
  static_assert(!(kPair && kFp8), "8-bit pools run lone CTAs");
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ TcShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_rank() : 0u;       // 0 = the CTA that issues the MMAs
  const int n_ctas = kPair ? 2 : 1;
  const int b_rows = n_pad / n_ctas;                       // query rows this CTA loads
  const int a_bytes = mt * kATileBytes;
  const int raw_off = a_bytes + b_rows * kBlockK * 2;       // 8-bit pools: the stage's codes
  const int stage_bytes = raw_off + (kFp8 ? mt * kCodeTileBytes : 0);
  // dynamic shared memory: [stages][mt key tiles | query tile | codes] | lists | queue | state
  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = base;
  unsigned char* list_mem = ring + (size_t)n_stages * stage_bytes;              // [nq_c][kk]
  ListStore lists;
  lists.global = global_lists != 0;
  lists.slots = lists.global ? partial + ((size_t)blockIdx.x * nq_total + q0) * kk
                             : reinterpret_cast<u64*>(list_mem);
  lists.kk = kk;
  u64* q_key = reinterpret_cast<u64*>(list_mem + (lists.global ? 0 : (size_t)nq_c * kk * 8));
                                                               // [n_pad][q_cap]
  uint64_t* s_ex = reinterpret_cast<uint64_t*>(q_key + kQueueCap);              // [n_pad]
  float* thr_s = reinterpret_cast<float*>(s_ex + n_pad);                        // [n_pad]
  uint32_t* s_qmax = reinterpret_cast<uint32_t*>(thr_s + n_pad);                // [n_pad]
  int* q_cnt = reinterpret_cast<int*>(s_qmax + n_pad);                          // [n_pad]
  const int q_cap = kQueueCap / n_pad;       // queue slots per query (8 at 256 queries)
  // Cross-CTA threshold exchange (global memory, reset to -inf by the query preparation):
  // lmax[q][cta] = best score CTA `cta` has seen for query q; gthr[q] = a score that at
  // least k distinct rows of the pool are known to reach, namely the k-th largest of the
  // CTAs' bests (one row per CTA).  No row below gthr[q] can be among the k best, so the
  // filter threshold of a query is max(its local k-th score, just below gthr[q]).  Local
  // thresholds only see one CTA's rows (1/148 of the pool); with the exchange the number of
  // candidates that reach the sorted lists after a CTA's first tiles drops by about two
  // orders of magnitude.  Values only grow, so stale reads are merely weaker bounds.
  float* lmax = xchg;
  float* gthr = xchg + (size_t)OILBIRD_MAX_NQ * kTcMaxCtas;
  unsigned* arrivals = reinterpret_cast<unsigned*>(xchg + kTcXchgFloats);       // two counters
  const bool use_xchg = (int)gridDim.x >= k && (int)gridDim.x <= kTcMaxCtas;

  // a macro tile: mt tiles of 128 rows of this CTA, or one of each CTA of the pair; the
  // tiles of a grid are dealt out to its units (CTAs or pairs) round robin
  const int rows_per_macro = (kPair ? 2 : 1) * mt * kTileM;
  const int n_tiles = (pv.n_rows + rows_per_macro - 1) / rows_per_macro;
  const int unit = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_units = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int n_kb = (pv.d + kBlockK - 1) / kBlockK;
  volatile int* abort_flag = &sh.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
      mbar_init(&sh.cvt[s], kConvWarps);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sh.tmem_full[b], 1);
      mbar_init(&sh.tmem_empty[b], 4 * n_ctas);
    }
    mbar_init(&sh.drain, 1);
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation is a whole-warp operation (the same warp of both CTAs of a pair)
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&sh.tmem_base)), "r"((uint32_t)tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(&sh.tmem_base)), "r"((uint32_t)tmem_cols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();     // the other CTA's barriers exist before anything is counted on them
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  pdl_enter();   // appended rows, normalised queries, exclusion tags; set-up above overlapped
  for (int i = threadIdx.x; i < n_pad; i += (int)blockDim.x) {
    thr_s[i] = i < nq_c ? -INFINITY : INFINITY;        // padded columns never pass the filter
    s_qmax[i] = 0u;
    q_cnt[i] = 0;
    s_ex[i] = (exclude_tag && i < nq_c) ? exclude_tag[q0 + i] : 0;
  }
  for (int i = threadIdx.x; i < nq_c * kk; i += (int)blockDim.x) lists.store(i / kk, i % kk, 0);
  __syncthreads();

  if (warp == 0) {
    // ===================================================== TMA producer ==========
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&key_map) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int tile = unit; tile < n_tiles && ok; tile += n_units) {
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          const uint32_t ph = (it / n_stages) & 1u;
          if (!mbar_wait(&sh.empty[s], ph ^ 1u, abort_flag, stats)) { ok = false; break; }
          unsigned char* a_dst = ring + (size_t)s * stage_bytes;
          if (kPair) {
            // Both CTAs' bytes are counted on the leader's barrier, and the leader's producer
            // announces them all (the other CTA's bytes may land first: the count then
            // dips below zero until the announcement, and the phase cannot complete before
            // the leader's arrival).  Nothing but the copies' own completions crosses between
            // the CTAs here: an arrival from the other CTA with release semantics was
            // measured at ~600 cycles per stage for the thread that makes it.
            const uint32_t full_at = smem_of_rank(&sh.full[s], 0);
            if (rank == 0) mbar_arrive_expect_tx(&sh.full[s], 2u * (uint32_t)stage_bytes);
            for (int sub = 0; sub < mt; ++sub)
              tma_load_2d_pair(a_dst + sub * kATileBytes, &key_map, kb * kBlockK,
                               ((tile * mt + sub) * 2 + (int)rank) * kTileM, full_at);
            tma_load_2d_pair(a_dst + a_bytes, &q_map, kb * kBlockK, q0 + (int)rank * b_rows, full_at);
          } else if (kFp8) {
            mbar_arrive_expect_tx(&sh.full[s], (uint32_t)(stage_bytes - a_bytes));
            for (int sub = 0; sub < mt; ++sub)    // codes: 64 bytes x 128 rows, rows as they are
              tma_load_2d(a_dst + raw_off + sub * kCodeTileBytes, &key_map, kb * kBlockK,
                          (tile * mt + sub) * kTileM, &sh.full[s]);
            tma_load_2d(a_dst + a_bytes, &q_map, kb * kBlockK, q0, &sh.full[s]);
          } else {
            mbar_arrive_expect_tx(&sh.full[s], (uint32_t)stage_bytes);
            for (int sub = 0; sub < mt; ++sub)    // rows past the pool's capacity read as zero
              tma_load_2d(a_dst + sub * kATileBytes, &key_map, kb * kBlockK,
                          (tile * mt + sub) * kTileM, &sh.full[s]);
            tma_load_2d(a_dst + a_bytes, &q_map, kb * kBlockK, q0, &sh.full[s]);
          }
        }
      }
      if (!ok) {
        // gave up: let the copies already issued land before the CTA's memory goes away
        const uint32_t back = it < (uint32_t)n_stages ? it : (uint32_t)n_stages;
        for (uint32_t j = 0; j < back && rank == 0; ++j) {   // (a pair's copies are counted in the leader)
          const uint32_t i2 = it - 1 - j;
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&sh.full[i2 % n_stages], (i2 / n_stages) & 1u) &&
                 global_ns() - t0 < 2000000ull) {}
        }
        if (rank != 0) {                                     // let this CTA's own copies land
          const unsigned long long t0 = global_ns();
          while (global_ns() - t0 < 20000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================== MMA issuer ============
    // The whole warp walks the loop and one elected lane issues: everything the MMAs take
    // (descriptors, accumulator address, barrier addresses) is then computed in uniform
    // control flow, where the compiler can keep it in uniform registers, which is where
    // tcgen05.mma takes its operands from.
    if (rank == 0) {
      const bool issuer = elect_one();
      const uint32_t idesc = kFp8 ? umma_idesc_f16(n_pad) : umma_idesc_bf16(n_pad, kPair ? 2 * kTileM : kTileM);
      uint32_t it = 0, iter = 0;
      bool ok = true;
      for (int tile = unit; tile < n_tiles && ok; tile += n_units, ++iter) {
        const uint32_t buf = iter % (uint32_t)n_bufs;
        if (!warp_mbar_wait(&sh.tmem_empty[buf], ((iter / (uint32_t)n_bufs) & 1u) ^ 1u, abort_flag,
                            stats)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * (uint32_t)(mt * n_pad);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          if (!warp_mbar_wait(kFp8 ? &sh.cvt[s] : &sh.full[s], (it / n_stages) & 1u, abort_flag, stats)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(ring + (size_t)s * stage_bytes);
          const uint64_t a_desc = umma_desc_sw128(a_addr);
          const uint64_t b_desc = umma_desc_sw128(a_addr + a_bytes);
          const uint32_t acc = (uint32_t)(kb != 0);
          if (kPair) {
            const uint32_t empty0 = smem_of_rank(&sh.empty[s], 0), empty1 = smem_of_rank(&sh.empty[s], 1);
            const uint64_t a_desc1 = a_desc + (uint64_t)(kATileBytes >> 4);     // second key tile
            const uint32_t d_tmem1 = d_tmem + (uint32_t)n_pad;
            if (issuer) {
#pragma unroll
              for (int kq = 0; kq < kBlockK / 16; ++kq)
                tc_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(kq * 2), b_desc + (uint64_t)(kq * 2),
                                 idesc, kq != 0 ? 1u : acc);
              if (mt == 2) {
#pragma unroll
                for (int kq = 0; kq < kBlockK / 16; ++kq)
                  tc_mma_bf16_pair(d_tmem1, a_desc1 + (uint64_t)(kq * 2), b_desc + (uint64_t)(kq * 2),
                                   idesc, kq != 0 ? 1u : acc);
              }
              // the stage is reusable in both CTAs once the MMAs retire
              tc_commit_pair_at(empty0);
              tc_commit_pair_at(empty1);
            }
          } else {
            const uint64_t a_desc1 = a_desc + (uint64_t)(kATileBytes >> 4);     // second key tile
            const uint32_t d_tmem1 = d_tmem + (uint32_t)n_pad;
            if (issuer) {
#pragma unroll
              for (int kq = 0; kq < kBlockK / 16; ++kq)      // 32 bytes along K per MMA
                tc_mma_bf16(d_tmem, a_desc + (uint64_t)(kq * 2), b_desc + (uint64_t)(kq * 2), idesc,
                            kq != 0 ? 1u : acc);
              if (mt == 2) {
#pragma unroll
                for (int kq = 0; kq < kBlockK / 16; ++kq)
                  tc_mma_bf16(d_tmem1, a_desc1 + (uint64_t)(kq * 2), b_desc + (uint64_t)(kq * 2), idesc,
                              kq != 0 ? 1u : acc);
              }
              tc_commit(&sh.empty[s]);                        // stage reusable once the MMAs retire
            }
          }
        }
        __syncwarp();
        if (ok && issuer) {
          if (kPair) {
            tc_commit_pair_at(smem_of_rank(&sh.tmem_full[buf], 0));
            tc_commit_pair_at(smem_of_rank(&sh.tmem_full[buf], 1));
          } else {
            tc_commit(&sh.tmem_full[buf]);
          }
        }
      }
      // nothing may still be writing TMEM when it is freed
      __syncwarp();
      if (issuer) {
        if (kPair) tc_commit_pair_at(smem_of_rank(&sh.drain, 0));
        else tc_commit(&sh.drain);
        const unsigned long long t0 = global_ns();
        const unsigned long long limit = wait_limit_ns(stats);
        while (!mbar_try_wait(&sh.drain, 0) && global_ns() - t0 < limit) {}
      }
      __syncwarp();
    }
  } else if (kFp8 && warp >= 6) {
    // ===================================================== codes -> f16 ==========
    // thread ct takes the 16-byte pieces ct, ct + 128, ... of a stage's codes (consecutive
    // lanes read consecutive pieces: no bank conflict); piece g is codes 16 (g % 4) onward of
    // row g / 4, i.e. the row's 16-byte f16 chunks 2 (g % 4) and 2 (g % 4) + 1, which the
    // 128-byte swizzle keeps at chunk position (chunk ^ (row % 8)) of the row's 128 bytes
    const int ct = threadIdx.x - kTcThreads;
    uint32_t it = 0;
    bool ok = true;
    for (int tile = unit; tile < n_tiles && ok; tile += n_units) {
      for (int kb = 0; kb < n_kb; ++kb, ++it) {
        const int s = it % n_stages;
        if (!mbar_wait(&sh.full[s], (it / n_stages) & 1u, abort_flag, stats)) { ok = false; break; }
        unsigned char* a_dst = ring + (size_t)s * stage_bytes;
        const uint4* raw = reinterpret_cast<const uint4*>(a_dst + raw_off);
        // All of a thread's pieces are loaded before any is converted (one after the other, each
        // waiting for its own load, kept the whole scan at a third of its rate).
        constexpr int kConvThreads = 32 * kConvWarps;
        constexpr int kMaxPieces = (2 * kCodeTileBytes / 16 + kConvThreads - 1) / kConvThreads;
        const int n_total = mt * (kCodeTileBytes / 16);                 // 16-byte pieces of the stage
        uint4 c[kMaxPieces];
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i)
          if (ct + i * kConvThreads < n_total) c[i] = raw[ct + i * kConvThreads];
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i) {
          if (ct + i * kConvThreads < n_total) {
            const int g = ct + i * kConvThreads;
            const int row_all = g >> 2, c4 = g & 3;         // row over the stage's tiles
            unsigned char* row_dst = a_dst + (size_t)row_all * 128;
            const int sw = row_all & 7;
            uint4 lo, hi;
            e4m3x4_to_f16x4(c[i].x, lo.x, lo.y);
            e4m3x4_to_f16x4(c[i].y, lo.z, lo.w);
            e4m3x4_to_f16x4(c[i].z, hi.x, hi.y);
            e4m3x4_to_f16x4(c[i].w, hi.z, hi.w);
            *reinterpret_cast<uint4*>(row_dst + (((2 * c4) ^ sw) << 4)) = lo;
            *reinterpret_cast<uint4*>(row_dst + (((2 * c4 + 1) ^ sw) << 4)) = hi;
          }
        }
        // the tile was written through the generic proxy; the MMA reads it through the async one
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.cvt[s]);
      }
    }
  } else {
    // ===================================================== epilogue ==============
    const int ew = warp - 2;                    // 0..3: which queries this warp owns in drains
    const int lane_grp = warp & 3;              // TMEM lanes this warp may read
    const int et = threadIdx.x - 64;            // 0..127
    uint32_t iter = 0;
    bool ok = true;
    for (int tile = unit; tile < n_tiles && ok; tile += n_units, ++iter) {
      const uint32_t buf = iter % (uint32_t)n_bufs;
      mbar_wait(&sh.tmem_full[buf], (iter / (uint32_t)n_bufs) & 1u, abort_flag, stats);
      // one decision for all four warps, so that the barriers below always match up
      epilogue_bar();
      if (et == 0) sh.epi_go = *abort_flag ? 0 : 1;
      epilogue_bar();
      if (!sh.epi_go) { ok = false; break; }
      tc_fence_after();
      if (use_xchg && iter == 0) {
        // A CTA's first tile, before any threshold exists: every score would be a candidate
        // (sorted 32*E at a time and merged, a couple of tiles' worth of time during which
        // the accumulators stay full and the key stream stalls).  Instead the tile is read
        // twice.  First only its best score per query is taken (one redux per column and
        // warp) and published; the CTAs meet; the CTA responsible for a query takes the k-th
        // largest of the CTAs' bests, which k distinct rows of the pool reach, as the bound;
        // the CTAs meet again and adopt it.  The second reading of the tile is the regular
        // filter, now against a bound that a few rows per query pass.  The two meetings are
        // short waits that give up silently: a missing bound only means a weaker filter.
        for (int sub = 0; sub < mt; ++sub) {
          const int row = (kPair ? (tile * mt + sub) * 2 + (int)rank : tile * mt + sub) * kTileM + lane_grp * 32 + lane;
          const bool row_ok = row < pv.n_rows;
          uint64_t tag = 0;
          if (exclude_tag && row_ok) tag = pv.trace_tag[pv.trace_id[row]];
          const uint32_t t_row = tmem_base + ((uint32_t)(lane_grp * 32) << 16) +
                                 (uint32_t)sub * (uint32_t)n_pad;               // buffer 0
          // 8-bit pools: score = scale(row) * sum / 2^14 (the queries' scaling taken back)
          const float rs = (kFp8 && row_ok) ? scales[row] * (1.f / 16384.f) : 0.f;
          for (int c0 = 0; c0 < n_pad; c0 += kColsPerRound) {
            float v[kColsPerRound];
            tc_ld16(t_row + (uint32_t)c0, v);
            if (kFp8) {
#pragma unroll
              for (int j = 0; j < kColsPerRound; ++j) v[j] *= rs;
            }
            uint32_t mine = 0;
#pragma unroll
            for (int j = 0; j < kColsPerRound; ++j) {
              const bool skip = !row_ok || (s_ex[c0 + j] != 0 && tag == s_ex[c0 + j]);
              const uint32_t m = __reduce_max_sync(0xffffffffu, skip ? 0u : score_to_ord(v[j]));
              mine = lane == j ? m : mine;
            }
            if (lane < kColsPerRound && mine != 0u) atomicMax(&s_qmax[c0 + lane], mine);
          }
        }
        epilogue_bar();
        for (int q = et; q < nq_c; q += 128)
          if (s_qmax[q] != 0u)
            __stcg(&lmax[(size_t)(q0 + q) * kTcMaxCtas + blockIdx.x], ord_to_score(s_qmax[q]));
        __threadfence();
        epilogue_bar();
        if (et == 0) atomicAdd(&arrivals[0], 1u);
        // (the queries this CTA answers for, q0 + q = blockIdx.x mod gridDim.x, dealt out to
        // the four warps in turn: they are a stride of gridDim.x apart, which is often a
        // multiple of four)
        const int q_first = (((int)blockIdx.x - q0) % (int)gridDim.x + (int)gridDim.x) % (int)gridDim.x;
        for (int j = 0, q = q_first; q < nq_c; ++j, q += (int)gridDim.x) {
          if ((j & 3) != ew) continue;                                    // warp-uniform
          rendezvous_wait(&arrivals[0], gridDim.x);
          const float kth_best = kth_largest_best(lmax, q0 + q, k, lane);
          if (lane == 0 && kth_best > -INFINITY && kth_best > __ldcg(&gthr[q0 + q]))
            __stcg(&gthr[q0 + q], kth_best);
        }
        __threadfence();
        epilogue_bar();
        if (et == 0) {
          atomicAdd(&arrivals[1], 1u);
          rendezvous_wait(&arrivals[1], gridDim.x);
        }
        epilogue_bar();
      }
      if (use_xchg) {
        // adopt the agreed bounds: v > max(local, prev(g))  <=>  v > local and v >= g
        for (int q = et; q < nq_c; q += 128) {
          const float g = __ldcg(&gthr[q0 + q]);
          if (g > -INFINITY) thr_s[q] = fmaxf(thr_s[q], nextafterf(g, -INFINITY));
        }
      }
      epilogue_bar();
      bool long_way = false;                    // (see the rounds below) per tile, all warps alike
      for (int sub = 0; sub < mt; ++sub) {      // sub-tiles in row order: ties stay exact
      const int row = (kPair ? (tile * mt + sub) * 2 + (int)rank : tile * mt + sub) * kTileM + lane_grp * 32 + lane;
      const bool row_ok = row < pv.n_rows;
      uint64_t tag = 0;
      if (exclude_tag && row_ok) tag = pv.trace_tag[pv.trace_id[row]];
      const uint32_t t_row = tmem_base + ((uint32_t)(lane_grp * 32) << 16) +
                             (buf * (uint32_t)mt + (uint32_t)sub) * (uint32_t)n_pad;
      const float rs = (kFp8 && row_ok) ? scales[row] * (1.f / 16384.f) : 0.f;
      for (int c0 = 0; c0 < n_pad; c0 += kColsPerRound) {
        float v[kColsPerRound];
        tc_ld16(t_row + (uint32_t)c0, v);
        if (kFp8) {
#pragma unroll
          for (int j = 0; j < kColsPerRound; ++j) v[j] *= rs;
        }
        if (sub == mt - 1 && c0 + kColsPerRound >= n_pad) {
          // all of this macro tile's scores have been read: hand the accumulators back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (kPair) mbar_arrive_at(smem_of_rank(&sh.tmem_empty[buf], 0));
            else mbar_arrive(&sh.tmem_empty[buf]);
          }
        }
        // The round's sixteen thresholds are fetched together and compared without a
        // branch; only the (rare) passing columns are visited.  Comparing column by column
        // with the queue's atomics in the loop body keeps every threshold load behind the
        // previous column's possible store and costs ~2,000 cycles a round.
        uint32_t pass = 0;
        {
          const float4* t4 = reinterpret_cast<const float4*>(thr_s + c0);
          const float4 ta = t4[0], tb = t4[1], tc = t4[2], td = t4[3];
          const float t[kColsPerRound] = {ta.x, ta.y, ta.z, ta.w, tb.x, tb.y, tb.z, tb.w,
                                          tc.x, tc.y, tc.z, tc.w, td.x, td.y, td.z, td.w};
#pragma unroll
          for (int j = 0; j < kColsPerRound; ++j) pass |= (v[j] > t[j] ? 1u : 0u) << j;
          if (!row_ok) pass = 0;
        }
        // Lanes walk their passing columns from different starting points: while a CTA's
        // thresholds are still low every row passes in every column, and 128 threads taking
        // the columns in the same order would serialise on one counter at a time.
        const int rot = lane & (kColsPerRound - 1);
        pass = ((pass >> rot) | (pass << (kColsPerRound - rot))) & ((1u << kColsPerRound) - 1u);
        // Passing scores go into their query's queue; the queues are folded into the lists at
        // the end of the tile.  When a queue is full (thresholds still loose, or a stretch of
        // rows each better than the last) the tile goes on the long way: everything queued so
        // far is folded, and from then on a round's candidates go into queues of a whole
        // sub-tile's depth, which the queue memory holds for the sixteen columns of one round,
        // and are folded behind the round (sorted in batches of 32*E).
        uint32_t retry = 0;
        if (!long_way) {
          while (pass) {
            const uint32_t low = pass & (0u - pass);
            const int j = (__ffs(pass) - 1 + rot) & (kColsPerRound - 1);
            pass &= pass - 1;
            const int q = c0 + j;
            if (s_ex[q] != 0 && tag == s_ex[q]) continue;         // same-prompt trace: skipped
            float vj = v[0];
#pragma unroll
            for (int i = 1; i < kColsPerRound; ++i) vj = j == i ? v[i] : vj;
            const int pos = atomicAdd(&q_cnt[q], 1);
            if (pos < q_cap) q_key[(size_t)q * q_cap + pos] = pack_candidate(vj, (uint32_t)row);
            else retry |= low;
          }
          if (!epilogue_bar_or(retry != 0)) continue;             // every candidate found room
          if (kk == 32) flush_queues<1>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
          else if (kk == 64) flush_queues<2>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
          else flush_queues<4>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
          epilogue_bar();                                         // every queue is empty
          long_way = true;
          pass = retry;
        }
        bool pushed = false;
        while (pass) {
          const int j = (__ffs(pass) - 1 + rot) & (kColsPerRound - 1);
          pass &= pass - 1;
          if (s_ex[c0 + j] != 0 && tag == s_ex[c0 + j]) continue;
          float vj = v[0];
#pragma unroll
          for (int i = 1; i < kColsPerRound; ++i) vj = j == i ? v[i] : vj;
          const int pos = atomicAdd(&q_cnt[c0 + j], 1);           // < 128: one per row at most
          q_key[(size_t)j * kTileM + pos] = pack_candidate(vj, (uint32_t)row);
          pushed = true;
        }
        if (epilogue_bar_or(pushed)) {
          if (kk == 32) flush_queues<1>(lists, q_key, kTileM, q_cnt, n_pad, ew, k, thr_s, lane, c0);
          else if (kk == 64) flush_queues<2>(lists, q_key, kTileM, q_cnt, n_pad, ew, k, thr_s, lane, c0);
          else flush_queues<4>(lists, q_key, kTileM, q_cnt, n_pad, ew, k, thr_s, lane, c0);
          epilogue_bar();
        }
      }
      }
      // the tile's candidates, into the lists (the last round's barrier has seen them queued)
      if (kk == 32) flush_queues<1>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
      else if (kk == 64) flush_queues<2>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
      else flush_queues<4>(lists, q_key, q_cap, q_cnt, n_pad, ew, k, thr_s, lane);
      epilogue_bar();
      // The agreed bound tightens like 1/t: after the first tiles every fourth exchange is enough
      // (not behind a CTA's last tile: nothing of its own is left to filter, and the others
      // are at their last tiles too)
      if (use_xchg && (iter < 4 || (iter & 3u) == 3u) && tile + n_units < n_tiles) {
        // publish this CTA's best per query (the owner warp's lists are quiescent here) ...
        for (int q = ew + 4 * lane; q < nq_c; q += 128) {
          const u64 top = lists.load(q, 0);
          if (top != 0) __stcg(&lmax[(size_t)(q0 + q) * kTcMaxCtas + blockIdx.x], candidate_score(top));
        }
        // ... and, for the queries this CTA is responsible for, agree on the bound: the k-th
        // largest of all CTAs' bests, by k rounds of warp-wide maximum extraction
        const int q_first = (((int)blockIdx.x - q0) % (int)gridDim.x + (int)gridDim.x) % (int)gridDim.x;
        for (int j = 0, q = q_first; q < nq_c; ++j, q += (int)gridDim.x) {
          if ((j & 3) != ew) continue;                                    // warp-uniform
          const float kth_best = kth_largest_best(lmax, q0 + q, k, lane);
          if (lane == 0 && kth_best > -INFINITY && kth_best > __ldcg(&gthr[q0 + q]))
            __stcg(&gthr[q0 + q], kth_best);
        }
      }
    }
    // publish this CTA's per-query lists: already descending, empty slots are 0 (lists
    // kept in global memory are in place already)
    epilogue_bar();
    if (!lists.global) {
      for (int i = et; i < nq_c * kk; i += 128) {
        const int q = i / kk, j = i - q * kk;
        partial[((size_t)blockIdx.x * nq_total + (q0 + q)) * kk + j] = lists.load(q, j);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  // a pair: neither CTA goes away, nor is TMEM freed, while the other may still read this
  // CTA's shared memory, count on its barriers or run MMAs into its TMEM
  if (kPair) cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    if (kPair)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                   ::"r"(tmem_base), "r"((uint32_t)tmem_cols) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                   ::"r"(tmem_base), "r"((uint32_t)tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------ host side ---
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) ==
            cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// Tensor map over a row-major bf16 matrix [rows, d]; box = 64 elements x box_rows rows,
// 128B swizzle, out-of-range elements read as zero.
static bool make_bf16_map(CUtensorMap* map_out, const void* base, int64_t rows, int32_t d,
                          int32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map over a row-major matrix of E4M3 codes [rows, d]; box = 64 codes x 128 rows as they
// are (no swizzle: the codes are read back with plain loads), out-of-range codes read as zero.
static bool make_code_map(CUtensorMap* map_out, const void* base, int64_t rows, int32_t d) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d};
  cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map_out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)base, dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor maps of one pool: keys (fixed at creation: the map covers the whole capacity,
// rows past the current size are masked in the epilogue) and, made on first use, the
// normalised-query buffer for every box height.
struct TcCache {
  const void* qn;
  int64_t qn_rows;
  int32_t d;
  bool fp8;               // the keys are E4M3 codes (key_map covers bytes, the queries are f16)
  alignas(64) CUtensorMap key_map;
  alignas(64) CUtensorMap q_map[OILBIRD_MAX_NQ / 16];          // [n_pad / 16 - 1]
  bool q_ok[OILBIRD_MAX_NQ / 16];
  size_t pairs_smem;      // CTA pairs that fit the device at this much shared memory (the last
  int pairs;              // answer; kept per pool, whose calls are the caller's to serialise)
};

TcCache* tc_cache_create(const void* keys, int64_t capacity, int32_t d, const void* qn,
                         int64_t qn_rows, bool fp8) {
  TcCache* c = new (std::nothrow) TcCache();
  if (!c) return nullptr;
  c->qn = qn; c->qn_rows = qn_rows; c->d = d; c->fp8 = fp8;
  c->pairs_smem = 0; c->pairs = 0;
  for (bool& b : c->q_ok) b = false;
  if (!(fp8 ? make_code_map(&c->key_map, keys, capacity, d)
            : make_bf16_map(&c->key_map, keys, capacity, d, kTileM))) {
    delete c;
    return nullptr;
  }
  // every box height a query of this pool can ask for, encoded now: nothing is left to do
  // on the first call that uses one
  for (int n_pad = 16; n_pad <= OILBIRD_MAX_NQ && n_pad <= qn_rows; n_pad += 16)
    c->q_ok[n_pad / 16 - 1] = make_bf16_map(&c->q_map[n_pad / 16 - 1], qn, qn_rows, d, n_pad);
  return c;
}

void tc_cache_destroy(TcCache* c) { delete c; }

static const CUtensorMap* tc_q_map(TcCache* c, int n_pad) {
  const int slot = n_pad / 16 - 1;
  return (slot >= 0 && slot < OILBIRD_MAX_NQ / 16 && c->q_ok[slot]) ? &c->q_map[slot] : nullptr;
}

static size_t tc_fixed_smem(int nq_c, int n_pad, int kk, bool global_lists) {
  return (global_lists ? 0 : (size_t)nq_c * kk * 8) + (size_t)kQueueCap * 8 +
         (size_t)n_pad * (8 + 4 + 4 + 4) + 1024 /* alignment slack */;
}

// How a call is cut up: queries per pass, where the lists live, key tiles per query tile,
// ring stages, accumulator buffers.  With the lists in global memory any call (256 queries,
// k = 128) fits one pass over the keys.
struct TcPlan { int per_pass, n_pad, mt, stages, n_bufs, global_lists, pair; };

static bool tc_fits(int n, int kk, int mt, bool global_lists, int min_stages, size_t smem_limit,
                    int* stages, bool pair = false, bool fp8 = false) {
  const size_t stage = (size_t)mt * (kATileBytes + (fp8 ? kCodeTileBytes : 0)) +
                       (size_t)(pair ? n / 2 : n) * kBlockK * 2;
  // static shared memory (barriers etc.) is padded to the 1024-byte alignment of the ring
  const size_t fixed = tc_fixed_smem(n, n, kk, global_lists) + 1024 + 256;
  if (fixed + (size_t)min_stages * stage > smem_limit) return false;
  int st = (int)((smem_limit - fixed) / stage);
  *stages = st > kMaxStages ? kMaxStages : st;
  return true;
}

constexpr int kPairMinNq = 96;   // batches above this many queries go to CTA pairs
static TcPlan tc_plan_single(int nq, int k, int n_tiles128, int num_sms, size_t smem_limit,
                             bool fp8 = false);

static TcPlan tc_plan(int nq, int k, int n_tiles128, int num_sms, size_t smem_limit,
                      bool fp8 = false) {
  if (fp8) return tc_plan_single(nq, k, n_tiles128, num_sms, smem_limit, true);   // lone CTAs only
  // Around a hundred queries and more on a large pool: two CTAs per tile of 256 rows (see the
  // kernel); each loads half of the query rows, so their number is a multiple of 32.  Up to
  // 128 queries the accumulators leave room for two such tiles per query tile (a macro tile
  // of 512 rows), which is what makes the pair pay there: C4 at nq = 128 1.58 ms against
  // 1.635 for one CTA per two tiles, nq = 96 1.465 against 1.48, both under the power cap at
  // ~980 MHz; one tile per pair was slower than either (1.75 ms).
  if (nq > kPairMinNq && num_sms >= 2) {
    TcPlan p;
    p.per_pass = OILBIRD_MAX_NQ;
    p.n_pad = (nq + 31) / 32 * 32;
    p.pair = 1; p.global_lists = 1; p.stages = 0;
    // two tiles per CTA and query tile: with both accumulator sets up to 128 columns, with
    // one set above (what the shared query tile saves outweighs the epilogue no longer
    // overlapping the MMAs: C5 nq = 160 3.94 -> 3.63 ms, nq = 192 4.20 -> 3.93, nq = 224
    // 4.46 -> 4.35; at 256 columns it did not, 4.72 -> 4.71, until the epilogue folded its
    // candidates once per tile: 4.66 -> 4.48 ms)
    if (p.n_pad <= 256 && n_tiles128 >= 8 * num_sms) {
      p.mt = 2;
      p.n_bufs = 2 * 2 * p.n_pad <= 512 ? 2 : 1;
      if (tc_fits(p.n_pad, list_len(k), 2, true, 3, smem_limit, &p.stages, true)) return p;
    }
    // one tile per CTA: pays above 128 columns only (below, the lone CTA with two tiles is
    // faster: half the bytes per barrier round here)
    if (p.n_pad > 128 && n_tiles128 >= 4 * num_sms) {
      p.mt = 1; p.n_bufs = 2; p.stages = 0;
      if (tc_fits(p.n_pad, list_len(k), 1, true, 3, smem_limit, &p.stages, true)) return p;
    }
  }
  return tc_plan_single(nq, k, n_tiles128, num_sms, smem_limit);
}

static TcPlan tc_plan_single(int nq, int k, int n_tiles128, int num_sms, size_t smem_limit,
                             bool fp8) {
  const int kk = list_len(k);
  TcPlan p;
  p.per_pass = OILBIRD_MAX_NQ;
  const int n_pad = (nq + 15) / 16 * 16;
  int st = 0;
  p.pair = 0;
  p.n_pad = n_pad;
  // Sharing a query tile between two key tiles pays at every nq measured (fewer, larger
  // stages and half the query bytes from L2), given enough tiles to keep every SM busy and
  // room for both tiles' accumulators twice (a second accumulator set lets the next tile's
  // MMAs overlap this tile's epilogue).  Then the lists: in shared memory while the ring
  // beside them keeps its depth, else in global memory; a deep ring of two-tile stages with
  // the lists in L2 beats a shallower or one-tile ring with the lists on chip (nq = 128,
  // k = 64 at d = 8192: 2.61 ms against 3.11).
  const bool many_tiles = n_tiles128 >= 2 * num_sms;
  const bool two = many_tiles && 2 * 2 * n_pad <= 512 &&
                   tc_fits(n_pad, kk, 2, true, 3, smem_limit, &st, false, fp8);
  const int mt = two ? 2 : 1;
  const bool gl = !tc_fits(n_pad, kk, mt, false, kTcMinSmemStages, smem_limit, &st, false, fp8);
  p.global_lists = gl ? 1 : 0;
  p.mt = mt;
  p.stages = 0;
  tc_fits(n_pad, kk, p.mt, gl, 2, smem_limit, &p.stages, false, fp8);
  p.n_bufs = 2 * p.mt * n_pad <= 512 ? 2 : 1;
  return p;
}

int tc_queries_per_pass(int nq, int k, int n_rows, int num_sms, size_t smem_limit, bool fp8) {
  return tc_plan(nq, k, (n_rows + kTileM - 1) / kTileM, num_sms, smem_limit, fp8).per_pass;
}

// CTA pairs that can be resident at once for a given amount of dynamic shared memory
// (remembered in the pool's cache: the answer only depends on the device and the size).
static int max_pairs(TcCache* cache, size_t smem, int num_sms) {
  if (cache->pairs_smem == smem && cache->pairs > 0) return cache->pairs;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(num_sms / 2 * 2);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, scan_tc_kernel<true>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cache->pairs_smem = smem;
  cache->pairs = n;
  return n;
}

cudaError_t launch_scan_tc(TcCache* cache, const PoolView& pv, int32_t q0, int32_t nq_c,
                           int32_t nq_total, int32_t k, int32_t kk, const uint64_t* exclude_tag,
                           unsigned long long* partial, DeviceStats* stats, float* xchg,
                           int32_t num_sms, size_t smem_limit, int32_t* n_lists,
                           const float* scales, cudaStream_t st) {
  const int n_tiles128 = (pv.n_rows + kTileM - 1) / kTileM;
  const bool fp8 = cache->fp8;
  if (fp8 != (scales != nullptr)) return cudaErrorInvalidValue;
  TcPlan plan = tc_plan(nq_c, k, n_tiles128, num_sms, smem_limit, fp8);
  for (int attempt = 0; attempt < 2; ++attempt) {
    const int n_pad = plan.n_pad;
    const size_t stage = (size_t)plan.mt * (kATileBytes + (fp8 ? kCodeTileBytes : 0)) +
                         (size_t)(plan.pair ? n_pad / 2 : n_pad) * kBlockK * 2;
    const size_t fixed = tc_fixed_smem(nq_c, n_pad, kk, plan.global_lists != 0);
    if (plan.stages < 2) return cudaErrorInvalidConfiguration;
    const CUtensorMap* q_map = tc_q_map(cache, plan.pair ? n_pad / 2 : n_pad);
    if (!q_map) return cudaErrorInvalidValue;
    size_t smem = fixed + (size_t)plan.stages * stage;
    if (smem < 120 * 1024) smem = 120 * 1024;   // one CTA per SM: TMEM is allocated per CTA
    int tmem_cols = 32;
    while (tmem_cols < plan.n_bufs * plan.mt * n_pad) tmem_cols <<= 1;
    if (plan.pair) {
      const int pairs_fit = max_pairs(cache, smem, num_sms);
      if (pairs_fit < num_sms / 2 - 2) {        // the device will not seat (nearly) every SM in a pair
        plan = tc_plan_single(nq_c, k, n_tiles128, num_sms, smem_limit);
        continue;
      }
      const int n_tiles = (n_tiles128 + 2 * plan.mt - 1) / (2 * plan.mt);
      int pairs = n_tiles < pairs_fit ? n_tiles : pairs_fit;
      if (pairs > num_sms / 2) pairs = num_sms / 2;
      *n_lists = 2 * pairs;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(2 * pairs);
      cfg.blockDim = dim3(kTcThreads);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = st;
      cudaLaunchAttribute attr[2];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = (!tl_pdl_off && pdl_process_ok()) ? 2 : 1;
      return cudaLaunchKernelEx(&cfg, scan_tc_kernel<true>, cache->key_map, *q_map, pv, (int)q0,
                                (int)nq_c, (int)nq_total, n_pad, (int)k, (int)kk, plan.stages,
                                tmem_cols, plan.mt, plan.n_bufs, plan.global_lists, exclude_tag,
                                (u64*)partial, stats, xchg, (const float*)nullptr);
    }
    const int n_tiles = (n_tiles128 + plan.mt - 1) / plan.mt;
    int grid = n_tiles < num_sms ? n_tiles : num_sms;
    if (grid < 1) grid = 1;
    *n_lists = grid;
    if (fp8)
      return launch_pdl(scan_tc_kernel<false, true>, dim3(grid), dim3(kTcThreadsFp8), smem, st,
                        cache->key_map, *q_map, pv, q0, nq_c, nq_total, n_pad, k, kk, plan.stages,
                        tmem_cols, plan.mt, plan.n_bufs, plan.global_lists, exclude_tag, partial,
                        stats, xchg, scales);
    return launch_pdl(scan_tc_kernel<false>, dim3(grid), dim3(kTcThreads), smem, st,
                      cache->key_map, *q_map, pv, q0, nq_c, nq_total, n_pad, k, kk, plan.stages,
                      tmem_cols, plan.mt, plan.n_bufs, plan.global_lists, exclude_tag, partial, stats,
                      xchg, (const float*)nullptr);
  }
  return cudaErrorInvalidConfiguration;
}

// The three kinds of bounded wait on things that never happen (see launch_stall_selftest).
__global__ void __launch_bounds__(64)
stall_selftest_kernel(const unsigned long long* ready, DeviceStats* stats, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  __shared__ unsigned never_raised;
  pdl_enter();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    never_raised = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    // a row counter that nobody advances: the target is one past whatever it holds
    wait_fused_rows(ready, ld_acquire_u64(ready) + 1ull, stats);
  } else if (threadIdx.x == 32) {
    // phase 0 of a barrier nobody arrives at never completes
    const bool ok = mbar_wait(&bar, 0, &abort_flag, stats);
    if (gave_up) *gave_up = ok ? 0 : 1;
  } else if (threadIdx.x == 33) {
    // a flag word that no CTA raises (the index lookup's hand-over of the probes)
    wait_flag_u32(&never_raised, stats);
  }
}

cudaError_t launch_stall_selftest(const unsigned long long* ready, DeviceStats* stats,
                                  cudaStream_t st) {
  return launch_pdl(stall_selftest_kernel, dim3(1), dim3(64), 0, st, ready, stats, (int*)nullptr);
}

cudaError_t preload_scan_tc_kernels() {
  cudaError_t e = preload_kernel(scan_tc_kernel<false>, true);
  if (e == cudaSuccess) e = preload_kernel(scan_tc_kernel<true>, true);
  if (e == cudaSuccess) e = preload_kernel(scan_tc_kernel<false, true>, true);
  return e != cudaSuccess ? e : preload_kernel(stall_selftest_kernel);
}

}  // namespace oilbird

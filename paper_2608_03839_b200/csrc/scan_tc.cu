// K3: tensor-core scan for batched queries (many requests against one shared pool).
//
// Scoring line of Algorithm 1 (cosine of the query with every stored state) for nq queries at
// once: S[i, q] = <key_i, qn_q> is a [N x d] x [d x nq] contraction.  Keys are the M
// operand (tiles of 128 rows), the normalised queries the N operand (nq padded to a
// multiple of 16), d is walked in blocks of 64 elements.  Each CTA is persistent and
// warp-specialised:
//   warp 0      TMA producer: key tile + query tile per k-block into a 128B-swizzled
//               shared-memory ring (cp.async.bulk.tensor, mbarrier complete_tx)
//   warp 1      tcgen05.mma issuer (one thread), fp32 accumulators in TMEM, two
//               accumulator buffers so the next tile's MMAs overlap the epilogue
//   warps 2-5   epilogue: tcgen05.ld the 128 x nq scores, filter them against the
//               per-query running k-th best, and keep per-query top-k lists in shared
//               memory (Eq. 2); scores never go to global memory
// The key stream (N*d*2 bytes from HBM, once) bounds the kernel up to nq ~ 64-96; the
// epilogue warps then wait for accumulators 60-80 % of the time.  What is left above that:
//   - a CTA's first one or two macro tiles, whose scores nearly all pass the still-low
//     thresholds (sorted 32 at a time and merged): ~2.5 tiles' worth of time at nq = 128,
//     during which the accumulator buffers are full and the key stream stalls;
//   - at nq = 256 the query tile re-read from L2 per key tile (twice the key bytes) and the
//     single k-block per accumulator set; the tensor pipe reaches about half its peak.
// Small pools (a few tiles per SM): a query costs about 40 us plus the key bytes at HBM
// speed, against 12 us plus the same for the CUDA-core scan.  A tile's scores exist only
// after its whole K loop, so the first tile's latency chain is not overlapped, and one SM
// streams at most ~45-65 GB/s whatever the rest of the GPU does: cycle counters in the
// MMA-issuing thread show ~360 cycles to issue the four tcgen05.mma and the commit of a
// 16 KB k-block (~70 cycles per instruction, against ~90 cycles of waiting for the data
// when HBM is idle), i.e. with queries as the N operand a 128 x N x 16 instruction carries
// only 4 KB of keys and the issue rate, not the tensor pipe, bounds the per-SM rate.  Then
// come the first tile's epilogue (7-10 us), the query normalisation kernel and the merge.
// A variant with the roles swapped (queries as M = 128, one query per TMEM lane and per
// epilogue thread with its threshold in a register and a queue only it writes; 256 key rows
// as N, so that an instruction carries 8 KB of keys) was written and passes the same tests,
// but is slower everywhere: 0.90 instead of 1.03 of the measured HBM rate at nq = 16 and
// 0.73 instead of 0.81 at nq = 128 on the 8.6 GB pool (every stage carries a 16 KB query
// tile whatever nq is), and 2-3x slower on small pools, where only nq/32 of the four
// epilogue warps share the sorting of a CTA's first tile.  Cutting the pool into per-CTA row ranges at 32-row granularity
// (ragged ends fetched as 32-row boxes) so that all SMs get equal rows, ring depths up to
// 12 and seeding the first tile's thresholds from per-warp 32-bit sorts of the scores were
// measured and bring nothing.
// Measured and not kept: separate shared-memory rings for keys and query tiles (query
// tiles queue behind the key requests, so they need the same lead; 5-8 % slower); a
// 32-deep candidate queue with retry, to buy a ring stage (slower first tiles, no gain from
// the stage); ballot-packed per-warp queue segments instead of shared-memory atomics (drain
// 60 % slower); sorting every column of the first tile in registers without the queue (no
// faster than the queue's crowd path); a variant that transposes the scores through shared
// memory so that one warp owns a query's 128 rows (15-30 % slower).
//
// Every mbarrier wait is bounded: after about two seconds it raises the pool's `stalled`
// flag, the CTA drains what it has in flight, frees its TMEM and returns.
#include <cuda.h>

#include <new>

#include "common.cuh"
#include "internal.h"

namespace oilbird {

constexpr int kTcThreads = 192;
constexpr int kTileM = 128;            // key rows per tile = TMEM lanes
// bf16 elements per k-block = one 128-byte swizzle row.  (32-element blocks with the 64-byte
// swizzle were measured too: more, finer ring stages, but every 128-byte line is then
// requested twice and the scan runs 30-40 % slower at every nq.)
constexpr int kBlockK = 64;
constexpr int kATileBytes = kTileM * kBlockK * 2;   // 16 KB
constexpr int kColsPerRound = 16;      // score columns filtered between two drains
constexpr int kQueueCap = kTileM * kColsPerRound;
constexpr int kMaxStages = 8;

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
// Bounded wait.  Returns false if it gave up (or another role already did).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStats* stats) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns(), limit = wait_limit_ns(stats);
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
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
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
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
// Instruction descriptor: D fp32, A/B bf16, both K-major, M=128, N=n.
__host__ __device__ inline uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kTileM >> 4) << 24);
}

// ------------------------------------------------------------- per-query lists ---
struct TcShared {
  uint64_t full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], drain;
  uint32_t tmem_base;
  int abort_flag;
  int epi_go;
  int q_total;                  // nonzero: candidates were queued in the current round
  int q_cnt[kColsPerRound];     // ... per score column of the round
};

// Per-query candidate lists in shared memory.  Wide form: one packed 64-bit key per slot.
// Compact form (6 bytes per slot: fp32 score + 16-bit position), chosen when it lets a call
// run in fewer passes over the keys: a CTA's rows are numbered locally, its it-th macro tile
// holding local rows [it*rows_per_tile, (it+1)*rows_per_tile), so 16 bits cover the 65,536
// rows one CTA scans in pools of up to ~9.7 million rows.  An empty slot is key 0 / -inf.
struct ListStore {
  u64* wide;
  float* sc;
  uint16_t* loc;
  int kk, shift;          // rows per macro tile = 1 << shift
  bool compact;

  __device__ __forceinline__ u64 load(int q, int i) const {
    if (!compact) return wide[(size_t)q * kk + i];
    const float s = sc[(size_t)q * kk + i];
    if (s == -INFINITY) return 0;
    const uint32_t l = loc[(size_t)q * kk + i];
    const uint32_t tile = blockIdx.x + (l >> shift) * gridDim.x;
    return pack_candidate(s, (tile << shift) | (l & ((1u << shift) - 1u)));
  }
  __device__ __forceinline__ void store(int q, int i, u64 key) const {
    if (!compact) { wide[(size_t)q * kk + i] = key; return; }
    if (key == 0) { sc[(size_t)q * kk + i] = -INFINITY; loc[(size_t)q * kk + i] = 0; return; }
    const uint32_t row = (uint32_t)candidate_row(key);
    const uint32_t it = ((row >> shift) - blockIdx.x) / gridDim.x;
    sc[(size_t)q * kk + i] = candidate_score(key);
    loc[(size_t)q * kk + i] = (uint16_t)((it << shift) | (row & ((1u << shift) - 1u)));
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
__device__ __forceinline__ void drain_round(const ListStore& lists, int kk, const u64* q_key,
                                            const int* q_cnt, int c0, int ew, int nq_c, int k,
                                            float* thr_s, int lane) {
  u64 v[kDrainQ][E];
  u64 kth[kDrainQ];
  int n[kDrainQ];
  int n_max = 0, crowd_max = 0;
#pragma unroll
  for (int u = 0; u < kDrainQ; ++u) {
    const int j = ew + 4 * u, q = c0 + j;
    n[u] = q < nq_c ? q_cnt[j] : 0;
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
        const u64 key = (n[u] >= kCrowd && i < n[u]) ? q_key[(ew + 4 * u) * kTileM + i] : 0;
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
      u64 key = (n[u] < kCrowd && i < n[u]) ? q_key[(ew + 4 * u) * kTileM + i] : 0;
      key = key > kth[u] ? key : 0;
      warp_sorted_insert<E>(v[u], key, lane);
    }
  }
#pragma unroll
  for (int u = 0; u < kDrainQ; ++u) {
    if (n[u] > 0) {
      const int q = c0 + ew + 4 * u;
#pragma unroll
      for (int r = 0; r < E; ++r) lists.store(q, r * 32 + lane, v[u][r]);
      const u64 nk = warp_list_get<E>(v[u], k - 1);
      // never below a bound adopted from the other CTAs
      if (lane == 0 && nk != 0) thr_s[q] = fmaxf(thr_s[q], candidate_score(nk));
    }
  }
}

// ------------------------------------------------------------------- the kernel ---
// Queries [q0, q0+nq_c) of the call; n_pad = nq_c rounded up to 16 = MMA N.
// mt (1 or 2) key tiles of 128 rows share each query tile: with mt = 2 the query bytes
// pulled from L2 per key byte halve, which is what limits the kernel from nq ~ 64 up.
// n_bufs accumulator sets of mt*n_pad TMEM columns each (2 = the next macro tile's MMAs
// overlap the epilogue; 1 when 2*mt*n_pad would exceed the 512 columns).
__global__ void __launch_bounds__(kTcThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap key_map,
               const __grid_constant__ CUtensorMap q_map, PoolView pv, int q0, int nq_c,
               int nq_total, int n_pad, int k, int kk, int n_stages, int tmem_cols, int mt,
               int n_bufs, int compact, const uint64_t* __restrict__ exclude_tag,
               u64* __restrict__ partial, DeviceStats* stats, float* xchg) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ TcShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int a_bytes = mt * kATileBytes;
  const int stage_bytes = a_bytes + n_pad * kBlockK * 2;
  // dynamic shared memory: [stages][mt key tiles | query tile] | lists | queue | state
  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = base;
  unsigned char* list_mem = ring + (size_t)n_stages * stage_bytes;              // [nq_c][kk]
  ListStore lists;
  lists.wide = reinterpret_cast<u64*>(list_mem);
  lists.sc = reinterpret_cast<float*>(list_mem);
  lists.loc = reinterpret_cast<uint16_t*>(list_mem + (size_t)nq_c * kk * 4);
  lists.kk = kk;
  lists.shift = mt == 2 ? 8 : 7;
  lists.compact = compact != 0;
  u64* q_key = reinterpret_cast<u64*>(list_mem + (size_t)nq_c * kk * (compact ? 6 : 8));
                                                               // [kColsPerRound][kTileM]
  uint64_t* s_ex = reinterpret_cast<uint64_t*>(q_key + kQueueCap);              // [n_pad]
  float* thr_s = reinterpret_cast<float*>(s_ex + n_pad);                        // [n_pad]
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
  const bool use_xchg = (int)gridDim.x >= k && (int)gridDim.x <= kTcMaxCtas;

  const int n_tiles = (pv.n_rows + mt * kTileM - 1) / (mt * kTileM);   // macro tiles
  const int n_kb = (pv.d + kBlockK - 1) / kBlockK;
  volatile int* abort_flag = &sh.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sh.tmem_full[b], 1); mbar_init(&sh.tmem_empty[b], 4); }
    mbar_init(&sh.drain, 1);
    sh.abort_flag = 0;
    sh.q_total = 0;
    for (int j = 0; j < kColsPerRound; ++j) sh.q_cnt[j] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation is a whole-warp operation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&sh.tmem_base)), "r"((uint32_t)tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  pdl_enter();   // appended rows, normalised queries, exclusion tags; set-up above overlapped
  for (int i = threadIdx.x; i < n_pad; i += kTcThreads) {
    thr_s[i] = i < nq_c ? -INFINITY : INFINITY;        // padded columns never pass the filter
    s_ex[i] = (exclude_tag && i < nq_c) ? exclude_tag[q0 + i] : 0;
  }
  for (int i = threadIdx.x; i < nq_c * kk; i += kTcThreads) lists.store(i / kk, i % kk, 0);
  __syncthreads();

  if (warp == 0) {
    // ===================================================== TMA producer ==========
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&key_map) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          const uint32_t ph = (it / n_stages) & 1u;
          if (!mbar_wait(&sh.empty[s], ph ^ 1u, abort_flag, stats)) { ok = false; break; }
          unsigned char* a_dst = ring + (size_t)s * stage_bytes;
          mbar_arrive_expect_tx(&sh.full[s], (uint32_t)stage_bytes);
          for (int sub = 0; sub < mt; ++sub)    // rows past the pool's capacity read as zero
            tma_load_2d(a_dst + sub * kATileBytes, &key_map, kb * kBlockK,
                        (tile * mt + sub) * kTileM, &sh.full[s]);
          tma_load_2d(a_dst + a_bytes, &q_map, kb * kBlockK, q0, &sh.full[s]);
        }
      }
      if (!ok) {
        // gave up: let the copies already issued land before the CTA's memory goes away
        const uint32_t back = it < (uint32_t)n_stages ? it : (uint32_t)n_stages;
        for (uint32_t j = 0; j < back; ++j) {
          const uint32_t i2 = it - 1 - j;
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&sh.full[i2 % n_stages], (i2 / n_stages) & 1u) &&
                 global_ns() - t0 < 2000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================== MMA issuer ============
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(n_pad);
      uint32_t it = 0, iter = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++iter) {
        const uint32_t buf = iter % (uint32_t)n_bufs;
        if (!mbar_wait(&sh.tmem_empty[buf], ((iter / (uint32_t)n_bufs) & 1u) ^ 1u, abort_flag,
                       stats)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * (uint32_t)(mt * n_pad);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          if (!mbar_wait(&sh.full[s], (it / n_stages) & 1u, abort_flag, stats)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(ring + (size_t)s * stage_bytes);
          const uint64_t b_desc = umma_desc_sw128(a_addr + a_bytes);
          for (int sub = 0; sub < mt; ++sub) {
            const uint64_t a_desc = umma_desc_sw128(a_addr + sub * kATileBytes);
#pragma unroll
            for (int kq = 0; kq < kBlockK / 16; ++kq)      // 32 bytes along K per MMA
              tc_mma_bf16(d_tmem + (uint32_t)(sub * n_pad), a_desc + (uint64_t)(kq * 2),
                          b_desc + (uint64_t)(kq * 2), idesc, (kb | kq) != 0 ? 1u : 0u);
          }
          tc_commit(&sh.empty[s]);                          // stage reusable once the MMAs retire
        }
        if (ok) tc_commit(&sh.tmem_full[buf]);
      }
      // nothing may still be writing TMEM when it is freed
      tc_commit(&sh.drain);
      const unsigned long long t0 = global_ns();
      const unsigned long long limit = wait_limit_ns(stats);
      while (!mbar_try_wait(&sh.drain, 0) && global_ns() - t0 < limit) {}
    }
  } else {
    // ===================================================== epilogue ==============
    const int ew = warp - 2;                    // 0..3: which queries this warp owns in drains
    const int lane_grp = warp & 3;              // TMEM lanes this warp may read
    const int et = threadIdx.x - 64;            // 0..127
    uint32_t iter = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++iter) {
      const uint32_t buf = iter % (uint32_t)n_bufs;
      mbar_wait(&sh.tmem_full[buf], (iter / (uint32_t)n_bufs) & 1u, abort_flag, stats);
      // one decision for all four warps, so that the barriers below always match up
      epilogue_bar();
      if (et == 0) sh.epi_go = *abort_flag ? 0 : 1;
      if (use_xchg) {
        // adopt the agreed bounds: v > max(local, prev(g))  <=>  v > local and v >= g
        for (int q = et; q < nq_c; q += 128) {
          const float g = __ldcg(&gthr[q0 + q]);
          if (g > -INFINITY) thr_s[q] = fmaxf(thr_s[q], nextafterf(g, -INFINITY));
        }
      }
      epilogue_bar();
      if (!sh.epi_go) { ok = false; break; }
      tc_fence_after();
      for (int sub = 0; sub < mt; ++sub) {      // sub-tiles in row order: ties stay exact
      const int row = (tile * mt + sub) * kTileM + lane_grp * 32 + lane;
      const bool row_ok = row < pv.n_rows;
      uint64_t tag = 0;
      if (exclude_tag && row_ok) tag = pv.trace_tag[pv.trace_id[row]];
      const uint32_t t_row = tmem_base + ((uint32_t)(lane_grp * 32) << 16) +
                             (buf * (uint32_t)mt + (uint32_t)sub) * (uint32_t)n_pad;
      for (int c0 = 0; c0 < n_pad; c0 += kColsPerRound) {
        float v[kColsPerRound];
        tc_ld16(t_row + (uint32_t)c0, v);
        if (sub == mt - 1 && c0 + kColsPerRound >= n_pad) {
          // all of this macro tile's scores have been read: hand the accumulators back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.tmem_empty[buf]);
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
        while (pass) {
          const int j = (__ffs(pass) - 1 + rot) & (kColsPerRound - 1);
          pass &= pass - 1;
          const int q = c0 + j;
          if (s_ex[q] != 0 && tag == s_ex[q]) continue;           // same-prompt trace: skipped
          float vj = v[0];
#pragma unroll
          for (int i = 1; i < kColsPerRound; ++i) vj = j == i ? v[i] : vj;
          const int pos = atomicAdd(&sh.q_cnt[j], 1);
          q_key[j * kTileM + pos] = pack_candidate(vj, (uint32_t)row);
          sh.q_total = 1;
        }
        epilogue_bar();
        if (sh.q_total > 0) {
          // drain: warp ew folds the candidates of columns ew, ew+4, ... into their lists
          if (kk == 32) drain_round<1>(lists, kk, q_key, sh.q_cnt, c0, ew, nq_c, k, thr_s, lane);
          else if (kk == 64) drain_round<2>(lists, kk, q_key, sh.q_cnt, c0, ew, nq_c, k, thr_s, lane);
          else drain_round<4>(lists, kk, q_key, sh.q_cnt, c0, ew, nq_c, k, thr_s, lane);
          __syncwarp();
          if (lane < kDrainQ) sh.q_cnt[ew + 4 * lane] = 0;
          epilogue_bar();
          if (et == 0) sh.q_total = 0;
          epilogue_bar();
        }
      }
      }
      // The agreed bound tightens like 1/t: after the first tiles every fourth exchange is enough
      if (use_xchg && (iter < 4 || (iter & 3u) == 3u)) {
        // publish this CTA's best per query (the owner warp's lists are quiescent here) ...
        for (int q = ew + 4 * lane; q < nq_c; q += 128) {
          const u64 top = lists.load(q, 0);
          if (top != 0) __stcg(&lmax[(size_t)(q0 + q) * kTcMaxCtas + blockIdx.x], candidate_score(top));
        }
        // ... and, for the queries this CTA is responsible for, agree on the bound: the k-th
        // largest of all CTAs' bests, by k rounds of warp-wide maximum extraction
        for (int q = ew; q < nq_c; q += 4) {
          if ((q0 + q) % (int)gridDim.x != (int)blockIdx.x) continue;     // warp-uniform
          float mine[kTcMaxCtas / 32];
#pragma unroll
          for (int i = 0; i < kTcMaxCtas / 32; ++i) {
            const int c = i * 32 + lane;
            mine[i] = c < (int)gridDim.x ? __ldcg(&lmax[(size_t)(q0 + q) * kTcMaxCtas + c]) : -INFINITY;
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
          if (lane == 0 && kth_best > -INFINITY && kth_best > __ldcg(&gthr[q0 + q]))
            __stcg(&gthr[q0 + q], kth_best);
        }
      }
    }
    // publish this CTA's per-query lists: already descending, empty slots are 0
    epilogue_bar();
    for (int i = et; i < nq_c * kk; i += 128) {
      const int q = i / kk, j = i - q * kk;
      partial[((size_t)blockIdx.x * nq_total + (q0 + q)) * kk + j] = lists.load(q, j);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
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

// Tensor maps of one pool: keys (fixed at creation: the map covers the whole capacity,
// rows past the current size are masked in the epilogue) and, made on first use, the
// normalised-query buffer for every box height.
struct TcCache {
  const void* qn;
  int64_t qn_rows;
  int32_t d;
  alignas(64) CUtensorMap key_map;
  alignas(64) CUtensorMap q_map[OILBIRD_MAX_NQ / 16];          // [n_pad / 16 - 1]
  bool q_ok[OILBIRD_MAX_NQ / 16];
};

TcCache* tc_cache_create(const void* keys, int64_t capacity, int32_t d, const void* qn,
                         int64_t qn_rows) {
  TcCache* c = new (std::nothrow) TcCache();
  if (!c) return nullptr;
  c->qn = qn; c->qn_rows = qn_rows; c->d = d;
  for (bool& b : c->q_ok) b = false;
  if (!make_bf16_map(&c->key_map, keys, capacity, d, kTileM)) {
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

static size_t tc_fixed_smem(int nq_c, int n_pad, int kk, bool compact) {
  return (size_t)nq_c * kk * (compact ? 6 : 8) + (size_t)kQueueCap * 8 +
         (size_t)n_pad * (8 + 4) + 1024 /* alignment slack */;
}

// How a call is cut up: queries per pass, list format, key tiles per query tile, ring
// stages, accumulator buffers.  Fewest passes first (every pass re-reads the keys): the
// compact list format is taken when it saves a pass (two ring stages are then enough: ring
// depth was measured not to matter once the epilogue sets the pace); then two key tiles per
// query tile if at least three ring stages still fit, else one.
struct TcPlan { int per_pass, mt, stages, n_bufs, compact; };

static bool tc_fits(int n, int kk, int mt, bool compact, int min_stages, size_t smem_limit,
                    int* stages) {
  const size_t stage = (size_t)mt * kATileBytes + (size_t)n * kBlockK * 2;
  // static shared memory (barriers etc.) is padded to the 1024-byte alignment of the ring
  const size_t fixed = tc_fixed_smem(n, n, kk, compact) + 1024 + 256;
  if (fixed + (size_t)min_stages * stage > smem_limit) return false;
  int st = (int)((smem_limit - fixed) / stage);
  *stages = st > kMaxStages ? kMaxStages : st;
  return true;
}

static TcPlan tc_plan(int nq, int k, int n_tiles128, int num_sms, size_t smem_limit, int force_mt) {
  const int kk = list_len(k);
  int max_pass = 16, max_pass_c = 16, st = 0;
  for (int n = 16; n <= OILBIRD_MAX_NQ; n += 16) {
    if (tc_fits(n, kk, 1, false, 3, smem_limit, &st)) max_pass = n;
    if (tc_fits(n, kk, 1, true, 2, smem_limit, &st)) max_pass_c = n;
  }
  int n_pass = (nq + max_pass - 1) / max_pass;
  // 16-bit local positions: the rows one CTA scans must number at most 65,536
  const int grid = n_tiles128 < num_sms ? (n_tiles128 > 0 ? n_tiles128 : 1) : num_sms;
  const bool can_compact = ((int64_t)(n_tiles128 + grid - 1) / grid + 1) * kTileM <= 65536;
  TcPlan p;
  p.compact = 0;
  if (can_compact && (nq + max_pass_c - 1) / max_pass_c < n_pass) {
    p.compact = 1;
    n_pass = (nq + max_pass_c - 1) / max_pass_c;
  }
  const bool cp = p.compact != 0;
  p.per_pass = ((nq + n_pass - 1) / n_pass + 15) / 16 * 16;      // balanced passes
  const int n_pad = p.per_pass < nq ? p.per_pass : (nq + 15) / 16 * 16;
  // sharing a query tile between two key tiles pays at every nq measured (fewer, larger
  // stages and half the query bytes from L2), given enough tiles to keep every SM busy
  bool two = n_tiles128 >= 4 * num_sms && tc_fits(n_pad, kk, 2, cp, 3, smem_limit, &st);
  if (force_mt == 1) two = false;
  if (force_mt == 2) two = tc_fits(n_pad, kk, 2, cp, 2, smem_limit, &st);
  p.mt = two ? 2 : 1;
  tc_fits(n_pad, kk, p.mt, cp, 2, smem_limit, &p.stages);
  p.n_bufs = 2 * p.mt * n_pad <= 512 ? 2 : 1;
  return p;
}

int tc_queries_per_pass(int nq, int k, int n_rows, int num_sms, size_t smem_limit) {
  return tc_plan(nq, k, (n_rows + kTileM - 1) / kTileM, num_sms, smem_limit, 0).per_pass;
}

cudaError_t launch_scan_tc(TcCache* cache, const PoolView& pv, int32_t q0, int32_t nq_c,
                           int32_t nq_total, int32_t k, int32_t kk, const uint64_t* exclude_tag,
                           unsigned long long* partial, DeviceStats* stats, float* xchg,
                           int32_t num_sms, size_t smem_limit, int32_t* n_lists, cudaStream_t st) {
  const int n_pad = (nq_c + 15) / 16 * 16;
  const int n_tiles128 = (pv.n_rows + kTileM - 1) / kTileM;
  TcPlan plan = tc_plan(nq_c, k, n_tiles128, num_sms, smem_limit, 0);
  const size_t stage = (size_t)plan.mt * kATileBytes + (size_t)n_pad * kBlockK * 2;
  const size_t fixed = tc_fixed_smem(nq_c, n_pad, kk, plan.compact != 0);
  if (plan.stages < 2) return cudaErrorInvalidConfiguration;
  const CUtensorMap* q_map = tc_q_map(cache, n_pad);
  if (!q_map) return cudaErrorInvalidValue;
  size_t smem = fixed + (size_t)plan.stages * stage;
  if (smem < 120 * 1024) smem = 120 * 1024;   // one CTA per SM: TMEM is allocated per CTA
  int tmem_cols = 32;
  while (tmem_cols < plan.n_bufs * plan.mt * n_pad) tmem_cols <<= 1;
  const int n_tiles = (n_tiles128 + plan.mt - 1) / plan.mt;
  int grid = n_tiles < num_sms ? n_tiles : num_sms;
  if (grid < 1) grid = 1;
  *n_lists = grid;
  return launch_pdl(scan_tc_kernel, dim3(grid), dim3(kTcThreads), smem, st,
                    cache->key_map, *q_map, pv, q0, nq_c, nq_total, n_pad, k, kk, plan.stages,
                    tmem_cols, plan.mt, plan.n_bufs, plan.compact, exclude_tag, partial, stats,
                    xchg);
}

// Both kinds of bounded wait on things that never happen (see launch_stall_selftest).
__global__ void __launch_bounds__(64)
stall_selftest_kernel(const unsigned long long* ready, DeviceStats* stats, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  pdl_enter();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
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
  }
}

cudaError_t launch_stall_selftest(const unsigned long long* ready, DeviceStats* stats,
                                  cudaStream_t st) {
  return launch_pdl(stall_selftest_kernel, dim3(1), dim3(64), 0, st, ready, stats, (int*)nullptr);
}

cudaError_t preload_scan_tc_kernels() {
  cudaError_t e = preload_kernel(scan_tc_kernel, true);
  return e != cudaSuccess ? e : preload_kernel(stall_selftest_kernel);
}

}  // namespace oilbird

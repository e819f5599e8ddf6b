// K2: CUDA-core scan for one or two queries (single-request decode).
//
// Scoring line of Algorithm 1 (cosine of the query with every stored state), fused with the
// per-CTA part of Eq. 2's top-k: every stored key is streamed from HBM exactly once
// with 16-byte loads, multiplied against the normalised queries held in shared memory
// (bf16 x bf16 products accumulated in fp32), and each warp keeps its best rows in a
// descending register list (one shuffle-insertion per accepted row).  Scores never go
// to global memory; what leaves the CTA is one descending list of kk (= max(32, k
// rounded up to a power of two)) packed candidates per query.  The raw query states are
// normalised by every CTA itself (8-32 KB from L2), which saves a separate launch on
// the latency-critical path.
//
// The kernel is bound by the key stream (N*d*2 bytes); per 16 bytes of key a lane
// spends 8 integer unpack ops and 8*QT FMAs, well under the issue budget for QT <= 2.
// A plain streaming read of the same 537 MB (no arithmetic) takes 79-80 us with this
// access pattern and 78 us through a cp.async.bulk shared-memory ring, so the direct
// loads are kept.  Handing row groups out through a global ticket counter instead of the
// static split was measured 4 % slower (one hot atomic, no tail to win back).
#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"

namespace oilbird {

constexpr int kScanThreads = kNormThreads;
constexpr int kScanWarps = kScanThreads / 32;
template <int QT, int E>
__global__ void __launch_bounds__(kScanThreads, 2)
scan_gemv_kernel(PoolView pv, const uint16_t* __restrict__ q_raw, int nq, int k,
                 const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                 int32_t* __restrict__ q_valid, DeviceStats* stats, FusedAppend fa) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int KK = 32 * E;
  pdl_enter();   // the rows appended just before this query, and the query states themselves
  const int d = pv.d, n_chunks = d >> 3;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                       // [QT][n_chunks]
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)QT * d * 2);  // [warps][KK]
  __shared__ uint64_t s_ex[QT];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // contiguous, balanced share of the rows for this CTA; the fa.n CTAs that first append a
  // row of this step (~2.5 us) take 1/32 less than the others
  const int64_t n = pv.n_rows;
  const int64_t w_lo = 32ll * blockIdx.x - min((int)blockIdx.x, fa.n);
  const int64_t w_hi = 32ll * (blockIdx.x + 1) - min((int)blockIdx.x + 1, fa.n);
  const int64_t w_all = 32ll * gridDim.x - min((int)gridDim.x, fa.n);
  const int r_lo = (int)((n * w_lo) / w_all);
  const int r_hi = (int)((n * w_hi) / w_all);
  const uint4* keys4 = reinterpret_cast<const uint4*>(pv.keys);

  // the step's append (Section 4 "(i) Store", Eq. 1), one row per CTA
  if ((int)blockIdx.x < fa.n) {
    const int r = blockIdx.x;
    const int64_t row = (int64_t)fa.row0 + r;
    const int code = normalize_row<false>(fa.states + (size_t)r * d, fa.keys + row * d, d);
    if (threadIdx.x == 0) {
      fa.tok[row] = fa.tokens[r];
      fa.trace_id[row] = fa.trace;
      if (code != kRowOk) atomicAdd(&stats->degenerate_rows, 1ull);  // stored as a zero key
      if (r == 0) {
        fa.trace_end[fa.trace] = fa.row0 + fa.n;
        if (fa.set_tag) { fa.trace_tag[fa.trace] = fa.tag; fa.trace_gbase[fa.trace] = fa.gbase; }
      }
    }
    __threadfence();                   // this thread's part of the row, before the count
    __syncthreads();
    if (threadIdx.x == 0) {
      __threadfence();                 // cumulative: the whole CTA's row, as seen through the barrier
      atomicAdd(fa.ready, 1ull);
    }
  }
  bool fresh_ok = fa.n == 0;           // this warp has seen the appended rows arrive

  for (int q0 = 0; q0 < nq; q0 += QT) {
    __syncthreads();
    // query preparation: qs[q] = bf16(q / ||q||), exactly as a key is stored
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      uint16_t* dst = reinterpret_cast<uint16_t*>(qs + (size_t)q * n_chunks);
      if (q0 + q < nq) {
        const int code = normalize_row<true, 2>(q_raw + (size_t)(q0 + q) * d, dst, d);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
          q_valid[q0 + q] = code == kRowNonFinite ? 0 : 1;   // NaN/Inf: no neighbours
          if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
        }
      } else {
        for (int c = threadIdx.x; c < n_chunks; c += kScanThreads)
          qs[(size_t)q * n_chunks + c] = make_uint4(0, 0, 0, 0);
      }
    }
    if (threadIdx.x < QT)
      s_ex[threadIdx.x] = (exclude_tag && q0 + threadIdx.x < nq) ? exclude_tag[q0 + threadIdx.x] : 0;
    __syncthreads();

    // this warp's best rows so far, descending; kth = its k-th entry (0 while not full)
    u64 top[QT][E];
    u64 kth[QT];
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      kth[q] = 0;
#pragma unroll
      for (int r = 0; r < E; ++r) top[q][r] = 0;
    }

    for (int rb = r_lo + warp * kRowsPerIter; rb < r_hi; rb += kScanWarps * kRowsPerIter) {
      const uint4* rowp[kRowsPerIter];
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) {
        int row = rb + r < r_hi ? rb + r : r_hi - 1;      // clamp: result discarded below
        rowp[r] = keys4 + (size_t)row * n_chunks;
      }
      float acc[kRowsPerIter][QT];
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r)
#pragma unroll
        for (int q = 0; q < QT; ++q) acc[r][q] = 0.f;

      if (fa.n > 0 && rb + kRowsPerIter > fa.row0) {        // warp-uniform
        // rows of this step's append: wait (bounded) until all of them are in
        if (!fresh_ok) {
          wait_fused_rows(fa, stats);
          fresh_ok = true;
        }
        score_rows<QT, true>(rowp, qs, n_chunks, lane, acc);
      } else {
        score_rows<QT, false>(rowp, qs, n_chunks, lane, acc);
      }
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) {
        const int row = rb + r;
        if (row >= r_hi) break;                             // warp-uniform
        uint64_t tag = 0;
        if (exclude_tag) {
          // rows appended by this launch: their trace id and tag were written by another CTA
          // a moment ago, and this SM's L1 may hold the lines from before (it has read the
          // neighbouring rows' entries), so those are read through L2
          tag = (fa.n > 0 && row >= fa.row0) ? __ldcg(&pv.trace_tag[__ldcg(&pv.trace_id[row])])
                                             : pv.trace_tag[pv.trace_id[row]];
        }
#pragma unroll
        for (int q = 0; q < QT; ++q) {
          const float s = warp_sum(acc[r][q]);
          if (q0 + q >= nq) continue;
          if (s_ex[q] != 0 && tag == s_ex[q]) continue;     // same-prompt trace: skipped
          const u64 key = pack_candidate(s, (uint32_t)row);
          if (key > kth[q]) {
            warp_sorted_insert<E>(top[q], key, lane);
            kth[q] = warp_list_get<E>(top[q], k - 1);
          }
        }
      }
    }
    // merge the warps' lists of each query; warp 0 publishes the CTA's KK best, descending
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      if (q0 + q >= nq) break;
      block_merge_desc<E>(top[q], scratch, kScanWarps);
      if (threadIdx.x < 32) {
        u64* dst = partial + ((size_t)blockIdx.x * nq + (q0 + q)) * KK;
#pragma unroll
        for (int r = 0; r < E; ++r) dst[r * 32 + lane] = top[q][r];
      }
    }
  }
}

template <int QT, int E>
static cudaError_t launch_one(const PoolView& pv, const uint16_t* q_raw, int nq, int k,
                              const uint64_t* ex, u64* partial, int32_t* q_valid,
                              DeviceStats* stats, int grid, const FusedAppend& fa,
                              cudaStream_t st) {
  size_t smem = (size_t)QT * pv.d * 2 + (size_t)kScanWarps * 32 * E * sizeof(u64);
  return launch_pdl(scan_gemv_kernel<QT, E>, dim3(grid), dim3(kScanThreads), smem, st, pv, q_raw,
                    nq, k, ex, partial, q_valid, stats, fa);
}

template <int QT>
static cudaError_t launch_qt(int kk, const PoolView& pv, const uint16_t* q_raw, int nq, int k,
                             const uint64_t* ex, u64* partial, int32_t* q_valid,
                             DeviceStats* stats, int grid, const FusedAppend& fa,
                             cudaStream_t st) {
  if (kk == 32) return launch_one<QT, 1>(pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  if (kk == 64) return launch_one<QT, 2>(pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  return launch_one<QT, 4>(pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
}

cudaError_t launch_scan_gemv(const PoolView& pv, const uint16_t* q_raw, int32_t nq, int32_t k,
                             int32_t kk, const uint64_t* exclude_tag, u64* partial,
                             int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                             int32_t num_sms, int32_t* n_lists, const FusedAppend* fused,
                             cudaStream_t st) {
  const int grid = scan_gemv_grid(pv.n_rows, num_sms, max_lists);
  *n_lists = grid;
  FusedAppend fa = {};
  if (fused) {
    // every appending CTA must exist, and all CTAs be resident together (they are: at most
    // two per SM are launched), because scanning warps wait for the appending ones
    if (fused->n > grid || fused->n > kFuseMaxRows) return cudaErrorInvalidValue;
    fa = *fused;
  }
  if (nq >= 2)
    return launch_qt<2>(kk, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
  return launch_qt<1>(kk, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
}

cudaError_t preload_scan_gemv_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(scan_gemv_kernel<1, 1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_kernel<1, 2>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_kernel<1, 4>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_kernel<2, 1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_kernel<2, 2>, true)) != cudaSuccess) return e;
  return preload_kernel(scan_gemv_kernel<2, 4>, true);
}

}  // namespace oilbird

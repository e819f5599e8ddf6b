// K2: CUDA-core scan for a few queries (single-request decode).
//
// Scoring line of Algorithm 1, "s_i <- cos(h_t, h_i) for all i in P", fused with the
// per-CTA part of Eq. 2's top-k: every stored key is streamed from HBM exactly once
// with 16-byte loads, multiplied against the normalised queries held in shared memory
// (bf16 x bf16 products accumulated in fp32), and each warp keeps its k best rows in a
// small shared-memory list.  Scores never go to global memory; what leaves the CTA is
// one descending list of kk (= max(32, k rounded up to a power of two)) packed
// candidates per query.  The raw query states are normalised by every CTA itself
// (8-32 KB from L2), which saves a separate launch on the latency-critical path.
//
// The kernel is bound by the key stream (N*d*2 bytes); per 16 bytes of key a lane
// spends 8 integer unpack ops and 8*QT FMAs, well under the issue budget for QT <= 4.
#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"

namespace oilbird {

constexpr int kScanThreads = kNormThreads;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kRowsPerIter = 4;   // rows a warp scores together (shares each query load)

// Sort each warp's list, merge the warps' lists and let warp 0 publish the CTA's kk best.
template <int E>
__device__ __forceinline__ void publish_cta_list(const WarpTopK& top, u64* scratch,
                                                 u64* __restrict__ dst) {
  const int lane = threadIdx.x & 31;
  u64 v[E];
#pragma unroll
  for (int r = 0; r < E; ++r) v[r] = (r * 32 + lane < top.cnt) ? top.list[r * 32 + lane] : 0;
  warp_sort_desc<E>(v, lane);
  block_merge_desc<E>(v, scratch, kScanWarps);
  if (threadIdx.x < 32) {
#pragma unroll
    for (int r = 0; r < E; ++r) dst[r * 32 + lane] = v[r];
  }
}

template <int QT>
__global__ void __launch_bounds__(kScanThreads, 2)
scan_gemv_kernel(PoolView pv, const uint16_t* __restrict__ q_raw, int nq, int k, int kk,
                 const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                 int32_t* __restrict__ q_valid, DeviceStats* stats) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = pv.d, n_chunks = d >> 3;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                       // [QT][n_chunks]
  u64* lists = reinterpret_cast<u64*>(smem_raw + (size_t)QT * d * 2);    // [QT][warps][k]
  u64* scratch = lists + (size_t)QT * kScanWarps * k;                    // [warps][kk]
  __shared__ uint64_t s_ex[QT];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // contiguous, balanced share of the rows for this CTA
  const int64_t n = pv.n_rows;
  const int r_lo = (int)((n * blockIdx.x) / gridDim.x);
  const int r_hi = (int)((n * (blockIdx.x + 1)) / gridDim.x);
  const uint4* keys4 = reinterpret_cast<const uint4*>(pv.keys);

  for (int q0 = 0; q0 < nq; q0 += QT) {
    __syncthreads();
    // query preparation: qs[q] = bf16(q / ||q||), exactly as a key is stored
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      uint16_t* dst = reinterpret_cast<uint16_t*>(qs + (size_t)q * n_chunks);
      if (q0 + q < nq) {
        const int code = normalize_row(q_raw + (size_t)(q0 + q) * d, dst, d);
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

    WarpTopK top[QT];
#pragma unroll
    for (int q = 0; q < QT; ++q) top[q].init(lists + ((size_t)q * kScanWarps + warp) * k, k);

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

#pragma unroll 2
      for (int c = lane; c < n_chunks; c += 32) {
        uint4 kv[kRowsPerIter];
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) kv[r] = ld_stream16(rowp[r] + c);
#pragma unroll
        for (int q = 0; q < QT; ++q) {
          const uint4 qv = qs[q * n_chunks + c];
          const float q0f = bf16_lo(qv.x), q1f = bf16_hi(qv.x), q2f = bf16_lo(qv.y),
                      q3f = bf16_hi(qv.y), q4f = bf16_lo(qv.z), q5f = bf16_hi(qv.z),
                      q6f = bf16_lo(qv.w), q7f = bf16_hi(qv.w);
#pragma unroll
          for (int r = 0; r < kRowsPerIter; ++r) {
            float a = acc[r][q];
            a = fmaf(bf16_lo(kv[r].x), q0f, a);
            a = fmaf(bf16_hi(kv[r].x), q1f, a);
            a = fmaf(bf16_lo(kv[r].y), q2f, a);
            a = fmaf(bf16_hi(kv[r].y), q3f, a);
            a = fmaf(bf16_lo(kv[r].z), q4f, a);
            a = fmaf(bf16_hi(kv[r].z), q5f, a);
            a = fmaf(bf16_lo(kv[r].w), q6f, a);
            a = fmaf(bf16_hi(kv[r].w), q7f, a);
            acc[r][q] = a;
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) {
        const int row = rb + r;
        if (row >= r_hi) break;                             // warp-uniform
        uint64_t tag = 0;
        if (exclude_tag) tag = pv.trace_tag[pv.trace_id[row]];
#pragma unroll
        for (int q = 0; q < QT; ++q) {
          const float s = warp_sum(acc[r][q]);
          if (q0 + q >= nq) continue;
          if (s_ex[q] != 0 && tag == s_ex[q]) continue;     // same-prompt trace: skipped
          const u64 key = pack_candidate(s, (uint32_t)row);
          if (top[q].wants(key)) top[q].insert(key, lane);
        }
      }
    }
    // merge the warps' lists of each query and publish the CTA's kk best, descending
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      if (q0 + q >= nq) break;
      __syncwarp();
      u64* dst = partial + ((size_t)blockIdx.x * nq + (q0 + q)) * kk;
      if (kk == 32) publish_cta_list<1>(top[q], scratch, dst);
      else if (kk == 64) publish_cta_list<2>(top[q], scratch, dst);
      else publish_cta_list<4>(top[q], scratch, dst);
    }
  }
}

template <int QT>
static cudaError_t launch_qt(const PoolView& pv, const uint16_t* q_raw, int nq, int k, int kk,
                             const uint64_t* ex, u64* partial, int32_t* q_valid,
                             DeviceStats* stats, int grid, cudaStream_t st) {
  size_t smem = (size_t)QT * pv.d * 2 + (size_t)QT * kScanWarps * k * sizeof(u64) +
                (size_t)kScanWarps * kk * sizeof(u64);
  cudaError_t e = cudaFuncSetAttribute(scan_gemv_kernel<QT>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  scan_gemv_kernel<QT><<<grid, kScanThreads, smem, st>>>(pv, q_raw, nq, k, kk, ex, partial,
                                                         q_valid, stats);
  return cudaGetLastError();
}

cudaError_t launch_scan_gemv(const PoolView& pv, const uint16_t* q_raw, int32_t nq, int32_t k,
                             int32_t kk, const uint64_t* exclude_tag, u64* partial,
                             int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                             int32_t num_sms, int32_t* n_lists, cudaStream_t st) {
  // at least 32 rows per CTA, at most two CTAs per SM
  int64_t want = (pv.n_rows + 31) / 32;
  int grid = (int)(want < 1 ? 1 : want);
  if (grid > 2 * num_sms) grid = 2 * num_sms;
  if (grid > max_lists) grid = max_lists;
  *n_lists = grid;
  // queries held in shared memory together: bounded by 64 KB of bf16 query data
  int qt = nq >= 4 ? 4 : (nq >= 2 ? 2 : 1);
  while (qt > 1 && (size_t)qt * pv.d * 2 > 65536) qt >>= 1;
  switch (qt) {
    case 4: return launch_qt<4>(pv, q_raw, nq, k, kk, exclude_tag, partial, q_valid, stats, grid, st);
    case 2: return launch_qt<2>(pv, q_raw, nq, k, kk, exclude_tag, partial, q_valid, stats, grid, st);
    default: return launch_qt<1>(pv, q_raw, nq, k, kk, exclude_tag, partial, q_valid, stats, grid, st);
  }
}

}  // namespace oilbird

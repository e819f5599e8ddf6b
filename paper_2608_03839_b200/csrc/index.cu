// Coarse index over a pool: an inverted file over centroids the caller supplies.
//
// The paper's Limitations section names "an index" next to eviction and quantisation as a way
// to keep the cost of the cosine lookup from growing with the store, and defines none.  The
// one here leaves the pool as it is (rows stay where they were appended, so positions, traces
// and continuations are untouched) and adds, per row, the number of a list:
//   assign   a row belongs to the list of the centroid that is the best neighbour of the row's
//            STORED key taken as a query (the library's own lookup with k = 1 against a small
//            pool that holds the centroids; ties to the lowest centroid);
//   probe    a query's lists are its n_probe best centroids (the same lookup, k = n_probe);
//   scan     the rows of those lists, found through row numbers kept list by list, plus every
//            row appended since the last refresh (the tail) are scored exactly as the full
//            scan scores them, and the k best by (score, lowest row) go through the same merge,
//            firing rule, depth and gather (Eq. 2, Eq. 3).
// The answer is the full scan's answer restricted to the candidate rows: exact with every
// list probed, approximate otherwise (recall is measured by the benchmark).  A key row is
// 2d contiguous bytes, so fetching rows by number costs HBM nothing in efficiency; a lookup
// moves n_lists*d*2 bytes of centroids plus the candidates' keys instead of the whole pool.
#include <math.h>
#include <stdio.h>

#include <new>

#include "common.cuh"
#include "gather.cuh"
#include "internal.h"
#include "normalize.cuh"
#include "pool_priv.h"
#include "quant8.cuh"

namespace oilbird {

constexpr int kIndexMaxLists = 65536;
constexpr int kIndexMaxProbe = OILBIRD_MAX_K;        // the probes are a k-lookup on the centroids
constexpr int kIndexAssignBatch = 256;               // rows assigned per lookup
// Batches up to here take the one-launch lookup.  It splits the CTAs of a launch between the
// queries, so from two queries on the separate launches (each with every CTA on every
// query's share, the centroids scanned once for all queries by the batched kernels) are
// faster: 45.9 against 42.7 us for two queries, 72.9 against 55.6 us for four (C4 pool,
// 4,096 lists, 4 probes).
constexpr int kLookupMaxNq = 1;

// ------------------------------------------------------------------ list building ---
__global__ void __launch_bounds__(256)
index_count_kernel(const int32_t* __restrict__ assign, int n, int32_t* __restrict__ counts,
                   int n_lists) {
  pdl_enter();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int l = assign[i];
    if (l >= 0 && l < n_lists) atomicAdd(&counts[l], 1);
  }
}

// list_off[l] = rows in lists below l (one block); cursor starts at zero.
__global__ void __launch_bounds__(1024)
index_offsets_kernel(const int32_t* __restrict__ counts, int32_t* __restrict__ list_off,
                     int32_t* __restrict__ cursor, int n_lists) {
  __shared__ int s_sum[1024];
  pdl_enter();
  const int per = (n_lists + 1023) / 1024;
  const int lo = threadIdx.x * per, hi = min(n_lists, lo + per);
  int sum = 0;
  for (int l = lo; l < hi; ++l) sum += counts[l];
  s_sum[threadIdx.x] = sum;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {                  // inclusive scan of the threads' sums
    const int v = threadIdx.x >= o ? s_sum[threadIdx.x - o] : 0;
    __syncthreads();
    s_sum[threadIdx.x] += v;
    __syncthreads();
  }
  int run = s_sum[threadIdx.x] - sum;
  for (int l = lo; l < hi; ++l) {
    list_off[l] = run;
    cursor[l] = 0;
    run += counts[l];
  }
  if (threadIdx.x == 1023) list_off[n_lists] = s_sum[1023];
}

__global__ void __launch_bounds__(256)
index_scatter_kernel(const int32_t* __restrict__ assign, int n, const int32_t* __restrict__ list_off,
                     int32_t* __restrict__ cursor, int32_t* __restrict__ list_rows, int n_lists) {
  pdl_enter();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int l = assign[i];
    if (l >= 0 && l < n_lists) list_rows[list_off[l] + atomicAdd(&cursor[l], 1)] = i;
  }
}

// ------------------------------------------------------------------- training ---
// One Lloyd update: block l turns centroid l into the mean of the stored keys of its list
// (a list without rows keeps its centroid).  Sums are taken in fixed point, element x
// contributing trunc(x * 2^30), so that they are exact and do not depend on the order in
// which the scatter kernel happened to place the rows; the new raw element is
// bf16(float(double(sum) / (count * 2^30))), both roundings to nearest even.
constexpr int kMeanChunks = 4;          // 16-byte chunks of the row width per thread: d <= 8192
__global__ void __launch_bounds__(256)
index_means_kernel(const uint16_t* __restrict__ keys, int d, const int32_t* __restrict__ list_off,
                   const int32_t* __restrict__ list_rows, uint16_t* __restrict__ cent_raw) {
  pdl_enter();
  const int l = blockIdx.x;
  const int lo = list_off[l], hi = list_off[l + 1];
  if (hi == lo) return;
  const int n_chunks = d >> 3;
  long long acc[kMeanChunks][8];
#pragma unroll
  for (int u = 0; u < kMeanChunks; ++u)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[u][j] = 0;
  for (int i = lo; i < hi; ++i) {
    const uint4* row = reinterpret_cast<const uint4*>(keys + (size_t)list_rows[i] * d);
#pragma unroll
    for (int u = 0; u < kMeanChunks; ++u) {
      const int c = threadIdx.x + u * 256;
      if (c < n_chunks) {
        const uint4 v = __ldg(row + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[u][2 * j] += (long long)((double)bf16_lo(w[j]) * 1073741824.0);      // truncates
          acc[u][2 * j + 1] += (long long)((double)bf16_hi(w[j]) * 1073741824.0);
        }
      }
    }
  }
  const double denom = (double)(hi - lo) * 1073741824.0;
  uint4* dst = reinterpret_cast<uint4*>(cent_raw + (size_t)l * d);
#pragma unroll
  for (int u = 0; u < kMeanChunks; ++u) {
    const int c = threadIdx.x + u * 256;
    if (c < n_chunks) {
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a = __double2float_rn(__ll2double_rn(acc[u][2 * j]) / denom);
        const float b = __double2float_rn(__ll2double_rn(acc[u][2 * j + 1]) / denom);
        o[j] = f32_to_bf16_bits(a) | (f32_to_bf16_bits(b) << 16);
      }
      dst[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// ------------------------------------------------------------- scan of the candidates ---
// Grid (G, nq): CTA (b, q) scores a contiguous share of query q's candidates (the rows of its
// probed lists in probe order, then the tail) and leaves one descending list of KK packed
// candidates in partial[b][q], as the full scans do.  Rows are fetched by number; everything
// else (query preparation, scoring, per-warp lists, block merge) is the CUDA-core scan's.
// One row against the query in shared memory with up to kWide 16-byte loads per lane in
// flight at once (a whole row of d <= 4096 in one round trip): for CTAs that hold a handful of
// rows, where the round trips, not the bytes, are the cost.  A lane adds its chunks in the
// order score_rows adds them, so the score has the same bits.
constexpr int kWide = 16;
__device__ __forceinline__ float score_row_wide(const uint4* row, const uint4* qs, int n_chunks,
                                                int lane) {
  float a = 0.f;
  for (int c0 = lane; c0 < n_chunks; c0 += 32 * kWide) {
    uint4 kv[kWide];
#pragma unroll
    for (int u = 0; u < kWide; ++u) {
      const int c = c0 + 32 * u;
      kv[u] = c < n_chunks ? ld_stream16(row + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kWide; ++u) {
      const int c = c0 + 32 * u;
      if (c < n_chunks) {
        const uint4 qv = qs[c];
        a = fmaf(bf16_lo(kv[u].x), bf16_lo(qv.x), a);
        a = fmaf(bf16_hi(kv[u].x), bf16_hi(qv.x), a);
        a = fmaf(bf16_lo(kv[u].y), bf16_lo(qv.y), a);
        a = fmaf(bf16_hi(kv[u].y), bf16_hi(qv.y), a);
        a = fmaf(bf16_lo(kv[u].z), bf16_lo(qv.z), a);
        a = fmaf(bf16_hi(kv[u].z), bf16_hi(qv.z), a);
        a = fmaf(bf16_lo(kv[u].w), bf16_lo(qv.w), a);
        a = fmaf(bf16_hi(kv[u].w), bf16_hi(qv.w), a);
      }
    }
  }
  return warp_sum(a);
}
// CTAs with at most this many rows each take them one row per warp at a time
constexpr int kWideMaxRows = 64;

// One row of codes against the query in shared memory: a lane adds its elements in the order
// the 8-bit CUDA-core scan adds them (16-code chunks lane, lane + 32, ...; within a chunk
// element by element), so the score has that scan's bits.  Up to kWide8 chunks in flight.
constexpr int kWide8 = 8;
__device__ __forceinline__ float score_code_row(const uint4* row, const uint4* qs, int n16, int lane) {
  float a = 0.f;
  for (int c0 = lane; c0 < n16; c0 += 32 * kWide8) {
    uint4 kv[kWide8];
#pragma unroll
    for (int u = 0; u < kWide8; ++u) {
      const int c = c0 + 32 * u;
      kv[u] = c < n16 ? ld_stream16(row + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kWide8; ++u) {
      const int c = c0 + 32 * u;
      if (c < n16) {
        const uint4 qa = qs[2 * c], qb = qs[2 * c + 1];
        const uint32_t w[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
        const uint32_t qw[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 ka = e4m3x2_to_float2(w[j] & 0xffffu), kb = e4m3x2_to_float2(w[j] >> 16);
          a = fmaf(ka.x, bf16_lo(qw[2 * j]), a);
          a = fmaf(ka.y, bf16_hi(qw[2 * j]), a);
          a = fmaf(kb.x, bf16_lo(qw[2 * j + 1]), a);
          a = fmaf(kb.y, bf16_hi(qw[2 * j + 1]), a);
        }
      }
    }
  }
  return warp_sum(a);
}

// The candidate scan of CTA b of G for query q, whose normalised form is in qs.  k8: the pool
// holds E4M3 codes and one scale per row (scored as the 8-bit CUDA-core scan scores them).
template <int E, bool k8 = false>
__device__ __forceinline__ void scan_candidates(const PoolView& pv, const uint4* qs, u64* scratch,
                                                int q, int nq, int k, int b, int G,
                                                const int32_t* probes, int n_probe,
                                                const int32_t* __restrict__ list_off,
                                                const int32_t* __restrict__ list_rows, int n_indexed,
                                                const uint64_t* __restrict__ exclude_tag,
                                                u64* __restrict__ partial, int* s_pref, int* s_base,
                                                const uint8_t* __restrict__ codes = nullptr,
                                                const float* __restrict__ scales = nullptr) {
  constexpr int KK = 32 * E;
  constexpr int kWarps = kNormThreads / 32;
  const int n_chunks = pv.d >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // the probed lists of this query, laid end to end (the probes may have been written by
  // another CTA of this launch: read through L2)
  if (threadIdx.x < n_probe) {
    const int l = __ldcg(&probes[(size_t)q * n_probe + threadIdx.x]);
    s_base[threadIdx.x] = l >= 0 ? list_off[l] : 0;
    s_pref[threadIdx.x + 1] = l >= 0 ? list_off[l + 1] - list_off[l] : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    s_pref[0] = 0;
    for (int p = 0; p < n_probe; ++p) s_pref[p + 1] += s_pref[p];
  }
  __syncthreads();
  const int in_lists = s_pref[n_probe];
  const int total = in_lists + (pv.n_rows - n_indexed);
  const uint64_t ex = exclude_tag ? exclude_tag[q] : 0;
  const int c_lo = (int)(((long long)total * b) / G);
  const int c_hi = (int)(((long long)total * (b + 1)) / G);
  const uint4* keys4 = reinterpret_cast<const uint4*>(pv.keys);

  auto row_of = [&](int c) -> int {
    if (c >= in_lists) return n_indexed + (c - in_lists);          // the tail
    int lo = 0, hi = n_probe;                                      // last p with s_pref[p] <= c
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_pref[mid] <= c) lo = mid; else hi = mid;
    }
    return list_rows[s_base[lo] + (c - s_pref[lo])];
  };

  u64 top[1][E];
  u64 kth = 0;
#pragma unroll
  for (int r = 0; r < E; ++r) top[0][r] = 0;
  if (k8) {
    const uint4* codes4 = reinterpret_cast<const uint4*>(codes);
    const int n16 = pv.d >> 4;
    for (int c = c_lo + warp; c < c_hi; c += kWarps) {
      const int row = row_of(c);
      const float sc = scales[row];
      const float s = score_code_row(codes4 + (size_t)row * n16, qs, n16, lane) * sc;
      if (ex != 0 && pv.trace_tag[pv.trace_id[row]] == ex) continue;       // same-prompt trace
      const u64 key = pack_candidate(s, (uint32_t)row);
      if (key > kth) {
        warp_sorted_insert<E>(top[0], key, lane);
        kth = warp_list_get<E>(top[0], k - 1);
      }
    }
  } else if (c_hi - c_lo <= kWideMaxRows) {
    for (int c = c_lo + warp; c < c_hi; c += kWarps) {
      const int row = row_of(c);
      const float s = score_row_wide(keys4 + (size_t)row * n_chunks, qs, n_chunks, lane);
      if (ex != 0 && pv.trace_tag[pv.trace_id[row]] == ex) continue;       // same-prompt trace
      const u64 key = pack_candidate(s, (uint32_t)row);
      if (key > kth) {
        warp_sorted_insert<E>(top[0], key, lane);
        kth = warp_list_get<E>(top[0], k - 1);
      }
    }
  } else
  for (int cb = c_lo + warp * kRowsPerIter; cb < c_hi; cb += kWarps * kRowsPerIter) {
    int rows[kRowsPerIter];
    const uint4* rowp[kRowsPerIter];
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) {
      rows[r] = row_of(cb + r < c_hi ? cb + r : c_hi - 1);          // clamp: result discarded below
      rowp[r] = keys4 + (size_t)rows[r] * n_chunks;
    }
    float acc[kRowsPerIter][1];
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) acc[r][0] = 0.f;
    score_rows<1, false>(rowp, qs, n_chunks, lane, acc);
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) {
      if (cb + r >= c_hi) break;                                    // warp-uniform
      const float s = warp_sum(acc[r][0]);
      if (ex != 0 && pv.trace_tag[pv.trace_id[rows[r]]] == ex) continue;   // same-prompt trace
      const u64 key = pack_candidate(s, (uint32_t)rows[r]);
      if (key > kth) {
        warp_sorted_insert<E>(top[0], key, lane);
        kth = warp_list_get<E>(top[0], k - 1);
      }
    }
  }
  block_merge_desc<E>(top[0], scratch, kWarps);
  if (threadIdx.x < 32) {
    u64* dst = partial + ((size_t)b * nq + q) * KK;
#pragma unroll
    for (int r = 0; r < E; ++r) dst[r * 32 + lane] = top[0][r];
  }
}

template <int E>
__global__ void __launch_bounds__(kNormThreads, 2)
scan_ids_kernel(PoolView pv, const uint16_t* __restrict__ q_raw, int nq, int k,
                const int32_t* __restrict__ probes, int n_probe,
                const int32_t* __restrict__ list_off, const int32_t* __restrict__ list_rows,
                int n_indexed, const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                int32_t* __restrict__ q_valid, DeviceStats* stats) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_pref[kIndexMaxProbe + 1], s_base[kIndexMaxProbe];
  pdl_enter();
  const int d = pv.d;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [n_chunks]
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)d * 2);        // [warps][KK]
  const int q = blockIdx.y;
  const int code = normalize_row<true, 2>(q_raw + (size_t)q * d, reinterpret_cast<uint16_t*>(qs), d);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    q_valid[q] = code == kRowNonFinite ? 0 : 1;          // NaN/Inf: no neighbours
    if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
  }
  scan_candidates<E>(pv, qs, scratch, q, nq, k, blockIdx.x, gridDim.x, probes, n_probe, list_off,
                     list_rows, n_indexed, exclude_tag, partial, s_pref, s_base);
}

// ------------------------------------------------------------------- 8-bit pools ---
// What a stored row of an 8-bit pool is, as a state (the library's reading; the paper defines
// neither the quantised store nor the index): element j of row i is fp32(value(code_ij) *
// scale_i), one rounding.  As a query state (the assignment of a row to its list) the row is
// those elements rounded to bf16, like any state the library is handed.
__global__ void __launch_bounds__(256)
dequant_rows_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scales, int d,
                    int row0, uint16_t* __restrict__ out) {
  pdl_enter();
  const int r = blockIdx.x;
  const float sc = scales[row0 + r];
  const uint4* src = reinterpret_cast<const uint4*>(codes + (size_t)(row0 + r) * d);
  uint4* dst = reinterpret_cast<uint4*>(out + (size_t)r * d);
  for (int c = threadIdx.x; c < (d >> 4); c += blockDim.x) {
    const uint4 v = src[c];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 a = e4m3x2_to_float2(w[j] & 0xffffu), b = e4m3x2_to_float2(w[j] >> 16);
      o[2 * j] = f32_to_bf16_bits(__fmul_rn(a.x, sc)) | (f32_to_bf16_bits(__fmul_rn(a.y, sc)) << 16);
      o[2 * j + 1] = f32_to_bf16_bits(__fmul_rn(b.x, sc)) | (f32_to_bf16_bits(__fmul_rn(b.y, sc)) << 16);
    }
    dst[2 * c] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[2 * c + 1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

// The training means over an 8-bit pool: as index_means_kernel, each element contributing
// trunc(x * 2^30) with x = fp32(value(code) * scale).  A thread holds 16-code chunks.
constexpr int kMeanChunks8 = 2;         // 16-code chunks of the row width per thread: d <= 8192
__global__ void __launch_bounds__(256)
index_means_e4m3_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scales, int d,
                        const int32_t* __restrict__ list_off, const int32_t* __restrict__ list_rows,
                        uint16_t* __restrict__ cent_raw) {
  pdl_enter();
  const int l = blockIdx.x;
  const int lo = list_off[l], hi = list_off[l + 1];
  if (hi == lo) return;
  const int n16 = d >> 4;
  long long acc[kMeanChunks8][16];
#pragma unroll
  for (int u = 0; u < kMeanChunks8; ++u)
#pragma unroll
    for (int j = 0; j < 16; ++j) acc[u][j] = 0;
  for (int i = lo; i < hi; ++i) {
    const int row = list_rows[i];
    const float sc = scales[row];
    const uint4* src = reinterpret_cast<const uint4*>(codes + (size_t)row * d);
#pragma unroll
    for (int u = 0; u < kMeanChunks8; ++u) {
      const int c = threadIdx.x + u * 256;
      if (c < n16) {
        const uint4 v = __ldg(src + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 a = e4m3x2_to_float2(w[j] & 0xffffu), b = e4m3x2_to_float2(w[j] >> 16);
          acc[u][4 * j] += (long long)((double)__fmul_rn(a.x, sc) * 1073741824.0);       // truncates
          acc[u][4 * j + 1] += (long long)((double)__fmul_rn(a.y, sc) * 1073741824.0);
          acc[u][4 * j + 2] += (long long)((double)__fmul_rn(b.x, sc) * 1073741824.0);
          acc[u][4 * j + 3] += (long long)((double)__fmul_rn(b.y, sc) * 1073741824.0);
        }
      }
    }
  }
  const double denom = (double)(hi - lo) * 1073741824.0;
  uint4* dst = reinterpret_cast<uint4*>(cent_raw + (size_t)l * d);
#pragma unroll
  for (int u = 0; u < kMeanChunks8; ++u) {
    const int c = threadIdx.x + u * 256;
    if (c < n16) {
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float a = __double2float_rn(__ll2double_rn(acc[u][2 * j]) / denom);
        const float b = __double2float_rn(__ll2double_rn(acc[u][2 * j + 1]) / denom);
        o[j] = f32_to_bf16_bits(a) | (f32_to_bf16_bits(b) << 16);
      }
      dst[2 * c] = make_uint4(o[0], o[1], o[2], o[3]);
      dst[2 * c + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
  }
}

// The candidate scan over an 8-bit pool (separate launches).
template <int E>
__global__ void __launch_bounds__(kNormThreads, 2)
scan_ids_e4m3_kernel(PoolView pv, const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                     const uint16_t* __restrict__ q_raw, int nq, int k,
                     const int32_t* __restrict__ probes, int n_probe,
                     const int32_t* __restrict__ list_off, const int32_t* __restrict__ list_rows,
                     int n_indexed, const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                     int32_t* __restrict__ q_valid, DeviceStats* stats) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_pref[kIndexMaxProbe + 1], s_base[kIndexMaxProbe];
  pdl_enter();
  const int d = pv.d;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [d / 8] bf16
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)d * 2);        // [warps][KK]
  const int q = blockIdx.y;
  const int code = normalize_row<true, 2>(q_raw + (size_t)q * d, reinterpret_cast<uint16_t*>(qs), d);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    q_valid[q] = code == kRowNonFinite ? 0 : 1;          // NaN/Inf: no neighbours
    if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
  }
  scan_candidates<E, true>(pv, qs, scratch, q, nq, k, blockIdx.x, gridDim.x, probes, n_probe, list_off,
                           list_rows, n_indexed, exclude_tag, partial, s_pref, s_base, codes, scales);
}

template <int E>
static cudaError_t launch_scan_ids_e4m3(const PoolView& pv, const uint8_t* codes, const float* scales,
                                        const uint16_t* q, int nq, int k, const int32_t* probes,
                                        int n_probe, const int32_t* list_off, const int32_t* list_rows,
                                        int n_indexed, const uint64_t* ex, u64* partial,
                                        int32_t* q_valid, DeviceStats* stats, int grid, cudaStream_t st) {
  const size_t smem = (size_t)pv.d * 2 + (size_t)(kNormThreads / 32) * 32 * E * sizeof(u64);
  return launch_pdl(scan_ids_e4m3_kernel<E>, dim3(grid, nq), dim3(kNormThreads), smem, st, pv, codes,
                    scales, q, nq, k, probes, n_probe, list_off, list_rows, n_indexed, ex, partial,
                    q_valid, stats);
}

// ------------------------------------------------------------ folding lists on one CTA ---
// The `want` best entries of n descending lists (KK = 32*E entries each, `stride` apart, written
// during this launch: read through L2) into warp 0's registers.  A list's head is its best
// entry, and the want-th largest of any grouping's best heads is reached by `want` distinct
// lists, so no list whose head lies below that floor holds one of the `want` best: the heads
// come first, in one round of loads, then only the lists at or above the floor.
constexpr int kFoldMaxLists = 2 * kNormThreads;
template <int E>
__device__ __forceinline__ void fold_lists(const u64* lists, int n, size_t stride, int want,
                                           u64 (&v)[E], u64* scratch) {
  constexpr int kWarps = kNormThreads / 32;
  constexpr int PF = E == 1 ? 8 : (E == 2 ? 4 : 2);        // lists a warp has in flight
  __shared__ u64 s_floor, s_wmax[kWarps];
  __shared__ int s_live[kFoldMaxLists], s_nlive;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, t = threadIdx.x;
  const u64 h0 = t < n ? __ldcg(lists + (size_t)t * stride) : 0;
  const u64 h1 = t + kNormThreads < n ? __ldcg(lists + (size_t)(t + kNormThreads) * stride) : 0;
  const u64 hm = h0 > h1 ? h0 : h1;
  if (t == 0) s_nlive = 0;
  if (want <= kWarps) {
    // few wanted: the warps' best heads are grouping enough, and cheaper than a sort
    u64 m = hm;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const u64 x = shfl_xor_u64(m, o); m = x > m ? x : m; }
    if (lane == 0) s_wmax[warp] = m;
    __syncthreads();
    if (t == 0) {
      u64 w[kWarps];
#pragma unroll
      for (int i = 0; i < kWarps; ++i) w[i] = s_wmax[i];
      u64 fl = 0;
#pragma unroll
      for (int i = 0; i < kWarps; ++i) {                           // want-th largest of eight
        int above = 0;
#pragma unroll
        for (int j = 0; j < kWarps; ++j) above += (w[j] > w[i] || (w[j] == w[i] && j < i)) ? 1 : 0;
        if (above == want - 1) fl = w[i];
      }
      s_floor = fl;
    }
  } else {
    u64 hv[E];
#pragma unroll
    for (int r = 0; r < E; ++r) hv[r] = 0;
    u64 h[1] = {hm};
    warp_sort_desc<1>(h, lane);
    hv[0] = h[0];                                                  // sorted, zeros behind it
    block_merge_desc<E>(hv, scratch, kWarps);
    const u64 fl = want <= 32 * E ? warp_list_get<E>(hv, want - 1) : 0;   // warp 0 holds the merged heads
    if (t == 0) s_floor = fl;
  }
  __syncthreads();
  const u64 fl = s_floor;
  if (h0 != 0 && h0 >= fl) s_live[atomicAdd(&s_nlive, 1)] = t;
  if (h1 != 0 && h1 >= fl) s_live[atomicAdd(&s_nlive, 1)] = t + kNormThreads;
  __syncthreads();
  const int n_live = s_nlive;
#pragma unroll
  for (int r = 0; r < E; ++r) v[r] = 0;
  // (live list i goes to warp i mod kWarps: a handful of lists are spread over the warps)
  for (int i0 = warp; i0 < n_live; i0 += kWarps * PF) {
    u64 bl[PF][E];
#pragma unroll
    for (int u = 0; u < PF; ++u) {
      const int i = i0 + u * kWarps;
      const u64* src = lists + (size_t)s_live[i < n_live ? i : 0] * stride;
#pragma unroll
      for (int r = 0; r < E; ++r) bl[u][r] = i < n_live ? __ldcg(src + r * 32 + lane) : 0;
    }
#pragma unroll
    for (int u = 0; u < PF; ++u)
      if (i0 + u * kWarps < n_live) warp_merge_desc<E>(v, bl[u], lane);
  }
  block_merge_desc<E>(v, scratch, kWarps);
}

// ------------------------------------------------------------ one-launch lookup ---
// Centroid scan, choice of the probes and candidate scan in one launch (small batches, where
// a lookup is a chain of short dependent launches and their latencies are its cost).  Grid
// (g1 + g2, nq).  A CTA draws a ticket for its query when it starts.  The first g1 tickets
// score a share of the centroids each and leave a list of their 32 best; the last of them to
// finish merges the g1 lists, publishes the n_probe best centroids and raises the query's
// flag; none of them ever waits.  Tickets g1 and up prepare their query, wait for the flag
// (bounded, like every wait of this library) and then scan a share of the candidates.
// Whoever holds a ticket >= g1 knows that g1 CTAs have started before it, so what it waits
// for is running whether or not the whole grid fits on the GPU at once.  The last of the
// candidate CTAs to finish merges their lists and ends the lookup (firing rule, depth,
// gather: a4..a6), and the last CTA of a query to leave clears the query's words for the
// next launch.
struct LookupSync { unsigned ticket, scanned, ready, candidates, finished, pad[3]; };

template <int E, bool k8>
__global__ void __launch_bounds__(kNormThreads, 2)
index_lookup_kernel(PoolView pv, const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                    const uint16_t* __restrict__ cent_keys, int n_lists,
                    const uint16_t* __restrict__ q_raw, int nq, int k, int g1, int n_probe,
                    int32_t* probes, u64* cpartial, LookupSync* sync,
                    const int32_t* __restrict__ list_off, const int32_t* __restrict__ list_rows,
                    int n_indexed, const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                    DeviceStats* stats, GatherParams gp, oilbird_query_out out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_pref[kIndexMaxProbe + 1], s_base[kIndexMaxProbe];
  __shared__ int s_ticket, s_flag;
  constexpr int kWarps = kNormThreads / 32;
  pdl_enter();
  const int d = pv.d, n_chunks = d >> 3;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [n_chunks]
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)d * 2);        // [warps][KK]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.y;
  LookupSync* sy = sync + q;
  if (threadIdx.x == 0) s_ticket = (int)atomicAdd(&sy->ticket, 1u);
  const int code = normalize_row<true, 2>(q_raw + (size_t)q * d, reinterpret_cast<uint16_t*>(qs), d);
  __syncthreads();
  const int ticket = s_ticket;
  if (ticket >= (int)gridDim.x) {
    // words left over from a launch that gave up: no share is this CTA's to take.  The
    // status call reports it; oilbird_index_reset clears the words.
    if (threadIdx.x == 0) atomicExch(&stats->stalled, 1);
    return;
  }
  if (ticket < g1) {
    // ---- a share of the centroids
    const int r_lo = (int)(((long long)n_lists * ticket) / g1);
    const int r_hi = (int)(((long long)n_lists * (ticket + 1)) / g1);
    const uint4* keys4 = reinterpret_cast<const uint4*>(cent_keys);
    u64 top[1] = {0};
    u64 kth = 0;
    if (r_hi - r_lo <= kWideMaxRows) {
      for (int r = r_lo + warp; r < r_hi; r += kWarps) {
        const u64 key = pack_candidate(score_row_wide(keys4 + (size_t)r * n_chunks, qs, n_chunks, lane),
                                       (uint32_t)r);
        if (key > kth) {
          warp_sorted_insert<1>(top, key, lane);
          kth = warp_list_get<1>(top, n_probe - 1);
        }
      }
    } else
    for (int rb = r_lo + warp * kRowsPerIter; rb < r_hi; rb += kWarps * kRowsPerIter) {
      const uint4* rowp[kRowsPerIter];
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r)
        rowp[r] = keys4 + (size_t)(rb + r < r_hi ? rb + r : r_hi - 1) * n_chunks;
      float acc[kRowsPerIter][1];
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) acc[r][0] = 0.f;
      score_rows<1, false>(rowp, qs, n_chunks, lane, acc);
#pragma unroll
      for (int r = 0; r < kRowsPerIter; ++r) {
        if (rb + r >= r_hi) break;                                    // warp-uniform
        const u64 key = pack_candidate(warp_sum(acc[r][0]), (uint32_t)(rb + r));
        if (key > kth) {
          warp_sorted_insert<1>(top, key, lane);
          kth = warp_list_get<1>(top, n_probe - 1);
        }
      }
    }
    block_merge_desc<1>(top, scratch, kWarps);
    if (threadIdx.x < 32) {
      // warp 0 holds the list: it publishes it and arrives (the arrival releases the warp's
      // stores and, for the last one in, acquires everybody else's)
      cpartial[((size_t)ticket * nq + q) * 32 + lane] = top[0];
      __syncwarp();
      if (lane == 0) {
        unsigned prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(&sy->scanned) : "memory");
        s_flag = prev == (unsigned)(g1 - 1);
      }
    }
    __syncthreads();
    if (s_flag) {
      // ---- the last share is in: the g1 lists -> the probes
      u64 v[1];
      fold_lists<1>(cpartial + (size_t)q * 32, g1, (size_t)nq * 32, n_probe, v, scratch);
      if (threadIdx.x < 32) {
        if (lane < n_probe)
          probes[(size_t)q * n_probe + lane] = (v[0] != 0 && code != kRowNonFinite) ? candidate_row(v[0]) : -1;
        __syncwarp();
        if (lane == 0) {
          sy->scanned = 0;
          asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(&sy->ready), "r"(1u) : "memory");
        }
      }
    }
  } else {
    // ---- a share of the candidates, once the probes are known
    if (ticket == g1 && threadIdx.x == 0 && code == kRowNonFinite)
      atomicAdd(&stats->nonfinite_queries, 1ull);
    if (threadIdx.x == 0) s_flag = wait_flag_u32(&sy->ready, stats) ? 1 : 0;
    __syncthreads();
    const int b = ticket - g1, g2 = (int)gridDim.x - g1;
    const int woke = s_flag;
    __syncthreads();                                     // s_flag is written again below
    if (woke) {
      scan_candidates<E, k8>(pv, qs, scratch, q, nq, k, b, g2, probes, n_probe, list_off, list_rows,
                             n_indexed, exclude_tag, partial, s_pref, s_base, codes, scales);
    } else if (threadIdx.x < 32) {                         // gave up: an empty list
      constexpr int KK = 32 * E;
#pragma unroll
      for (int r = 0; r < E; ++r) partial[((size_t)b * nq + q) * KK + r * 32 + lane] = 0;
    }
    // ---- the last list in: merge them, fire, gather (warp 0 wrote this CTA's list)
    if (threadIdx.x < 32) {
      __syncwarp();
      if (lane == 0) {
        unsigned prev;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(&sy->candidates) : "memory");
        s_flag = prev == (unsigned)(g2 - 1);
      }
    }
    __syncthreads();
    if (s_flag) {
      constexpr int KK = 32 * E;
      __shared__ u64 s_best[OILBIRD_MAX_K];
      __shared__ int32_t s_idx[OILBIRD_MAX_K];
      __shared__ float s_score[OILBIRD_MAX_K];
      __shared__ int32_t s_len[OILBIRD_MAX_K];
      u64 v[E];
      fold_lists<E>(partial + (size_t)q * KK, g2, (size_t)nq * KK, gp.k, v, scratch);
      if (threadIdx.x < 32) {
#pragma unroll
        for (int r = 0; r < E; ++r) s_best[r * 32 + lane] = v[r];
      }
      __syncthreads();
      const int kq = gp.k;
      for (int j = threadIdx.x; j < kq; j += kNormThreads) {
        const u64 key = code != kRowNonFinite ? s_best[j] : 0;     // NaN/Inf query: no neighbours
        const int idx = key ? candidate_row(key) : -1;
        const float sc = key ? candidate_score(key) : -INFINITY;
        s_idx[j] = idx;
        s_score[j] = sc;
        out.idx[(size_t)q * kq + j] = idx;
        out.score[(size_t)q * kq + j] = sc;
      }
      __syncthreads();
      fire_depth_copy(pv, gp, q, s_idx, s_score, out, s_len);
      if (threadIdx.x == 0) sy->candidates = 0;
    }
  }
  // ---- the last CTA of the query leaves its words as it found them
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&sy->finished, 1u) == gridDim.x - 1) {
      sy->ticket = 0; sy->ready = 0; sy->finished = 0;
    }
  }
}

template <int E>
static cudaError_t launch_scan_ids(const PoolView& pv, const uint16_t* q, int nq, int k,
                                   const int32_t* probes, int n_probe, const int32_t* list_off,
                                   const int32_t* list_rows, int n_indexed, const uint64_t* ex,
                                   u64* partial, int32_t* q_valid, DeviceStats* stats, int grid,
                                   cudaStream_t st) {
  const size_t smem = (size_t)pv.d * 2 + (size_t)(kNormThreads / 32) * 32 * E * sizeof(u64);
  return launch_pdl(scan_ids_kernel<E>, dim3(grid, nq), dim3(kNormThreads), smem, st, pv, q, nq, k,
                    probes, n_probe, list_off, list_rows, n_indexed, ex, partial, q_valid, stats);
}

template <int E, bool k8>
static cudaError_t launch_index_lookup(const PoolView& pv, const uint8_t* codes, const float* scales,
                                       const uint16_t* cent_keys, int n_lists,
                                       const uint16_t* q, int nq, int k, int g1, int g2, int n_probe,
                                       int32_t* probes, u64* cpartial, LookupSync* sync,
                                       const int32_t* list_off, const int32_t* list_rows,
                                       int n_indexed, const uint64_t* ex, u64* partial,
                                       DeviceStats* stats, const GatherParams& gp,
                                       const oilbird_query_out& out, cudaStream_t st) {
  const size_t smem = (size_t)pv.d * 2 + (size_t)(kNormThreads / 32) * 32 * E * sizeof(u64);
  return launch_pdl(index_lookup_kernel<E, k8>, dim3(g1 + g2, nq), dim3(kNormThreads), smem, st, pv,
                    codes, scales, cent_keys, n_lists, q, nq, k, g1, n_probe, probes, cpartial, sync, list_off,
                    list_rows, n_indexed, ex, partial, stats, gp, out);
}

cudaError_t preload_index_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(index_count_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_offsets_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_scatter_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_means_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(dequant_rows_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_means_e4m3_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_ids_e4m3_kernel<1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_ids_e4m3_kernel<2>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_ids_e4m3_kernel<4>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<1, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<2, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<4, false>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<1, true>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<2, true>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(index_lookup_kernel<4, true>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_ids_kernel<1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_ids_kernel<2>, true)) != cudaSuccess) return e;
  return preload_kernel(scan_ids_kernel<4>, true);
}

}  // namespace oilbird

using namespace oilbird;

struct oilbird_index {
  oilbird_pool* pool;
  oilbird_pool* cent;            // the centroids, as a pool of n_lists rows
  int32_t n_lists;
  int64_t n_indexed;             // rows that have a list (enqueue-time truth)
  int64_t generation;            // the pool's row numbering the lists refer to
  unsigned char* mem;
  int32_t *assign, *list_rows, *list_off, *cursor, *counts;
  uint16_t* cent_raw;            // the raw centroid states the centroid pool was built from
  // results of the lookups on the centroids
  int32_t* probe_idx; float* probe_score; int32_t *probe_fired, *probe_len, *probe_tok;
  float* a_score; int32_t *a_fired, *a_len, *a_tok;
  oilbird::LookupSync* sync;     // one-launch lookups: four words per query, zero between launches
  uint16_t* as_query;            // 8-bit pools: a batch of stored rows as bf16 query states
};

static thread_local char g_index_err[256] = "";
static int index_fail(cudaError_t e, const char* what) {
  snprintf(g_index_err, sizeof g_index_err, "%s: %s", what, cudaGetErrorString(e));
  return e == cudaErrorMemoryAllocation ? OILBIRD_ENOMEM : OILBIRD_ECUDA;
}
#define ICU(call)                                         \
  do {                                                    \
    cudaError_t e_ = (call);                              \
    if (e_ != cudaSuccess) return index_fail(e_, #call);  \
  } while (0)

extern "C" {

const char* oilbird_index_last_error(void) { return g_index_err; }

int oilbird_index_create(oilbird_index_t** out, oilbird_pool_t* pool, const void* centroids_bf16,
                         int32_t n_lists, void* cuda_stream) {
  if (!out) return OILBIRD_EINVAL;
  *out = nullptr;
  if (!pool || !centroids_bf16 || n_lists < 1 || n_lists > kIndexMaxLists) return OILBIRD_EINVAL;
  if ((uintptr_t)centroids_bf16 & 15) return OILBIRD_EINVAL;
  ICU(cudaSetDevice(pool->device));
  oilbird_index* ix = new (std::nothrow) oilbird_index();
  if (!ix) return OILBIRD_ENOMEM;
  ix->pool = pool; ix->n_lists = n_lists; ix->n_indexed = 0; ix->cent = nullptr; ix->mem = nullptr;
  ix->generation = pool->generation;
  oilbird_pool_config cc = {};
  cc.d = pool->r.d; cc.capacity_rows = n_lists; cc.max_traces = 1; cc.max_nq = OILBIRD_MAX_NQ;
  cc.max_k = OILBIRD_MAX_K; cc.max_append = 1; cc.device = pool->device;
  cc.flags = pool->r.guards ? OILBIRD_DEBUG_GUARDS : 0;
  int rc = oilbird_pool_create(&ix->cent, &cc);
  if (rc) { delete ix; return rc; }
  const size_t cap = (size_t)pool->r.capacity, nl = (size_t)n_lists;
  const size_t rows_i32 = cap > nl ? cap : nl;
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  const size_t o_assign = 0, o_rows = o_assign + up(rows_i32 * 4), o_off = o_rows + up(rows_i32 * 4),
               o_cur = o_off + up((nl + 1) * 4), o_cnt = o_cur + up(nl * 4),
               o_pidx = o_cnt + up(nl * 4),
               o_psc = o_pidx + up((size_t)OILBIRD_MAX_NQ * kIndexMaxProbe * 4),
               o_pf = o_psc + up((size_t)OILBIRD_MAX_NQ * kIndexMaxProbe * 4),
               o_pl = o_pf + up((size_t)OILBIRD_MAX_NQ * 4),
               o_pt = o_pl + up((size_t)OILBIRD_MAX_NQ * kIndexMaxProbe * 4),
               o_as = o_pt + up((size_t)OILBIRD_MAX_NQ * kIndexMaxProbe * 4),
               o_af = o_as + up(kIndexAssignBatch * 4), o_al = o_af + up(kIndexAssignBatch * 4),
               o_at = o_al + up(kIndexAssignBatch * 4), o_sync = o_at + up(kIndexAssignBatch * 4),
               o_raw = o_sync + up((size_t)OILBIRD_MAX_NQ * sizeof(LookupSync)),
               o_asq = o_raw + up(nl * (size_t)pool->r.d * 2),
               total = o_asq + (pool->r.e4m3 ? up((size_t)kIndexAssignBatch * pool->r.d * 2) : 0);
  cudaError_t e = cudaMalloc((void**)&ix->mem, total);
  if (e != cudaSuccess) { oilbird_pool_destroy(ix->cent); delete ix; return index_fail(e, "cudaMalloc(index)"); }
  ix->assign = (int32_t*)(ix->mem + o_assign); ix->list_rows = (int32_t*)(ix->mem + o_rows);
  ix->list_off = (int32_t*)(ix->mem + o_off); ix->cursor = (int32_t*)(ix->mem + o_cur);
  ix->counts = (int32_t*)(ix->mem + o_cnt);
  ix->probe_idx = (int32_t*)(ix->mem + o_pidx); ix->probe_score = (float*)(ix->mem + o_psc);
  ix->probe_fired = (int32_t*)(ix->mem + o_pf); ix->probe_len = (int32_t*)(ix->mem + o_pl);
  ix->probe_tok = (int32_t*)(ix->mem + o_pt);
  ix->a_score = (float*)(ix->mem + o_as); ix->a_fired = (int32_t*)(ix->mem + o_af);
  ix->a_len = (int32_t*)(ix->mem + o_al); ix->a_tok = (int32_t*)(ix->mem + o_at);
  ix->cent_raw = (uint16_t*)(ix->mem + o_raw);
  ix->sync = (LookupSync*)(ix->mem + o_sync);
  ix->as_query = pool->r.e4m3 ? (uint16_t*)(ix->mem + o_asq) : nullptr;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // the centroids become the rows of a one-trace pool (their tokens are never looked at);
  // all lists start empty
  e = cudaMemsetAsync(ix->mem, 0, o_pidx, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(ix->sync, 0, (size_t)OILBIRD_MAX_NQ * sizeof(LookupSync), st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(ix->cent_raw, centroids_bf16, nl * (size_t)pool->r.d * 2,
                        cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess)
    rc = oilbird_pool_append(ix->cent, ix->cent_raw, ix->list_rows, n_lists, 0, OILBIRD_NEW_TRACE, st);
  if (e != cudaSuccess || rc) {
    cudaFree(ix->mem); oilbird_pool_destroy(ix->cent); delete ix;
    return e != cudaSuccess ? index_fail(e, "cudaMemsetAsync(index)") : rc;
  }
  *out = ix;
  return OILBIRD_OK;
}

int oilbird_index_destroy(oilbird_index_t* ix) {
  if (!ix) return OILBIRD_EINVAL;
  cudaSetDevice(ix->pool->device);
  cudaDeviceSynchronize();
  oilbird_pool_destroy(ix->cent);
  cudaFree(ix->mem);
  delete ix;
  return OILBIRD_OK;
}

int64_t oilbird_index_rows(const oilbird_index_t* ix) { return ix ? ix->n_indexed : 0; }

int oilbird_index_reset(oilbird_index_t* ix, void* cuda_stream) {
  if (!ix) return OILBIRD_EINVAL;
  ICU(cudaSetDevice(ix->pool->device));
  // every list empty again: offsets all zero
  ICU(cudaMemsetAsync(ix->list_off, 0, ((size_t)ix->n_lists + 1) * 4, (cudaStream_t)cuda_stream));
  ICU(cudaMemsetAsync(ix->sync, 0, (size_t)OILBIRD_MAX_NQ * sizeof(LookupSync), (cudaStream_t)cuda_stream));
  ix->n_indexed = 0;
  ix->generation = ix->pool->generation;
  return OILBIRD_OK;
}

int oilbird_index_refresh(oilbird_index_t* ix, void* cuda_stream) {
  if (!ix) return OILBIRD_EINVAL;
  oilbird_pool* p = ix->pool;
  ICU(cudaSetDevice(p->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int64_t n = p->n_rows;
  // the pool was reset or evicted from since: its rows have other numbers now
  if (p->generation != ix->generation && ix->n_indexed > 0) return OILBIRD_EINVAL;
  if (n < ix->n_indexed) return OILBIRD_EINVAL;
  ix->generation = p->generation;
  if (n == ix->n_indexed) return OILBIRD_OK;
  // assign the new rows: their stored keys, a batch at a time, as queries against the centroids
  oilbird_query_params pr;
  oilbird_query_params_default(&pr);
  pr.k = 1; pr.theta = -INFINITY; pr.depth_mode = OILBIRD_DEPTH_FIXED; pr.cont_len = 1;
  for (int64_t r0 = ix->n_indexed; r0 < n; r0 += kIndexAssignBatch) {
    const int32_t nq = (int32_t)(n - r0 < kIndexAssignBatch ? n - r0 : kIndexAssignBatch);
    oilbird_query_out o;
    o.idx = ix->assign + r0; o.score = ix->a_score; o.fired = ix->a_fired;
    o.cont_len = ix->a_len; o.cont_tok = ix->a_tok;
    const uint16_t* states = p->keys + (size_t)r0 * p->r.d;       // the stored keys as queries
    if (p->r.e4m3) {
      // 8-bit pools: the stored rows as bf16 states (fp32(value(code) * scale) rounded to bf16)
      cudaError_t e = launch_pdl(dequant_rows_kernel, dim3(nq), dim3(256), 0, st,
                                 (const uint8_t*)p->codes, (const float*)p->scales, (int)p->r.d,
                                 (int)r0, ix->as_query);
      if (e != cudaSuccess) return index_fail(e, "dequantise kernel");
      p->launches += 1;
      states = ix->as_query;
    }
    int rc = oilbird_pool_query(ix->cent, states, nq, &pr, &o, st);
    if (rc) return rc;
  }
  // rebuild the lists over all indexed rows: count, offsets, scatter
  const int n_all = (int)n;
  int grid = (n_all + 255) / 256;
  if (grid > 4 * p->num_sms) grid = 4 * p->num_sms;
  ICU(cudaMemsetAsync(ix->counts, 0, (size_t)ix->n_lists * 4, st));
  cudaError_t e = launch_pdl(index_count_kernel, dim3(grid), dim3(256), 0, st,
                             (const int32_t*)ix->assign, n_all, ix->counts, ix->n_lists);
  if (e == cudaSuccess)
    e = launch_pdl(index_offsets_kernel, dim3(1), dim3(1024), 0, st, (const int32_t*)ix->counts,
                   ix->list_off, ix->cursor, ix->n_lists);
  if (e == cudaSuccess)
    e = launch_pdl(index_scatter_kernel, dim3(grid), dim3(256), 0, st, (const int32_t*)ix->assign,
                   n_all, (const int32_t*)ix->list_off, ix->cursor, ix->list_rows, ix->n_lists);
  if (e != cudaSuccess) return index_fail(e, "index list kernels");
  p->launches += 3;
  ix->n_indexed = n;
  return OILBIRD_OK;
}

int oilbird_index_train(oilbird_index_t* ix, int32_t iterations, void* cuda_stream) {
  if (!ix || iterations < 0) return OILBIRD_EINVAL;
  oilbird_pool* p = ix->pool;
  if (p->r.d > kMeanChunks * 256 * 8) return OILBIRD_EINVAL;
  ICU(cudaSetDevice(p->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  for (int32_t it = 0; it < iterations; ++it) {
    int rc = oilbird_index_reset(ix, cuda_stream);
    if (!rc) rc = oilbird_index_refresh(ix, cuda_stream);
    if (rc) return rc;
    if (ix->n_indexed == 0) break;                     // no rows: nothing to learn from
    cudaError_t e =
        p->r.e4m3 ? launch_pdl(index_means_e4m3_kernel, dim3(ix->n_lists), dim3(256), 0, st,
                               (const uint8_t*)p->codes, (const float*)p->scales, (int)p->r.d,
                               (const int32_t*)ix->list_off, (const int32_t*)ix->list_rows, ix->cent_raw)
                  : launch_pdl(index_means_kernel, dim3(ix->n_lists), dim3(256), 0, st,
                               (const uint16_t*)p->keys, (int)p->r.d, (const int32_t*)ix->list_off,
                               (const int32_t*)ix->list_rows, ix->cent_raw);
    if (e != cudaSuccess) return index_fail(e, "index means kernel");
    p->launches += 1;
    // the centroid pool, rebuilt from the new raw states (tokens are never looked at)
    rc = oilbird_pool_reset(ix->cent, cuda_stream);
    if (!rc)
      rc = oilbird_pool_append(ix->cent, ix->cent_raw, ix->cursor, ix->n_lists, 0, OILBIRD_NEW_TRACE,
                               cuda_stream);
    if (rc) return rc;
  }
  int rc = oilbird_index_reset(ix, cuda_stream);
  return rc ? rc : oilbird_index_refresh(ix, cuda_stream);
}

int oilbird_index_read_centroids(oilbird_index_t* ix, void* centroids_bf16_host) {
  if (!ix || !centroids_bf16_host) return OILBIRD_EINVAL;
  ICU(cudaSetDevice(ix->pool->device));
  ICU(cudaDeviceSynchronize());
  ICU(cudaMemcpy(centroids_bf16_host, ix->cent_raw, (size_t)ix->n_lists * ix->pool->r.d * 2,
                 cudaMemcpyDeviceToHost));
  return OILBIRD_OK;
}

int oilbird_index_query(oilbird_index_t* ix, const void* q_bf16, int32_t nq, int32_t n_probe,
                        const oilbird_query_params* pr, const oilbird_query_out* out,
                        void* cuda_stream) {
  if (!ix || !q_bf16 || !pr || !out || !out->idx || !out->score || !out->fired || !out->cont_len ||
      !out->cont_tok)
    return OILBIRD_EINVAL;
  oilbird_pool* p = ix->pool;
  GatherParams gp;
  int rc = check_query_params(nq, p->r.max_nq, p->r.max_k, pr, &gp);
  if (rc) return rc;
  if (n_probe < 1) return OILBIRD_EINVAL;
  if (n_probe > kIndexMaxProbe) n_probe = kIndexMaxProbe;
  if (((uintptr_t)q_bf16 & 15) || ((uintptr_t)pr->exclude_tag & 7) ||
      (((uintptr_t)out->idx | (uintptr_t)out->score | (uintptr_t)out->fired |
        (uintptr_t)out->cont_len | (uintptr_t)out->cont_tok) & 3)) {
    snprintf(g_index_err, sizeof g_index_err, "misaligned pointer");
    return OILBIRD_EINVAL;
  }
  // pool reset or evicted from since the lists were built: reset the index first
  if ((p->generation != ix->generation && ix->n_indexed > 0) || p->n_rows < ix->n_indexed)
    return OILBIRD_EINVAL;
  ICU(cudaSetDevice(p->device));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int kk = list_len(pr->k);
  PoolView pv = pool_view(p);
  const uint16_t* q = (const uint16_t*)q_bf16;
  if (nq <= kLookupMaxNq && n_probe <= 32 && pr->path == OILBIRD_PATH_AUTO) {
    // small batches: centroid scan, probes and candidate scan in one launch, then the merge
    if (preload_all_kernels() != cudaSuccess) return OILBIRD_ECUDA;
    // Twice the CTAs that fit at once (two per SM): the first half takes the centroids and
    // leaves, the second half moves in behind it, prepares the query while the probes are
    // being chosen, and takes the candidates; each side has the whole GPU for its round trips.
    // (Sharing one GPU-full of CTAs between the two sides, six to one: 17.4 us against 20.1 us
    // for an even split on 4,096 lists and ~1,000 candidates; this form is faster than both.)
    int g_all = 2 * p->num_sms / nq;
    if (g_all < 4) g_all = 4;
    if (g_all > kFoldMaxLists) g_all = kFoldMaxLists;
    int g1 = g_all, g2 = g_all;
    if (g1 > ix->cent->r.max_lists) g1 = ix->cent->r.max_lists;
    if (g2 > p->r.max_lists) g2 = p->r.max_lists;
    cudaError_t e;
#define LOOKUP(E, K8)                                                                             \
    launch_index_lookup<E, K8>(pv, p->codes, p->scales, ix->cent->keys, ix->n_lists, q, nq, pr->k,    \
                               g1, g2, n_probe, ix->probe_idx, ix->cent->partial, ix->sync,           \
                               ix->list_off, ix->list_rows, (int)ix->n_indexed, pr->exclude_tag,      \
                               p->partial, p->stats, gp, *out, st)
    if (p->r.e4m3) e = kk == 32 ? LOOKUP(1, true) : (kk == 64 ? LOOKUP(2, true) : LOOKUP(4, true));
    else e = kk == 32 ? LOOKUP(1, false) : (kk == 64 ? LOOKUP(2, false) : LOOKUP(4, false));
#undef LOOKUP
    if (e != cudaSuccess) return index_fail(e, "lookup launch");
    p->launches += 1;
    return OILBIRD_OK;
  }
  // probe: the n_probe best centroids of every query
  oilbird_query_params pp;
  oilbird_query_params_default(&pp);
  pp.k = n_probe; pp.theta = -INFINITY; pp.depth_mode = OILBIRD_DEPTH_FIXED; pp.cont_len = 1;
  oilbird_query_out po;
  po.idx = ix->probe_idx; po.score = ix->probe_score; po.fired = ix->probe_fired;
  po.cont_len = ix->probe_len; po.cont_tok = ix->probe_tok;
  rc = oilbird_pool_query(ix->cent, q_bf16, nq, &pp, &po, st);
  if (rc) return rc;
  // scan the candidates, merge, fire, gather
  // blocks per query: all the SMs twice over for a single lookup (a block holds a few rows
  // and the lookup is latency-bound), fewer per query as the batch grows (every block
  // prepares its query first, which a batch would otherwise pay thousands of times over)
  int grid = 2 * p->num_sms;
  if (nq > 1) {
    grid = (8 * p->num_sms + nq - 1) / nq;
    if (grid < 8) grid = 8;
    if (grid > 2 * p->num_sms) grid = 2 * p->num_sms;
  }
  if (grid > p->r.max_lists) grid = p->r.max_lists;
  cudaError_t e;
  if (p->r.e4m3) {
#define SCAN8(E)                                                                                  \
    launch_scan_ids_e4m3<E>(pv, p->codes, p->scales, q, nq, pr->k, ix->probe_idx, n_probe,       \
                            ix->list_off, ix->list_rows, (int)ix->n_indexed, pr->exclude_tag,     \
                            p->partial, p->q_valid, p->stats, grid, st)
    e = kk == 32 ? SCAN8(1) : (kk == 64 ? SCAN8(2) : SCAN8(4));
#undef SCAN8
  } else if (kk == 32)
    e = launch_scan_ids<1>(pv, q, nq, pr->k, ix->probe_idx, n_probe, ix->list_off, ix->list_rows,
                           (int)ix->n_indexed, pr->exclude_tag, p->partial, p->q_valid, p->stats, grid, st);
  else if (kk == 64)
    e = launch_scan_ids<2>(pv, q, nq, pr->k, ix->probe_idx, n_probe, ix->list_off, ix->list_rows,
                           (int)ix->n_indexed, pr->exclude_tag, p->partial, p->q_valid, p->stats, grid, st);
  else
    e = launch_scan_ids<4>(pv, q, nq, pr->k, ix->probe_idx, n_probe, ix->list_off, ix->list_rows,
                           (int)ix->n_indexed, pr->exclude_tag, p->partial, p->q_valid, p->stats, grid, st);
  if (e != cudaSuccess) return index_fail(e, "candidate scan launch");
  e = launch_merge_gather(pv, p->partial, grid, nq, kk, p->q_valid, gp, *out, st);
  if (e != cudaSuccess) return index_fail(e, "merge launch");
  p->launches += 2;
  return OILBIRD_OK;
}

int oilbird_index_read(oilbird_index_t* ix, int32_t* assign_host, int32_t* list_off_host,
                       int32_t* list_rows_host) {
  if (!ix) return OILBIRD_EINVAL;
  ICU(cudaSetDevice(ix->pool->device));
  ICU(cudaDeviceSynchronize());
  const size_t n = (size_t)ix->n_indexed;
  if (assign_host && n) ICU(cudaMemcpy(assign_host, ix->assign, n * 4, cudaMemcpyDeviceToHost));
  if (list_off_host)
    ICU(cudaMemcpy(list_off_host, ix->list_off, ((size_t)ix->n_lists + 1) * 4, cudaMemcpyDeviceToHost));
  if (list_rows_host && n) ICU(cudaMemcpy(list_rows_host, ix->list_rows, n * 4, cudaMemcpyDeviceToHost));
  return OILBIRD_OK;
}

}  // extern "C"

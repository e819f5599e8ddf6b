// 8-bit keys for a bounded store: append and CUDA-core scan for pools whose keys are
// FP8 E4M3 codes with one fp32 scale per row.
//
// The paper's Limitations section leaves "keeping the store bounded ... by eviction, an
// index, or quantization" as future work and fixes no format; the one implemented here:
//   v_j   = x_j / ||x||                       (double, as for 16-bit keys)
//   scale = fp32( max_j |v_j| / 448 )         (448 = largest finite E4M3 magnitude)
//   c_j   = e4m3_rne( v_j / scale )           (ties to the even code, saturating)
// and a score is fp32( scale * sum_j qn_j * value(c_j) ) with the query normalised and
// rounded to bf16 exactly as for 16-bit pools.  A row costs d + 4 bytes instead of 2d, so
// the scan, which is bound by the key stream, moves half the bytes.
//
// Everything after the scan (merge, firing rule, depth, gather) is format-independent and
// shared with the 16-bit path.  The tcgen05 scan is not offered for 8-bit pools (its query
// operand would have to be quantised to 8 bits too); batches of three queries and more go
// to the warp-level tensor scan (scan_mma.cu, codes as f16) where the width allows, else
// they run here two queries per pass.  As in the 16-bit scan, the rows of a serving step can be appended
// by the scan's first CTAs themselves (see FusedAppend).
#include <cuda_fp16.h>

#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"
#include "quant8.cuh"

namespace oilbird {

// One CTA per row.
__global__ void __launch_bounds__(kNormThreads, 4)
append_e4m3_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens,
                   int64_t n, int d, uint8_t* __restrict__ codes, float* __restrict__ scales,
                   int32_t* __restrict__ tok, int32_t* __restrict__ trace_id, int64_t row0,
                   int32_t trace, int32_t* __restrict__ trace_end,
                   uint64_t* __restrict__ trace_tag, uint64_t tag,
                   int64_t* __restrict__ trace_gbase, int64_t gbase, int set_tag,
                   DeviceStats* stats) {
  pdl_enter();   // earlier queries may still be reading the trace table and token stream
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) { trace_tag[trace] = tag; trace_gbase[trace] = gbase; }
  }
  for (int64_t r = blockIdx.x; r < n; r += gridDim.x) {
    const int64_t row = row0 + r;
    const bool ok = quantize_row_e4m3<true>(states + r * d, d, codes + row * d, scales + row);
    if (threadIdx.x == 0) {
      tok[row] = tokens[r];
      trace_id[row] = trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);           // stored as a zero key
    }
  }
}

cudaError_t launch_append_e4m3(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                               uint8_t* codes, float* scales, int32_t* tok, int32_t* trace_id,
                               int64_t row0, int32_t trace, int32_t* trace_end,
                               uint64_t* trace_tag, uint64_t tag, int64_t* trace_gbase,
                               int64_t gbase, int set_tag, DeviceStats* stats, cudaStream_t st) {
  int64_t grid = n < 1 ? 1 : (n > 65535 * 8 ? 65535 * 8 : n);
  return launch_pdl(append_e4m3_kernel, dim3((unsigned)grid), dim3(kNormThreads), 0, st, states,
                    tokens, n, d, codes, scales, tok, trace_id, row0, trace, trace_end, trace_tag,
                    tag, trace_gbase, gbase, set_tag, stats);
}

// ----------------------------------------------------------------------- scan ---
constexpr int kQ8Threads = kNormThreads;
constexpr int kQ8Warps = kQ8Threads / 32;
constexpr int kQ8Rows = 4;        // rows a warp scores together

// Same structure as the 16-bit CUDA-core scan: 2 CTAs x 8 warps per SM, contiguous row
// split, 16-byte streaming loads (16 codes), the normalised bf16 queries in shared memory,
// fp32 accumulation, per-warp sorted register lists, one list per CTA and query.
template <int QT, int E>
__global__ void __launch_bounds__(kQ8Threads, 2)
scan_gemv_e4m3_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                      PoolView pv, const uint16_t* __restrict__ q_raw, int nq, int k,
                      const uint64_t* __restrict__ exclude_tag, u64* __restrict__ partial,
                      int32_t* __restrict__ q_valid, DeviceStats* stats, FusedAppend fa) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int KK = 32 * E;
  pdl_enter();
  const int d = pv.d, n8 = d >> 3, n16 = d >> 4;
  uint4* qs = reinterpret_cast<uint4*>(smem_raw);                        // [QT][n8] bf16
  u64* scratch = reinterpret_cast<u64*>(smem_raw + (size_t)QT * d * 2);   // [warps][KK]
  __shared__ uint64_t s_ex[QT];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // contiguous, balanced share of the rows; the fa.n CTAs that first append a row of this
  // step take 1/16 less (quantising a row costs about twice what normalising one does)
  const int64_t n = pv.n_rows;
  const int64_t w_lo = 16ll * blockIdx.x - min((int)blockIdx.x, fa.n);
  const int64_t w_hi = 16ll * (blockIdx.x + 1) - min((int)blockIdx.x + 1, fa.n);
  const int64_t w_all = 16ll * gridDim.x - min((int)gridDim.x, fa.n);
  const int r_lo = (int)((n * w_lo) / w_all);
  const int r_hi = (int)((n * w_hi) / w_all);
  const uint4* codes4 = reinterpret_cast<const uint4*>(codes);

  // the step's append, one row per CTA (as in the 16-bit scan)
  if ((int)blockIdx.x < fa.n) {
    const int r = blockIdx.x;
    const int64_t row = (int64_t)fa.row0 + r;
    const bool ok = quantize_row_e4m3<true>(fa.states + (size_t)r * d, d,
                                      const_cast<uint8_t*>(codes) + row * d,
                                      const_cast<float*>(scales) + row);
    if (threadIdx.x == 0) {
      fa.tok[row] = fa.tokens[r];
      fa.trace_id[row] = fa.trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);
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
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      uint16_t* dst = reinterpret_cast<uint16_t*>(qs + (size_t)q * n8);
      if (q0 + q < nq) {
        const int code = normalize_row<false>(q_raw + (size_t)(q0 + q) * d, dst, d);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
          q_valid[q0 + q] = code == kRowNonFinite ? 0 : 1;
          if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
        }
      } else {
        for (int c = threadIdx.x; c < n8; c += kQ8Threads) qs[(size_t)q * n8 + c] = make_uint4(0, 0, 0, 0);
      }
    }
    if (threadIdx.x < QT)
      s_ex[threadIdx.x] = (exclude_tag && q0 + threadIdx.x < nq) ? exclude_tag[q0 + threadIdx.x] : 0;
    __syncthreads();

    u64 top[QT][E];
    u64 kth[QT];
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      kth[q] = 0;
#pragma unroll
      for (int r = 0; r < E; ++r) top[q][r] = 0;
    }

    for (int rb = r_lo + warp * kQ8Rows; rb < r_hi; rb += kQ8Warps * kQ8Rows) {
      const uint4* rowp[kQ8Rows];
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r) {
        const int row = rb + r < r_hi ? rb + r : r_hi - 1;      // clamp: result discarded below
        rowp[r] = codes4 + (size_t)row * n16;
      }
      float acc[kQ8Rows][QT];
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r)
#pragma unroll
        for (int q = 0; q < QT; ++q) acc[r][q] = 0.f;

      const bool fresh = fa.n > 0 && rb + kQ8Rows > fa.row0;       // warp-uniform
      if (fresh && !fresh_ok) {
        wait_fused_rows(fa, stats);       // rows of this step's append
        fresh_ok = true;
      }
      // the rows' scales are asked for ahead of the codes, not behind the sums
      float sc[kQ8Rows];
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r) {
        const int row = rb + r < r_hi ? rb + r : r_hi - 1;
        sc[r] = (fa.n > 0 && row >= fa.row0) ? __ldcg(scales + row) : scales[row];
      }
#pragma unroll 4
      for (int c = lane; c < n16; c += 32) {
        uint4 kv[kQ8Rows];
#pragma unroll
        for (int r = 0; r < kQ8Rows; ++r)
          kv[r] = fresh ? ld_cg16(rowp[r] + c) : ld_stream16(rowp[r] + c);
        uint4 qv[QT][2];
#pragma unroll
        for (int q = 0; q < QT; ++q) { qv[q][0] = qs[q * n8 + 2 * c]; qv[q][1] = qs[q * n8 + 2 * c + 1]; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {                     // word j of the 16 bytes: 4 codes
          float2 ka[kQ8Rows], kb[kQ8Rows];
#pragma unroll
          for (int r = 0; r < kQ8Rows; ++r) {
            const uint32_t w = j == 0 ? kv[r].x : (j == 1 ? kv[r].y : (j == 2 ? kv[r].z : kv[r].w));
            ka[r] = e4m3x2_to_float2(w & 0xffffu);
            kb[r] = e4m3x2_to_float2(w >> 16);
          }
#pragma unroll
          for (int q = 0; q < QT; ++q) {
            // elements 4j..4j+3 of the chunk: query words 2j and 2j+1 of its 8
            const uint4 h = qv[q][j >> 1];
            const uint32_t w0 = (j & 1) ? h.z : h.x, w1 = (j & 1) ? h.w : h.y;
            const float q0f = bf16_lo(w0), q1f = bf16_hi(w0), q2f = bf16_lo(w1), q3f = bf16_hi(w1);
#pragma unroll
            for (int r = 0; r < kQ8Rows; ++r) {
              float a = acc[r][q];
              a = fmaf(ka[r].x, q0f, a);
              a = fmaf(ka[r].y, q1f, a);
              a = fmaf(kb[r].x, q2f, a);
              a = fmaf(kb[r].y, q3f, a);
              acc[r][q] = a;
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kQ8Rows; ++r) {
        const int row = rb + r;
        if (row >= r_hi) break;                             // warp-uniform
        const bool fresh_row = fa.n > 0 && row >= fa.row0;     // written by another CTA just now
        uint64_t tag = 0;
        if (exclude_tag)
          tag = fresh_row ? __ldcg(&pv.trace_tag[__ldcg(&pv.trace_id[row])])
                          : pv.trace_tag[pv.trace_id[row]];
#pragma unroll
        for (int q = 0; q < QT; ++q) {
          const float s = warp_sum(acc[r][q]) * sc[r];
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
#pragma unroll
    for (int q = 0; q < QT; ++q) {
      if (q0 + q >= nq) break;
      block_merge_desc<E>(top[q], scratch, kQ8Warps);
      if (threadIdx.x < 32) {
        u64* dst = partial + ((size_t)blockIdx.x * nq + (q0 + q)) * KK;
#pragma unroll
        for (int r = 0; r < E; ++r) dst[r * 32 + lane] = top[q][r];
      }
    }
  }
}

template <int QT, int E>
static cudaError_t launch_q8(const uint8_t* codes, const float* scales, const PoolView& pv,
                             const uint16_t* q_raw, int nq, int k, const uint64_t* ex, u64* partial,
                             int32_t* q_valid, DeviceStats* stats, int grid, const FusedAppend& fa,
                             cudaStream_t st) {
  const size_t smem = (size_t)QT * pv.d * 2 + (size_t)kQ8Warps * 32 * E * sizeof(u64);
  return launch_pdl(scan_gemv_e4m3_kernel<QT, E>, dim3(grid), dim3(kQ8Threads), smem, st, codes,
                    scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, fa);
}

template <int QT>
static cudaError_t launch_q8_qt(int kk, const uint8_t* codes, const float* scales,
                                const PoolView& pv, const uint16_t* q_raw, int nq, int k,
                                const uint64_t* ex, u64* partial, int32_t* q_valid,
                                DeviceStats* stats, int grid, const FusedAppend& fa,
                                cudaStream_t st) {
  if (kk == 32) return launch_q8<QT, 1>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  if (kk == 64) return launch_q8<QT, 2>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
  return launch_q8<QT, 4>(codes, scales, pv, q_raw, nq, k, ex, partial, q_valid, stats, grid, fa, st);
}

cudaError_t launch_scan_gemv_e4m3(const uint8_t* codes, const float* scales, const PoolView& pv,
                                  const uint16_t* q_raw, int32_t nq, int32_t k, int32_t kk,
                                  const uint64_t* exclude_tag, unsigned long long* partial,
                                  int32_t* q_valid, DeviceStats* stats, int32_t max_lists,
                                  int32_t num_sms, int32_t* n_lists, const FusedAppend* fused,
                                  cudaStream_t st) {
  const int grid = scan_gemv_grid(pv.n_rows, num_sms, max_lists);
  *n_lists = grid;
  FusedAppend fa = {};
  if (fused) {
    if (fused->n > grid || fused->n > kFuseMaxRows) return cudaErrorInvalidValue;
    fa = *fused;
  }
  if (nq >= 2)
    return launch_q8_qt<2>(kk, codes, scales, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
  return launch_q8_qt<1>(kk, codes, scales, pv, q_raw, nq, k, exclude_tag, partial, q_valid, stats, grid, fa, st);
}

cudaError_t preload_quant8_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(append_e4m3_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_e4m3_kernel<1, 1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_e4m3_kernel<1, 2>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_e4m3_kernel<1, 4>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_e4m3_kernel<2, 1>, true)) != cudaSuccess) return e;
  if ((e = preload_kernel(scan_gemv_e4m3_kernel<2, 2>, true)) != cudaSuccess) return e;
  return preload_kernel(scan_gemv_e4m3_kernel<2, 4>, true);
}

}  // namespace oilbird

// K1 append / query normalisation.
//
// Store step of the paper (Section 4 "(i) Store", Eq. 1): each committed position's
// hidden state is kept L2-normalised in half precision next to its token.  The same
// normalisation is applied to the query states so that the cosine of Algorithm 1's
// scoring line is a plain dot product of two stored-format vectors.
//
// One CTA per row (see normalize.cuh for the arithmetic).  The work is a single pass
// over n*d*2 bytes in and out.  Measured on bulk loads (tens of thousands of rows per call):
// 5.7 TB/s read+write at d = 8192 and 5.1 TB/s at d = 4096, where the per-row block
// reduction (three barriers and one thread's square root and division per 8 KB) weighs more
// and a block therefore takes two rows at a time.
// Before the conversion-free fast path of normalize.cuh the kernel sat at 4.4 TB/s with the
// conversion unit as its busiest pipe.
#include <cuda_fp16.h>

#include "common.cuh"
#include "internal.h"
#include "normalize.cuh"

namespace oilbird {

__global__ void __launch_bounds__(kNormThreads, 4)
append_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens, int64_t n,
              int d, uint16_t* __restrict__ keys, int32_t* __restrict__ tok,
              int32_t* __restrict__ trace_id, int64_t row0, int32_t trace,
              int32_t* __restrict__ trace_end, uint64_t* __restrict__ trace_tag, uint64_t tag,
              int64_t* __restrict__ trace_gbase, int64_t gbase, int set_tag, DeviceStats* stats) {
  pdl_enter();   // earlier queries may still be reading the trace table and token stream
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) { trace_tag[trace] = tag; trace_gbase[trace] = gbase; }
  }
  for (int64_t r = blockIdx.x; r < n; r += gridDim.x) {
    const int64_t row = row0 + r;
    const int code = normalize_row<true, 4, true>(states + r * d, keys + row * d, d);
    if (threadIdx.x == 0) {
      tok[row] = tokens[r];
      trace_id[row] = trace;
      if (code != kRowOk) atomicAdd(&stats->degenerate_rows, 1ull);  // stored as a zero key
    }
  }
}

// Bulk form of the append (trace loads of thousands of rows): a grid of a few blocks per SM
// walks the rows, and each block issues the loads of its next row before it reduces and
// writes the current one, so that the row-to-row dependency (load, block reduction, store)
// no longer leaves the memory system idle between rows.  Same arithmetic, same results.
template <int kHeld>
__global__ void __launch_bounds__(kNormThreads, 4)
append_bulk_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens,
                   int64_t n, int d, uint16_t* __restrict__ keys, int32_t* __restrict__ tok,
                   int32_t* __restrict__ trace_id, int64_t row0, int32_t trace,
                   int32_t* __restrict__ trace_end, uint64_t* __restrict__ trace_tag, uint64_t tag,
                   int64_t* __restrict__ trace_gbase, int64_t gbase, int set_tag,
                   DeviceStats* stats) {
  pdl_enter();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) { trace_tag[trace] = tag; trace_gbase[trace] = gbase; }
  }
  uint4 cur[kHeld], nxt[kHeld];
  int64_t r = blockIdx.x;
  if (r < n) load_row_chunks<kHeld>(states + r * d, d, cur);
  for (; r < n; r += gridDim.x) {
    const int64_t rn = r + gridDim.x;
    if (rn < n) load_row_chunks<kHeld>(states + rn * d, d, nxt);
    const int64_t row = row0 + r;
    const int code = normalize_row_regs<true, kHeld, true>(cur, states + r * d, keys + row * d, d);
    if (threadIdx.x == 0) {
      tok[row] = tokens[r];
      trace_id[row] = trace;
      if (code != kRowOk) atomicAdd(&stats->degenerate_rows, 1ull);
    }
#pragma unroll
    for (int i = 0; i < kHeld; ++i) cur[i] = nxt[i];
  }
}

// Bulk append of rows that fit two chunks per thread (d <= 4096): a block takes two rows at
// a time (normalize_two_rows_fast), which halves the barriers and the one-thread arithmetic
// per row, and loads the next pair while it works on this one.
__global__ void __launch_bounds__(kNormThreads, 4)
append_bulk2_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens,
                    int64_t n, int d, uint16_t* __restrict__ keys, int32_t* __restrict__ tok,
                    int32_t* __restrict__ trace_id, int64_t row0, int32_t trace,
                    int32_t* __restrict__ trace_end, uint64_t* __restrict__ trace_tag, uint64_t tag,
                    int64_t* __restrict__ trace_gbase, int64_t gbase, int set_tag,
                    DeviceStats* stats) {
  constexpr int kHeld = 2;
  pdl_enter();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) { trace_tag[trace] = tag; trace_gbase[trace] = gbase; }
  }
  uint4 ca[kHeld], cb[kHeld], na[kHeld], nb[kHeld];
  const int64_t stride = 2ll * gridDim.x;
  int64_t r = 2ll * blockIdx.x;
  if (r < n) load_row_chunks<kHeld>(states + r * d, d, ca);
  if (r + 1 < n) load_row_chunks<kHeld>(states + (r + 1) * d, d, cb);
  for (; r < n; r += stride) {
    const int64_t rn = r + stride;
    if (rn < n) load_row_chunks<kHeld>(states + rn * d, d, na);
    if (rn + 1 < n) load_row_chunks<kHeld>(states + (rn + 1) * d, d, nb);
    const int64_t row = row0 + r;
    int code_a, code_b = kRowOk;
    if (r + 1 < n) {
      normalize_two_rows_fast<kHeld>(ca, cb, keys + row * d, keys + (row + 1) * d, d, code_a, code_b);
      if (code_a < 0)
        code_a = normalize_row_regs<true, kHeld, false>(ca, states + r * d, keys + row * d, d);
      if (code_b < 0)
        code_b = normalize_row_regs<true, kHeld, false>(cb, states + (r + 1) * d, keys + (row + 1) * d, d);
    } else {
      code_a = normalize_row_regs<true, kHeld, true>(ca, states + r * d, keys + row * d, d);
    }
    if (threadIdx.x < 2 && r + threadIdx.x < n) {
      tok[row + threadIdx.x] = tokens[r + threadIdx.x];
      trace_id[row + threadIdx.x] = trace;
      if ((threadIdx.x ? code_b : code_a) != kRowOk) atomicAdd(&stats->degenerate_rows, 1ull);
    }
#pragma unroll
    for (int i = 0; i < kHeld; ++i) { ca[i] = na[i]; cb[i] = nb[i]; }
  }
}

__global__ void __launch_bounds__(kNormThreads)
qnorm_kernel(const uint16_t* __restrict__ q, int nq, int d, uint16_t* __restrict__ qn,
             int32_t* __restrict__ q_valid, DeviceStats* stats, float* __restrict__ xchg,
             int n_xchg, int f16_scaled) {
  pdl_enter();
  // the tensor scan's cross-CTA threshold exchange starts every call at -inf
  for (int i = blockIdx.x * kNormThreads + threadIdx.x; i < n_xchg; i += gridDim.x * kNormThreads)
    xchg[i] = -INFINITY;
  if (blockIdx.x == 0 && threadIdx.x < kTcXchgCounters && n_xchg > 0)
    reinterpret_cast<unsigned*>(xchg + n_xchg)[threadIdx.x] = 0u;
  const int r = blockIdx.x;
  if (r < nq) {
    // A query holding NaN/Inf returns no neighbours; an all-zero query is legal and
    // scores 0 against every row.
    const int code = normalize_row(q + (size_t)r * d, qn + (size_t)r * d, d);
    if (threadIdx.x == 0) {
      q_valid[r] = code == kRowNonFinite ? 0 : 1;
      if (code == kRowNonFinite) atomicAdd(&stats->nonfinite_queries, 1ull);
    }
    if (f16_scaled) {
      // the normalised bf16 query as f16 scaled by 2^14, as the warp-level scan of 8-bit
      // pools holds it (exact but for elements below 2^-31)
      __syncthreads();
      uint32_t* w32 = reinterpret_cast<uint32_t*>(qn + (size_t)r * d);
      for (int i = threadIdx.x; i < d / 2; i += kNormThreads) {
        const uint32_t w = w32[i];
        const __half2 h = __floats2half2_rn(bf16_lo(w) * 16384.f, bf16_hi(w) * 16384.f);
        w32[i] = *reinterpret_cast<const uint32_t*>(&h);
      }
    }
  } else {
    uint4* dst4 = reinterpret_cast<uint4*>(qn + (size_t)r * d);
    for (int c = threadIdx.x; c < (d >> 3); c += kNormThreads) dst4[c] = make_uint4(0, 0, 0, 0);
  }
}

cudaError_t launch_append(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                          uint16_t* keys, int32_t* tok, int32_t* trace_id, int64_t row0,
                          int32_t trace, int32_t* trace_end, uint64_t* trace_tag, uint64_t tag,
                          int64_t* trace_gbase, int64_t gbase, int set_tag, DeviceStats* stats,
                          int32_t num_sms, cudaStream_t st) {
  // from a few rows per resident block on, the prefetching kernel
  const int64_t bulk_grid = (int64_t)num_sms * 4;
  if (n >= bulk_grid * 4) {
    if (d <= 4096)
      return launch_pdl(append_bulk2_kernel, dim3((unsigned)bulk_grid), dim3(kNormThreads), 0, st,
                        states, tokens, n, d, keys, tok, trace_id, row0, trace, trace_end,
                        trace_tag, tag, trace_gbase, gbase, set_tag, stats);
    return launch_pdl(append_bulk_kernel<4>, dim3((unsigned)bulk_grid), dim3(kNormThreads), 0, st,
                      states, tokens, n, d, keys, tok, trace_id, row0, trace, trace_end, trace_tag,
                      tag, trace_gbase, gbase, set_tag, stats);
  }
  int64_t grid = n < 1 ? 1 : (n > 65535 * 8 ? 65535 * 8 : n);
  return launch_pdl(append_kernel, dim3((unsigned)grid), dim3(kNormThreads), 0, st, states, tokens,
                    n, d, keys, tok, trace_id, row0, trace, trace_end, trace_tag, tag, trace_gbase,
                    gbase, set_tag, stats);
}

cudaError_t launch_qnorm(const uint16_t* q, int32_t nq, int32_t nq_pad, int32_t d, uint16_t* qn,
                         int32_t* q_valid, DeviceStats* stats, float* xchg, int32_t n_xchg,
                         bool f16_scaled, cudaStream_t st) {
  return launch_pdl(qnorm_kernel, dim3(nq_pad), dim3(kNormThreads), 0, st, q, nq, d, qn, q_valid,
                    stats, xchg, n_xchg, f16_scaled ? 1 : 0);
}

cudaError_t preload_append_kernels() {
  cudaError_t e;
  if ((e = preload_kernel(append_kernel)) != cudaSuccess) return e;
  if ((e = preload_kernel(append_bulk_kernel<4>)) != cudaSuccess) return e;
  if ((e = preload_kernel(append_bulk2_kernel)) != cudaSuccess) return e;
  return preload_kernel(qnorm_kernel);
}

}  // namespace oilbird

// K1 append / query normalisation.
//
// Store step of the paper (Section 4 "(i) Store", Eq. 1): each committed position's
// hidden state is kept L2-normalised in half precision next to its token.  The same
// normalisation is applied to the query states so that the cosine of Algorithm 1's
// scoring line is a plain dot product of two stored-format vectors.
//
// One CTA per row.  The squared norm is accumulated in double precision (products of
// bf16 values are exact there), the scale 1/sqrt is IEEE double, and each element is
// rounded once to float and once to bf16 (nearest even).  The work is a single pass
// over n*d*2 bytes in and out; it is bound by HBM traffic, not by the fp64 pipe.
#include "common.cuh"
#include "internal.h"

namespace oilbird {

constexpr int kNormThreads = 256;

// Normalise one row of d bf16 values (d % 8 == 0) from src to dst.  All threads of the
// block take part.  Returns (to every thread) whether the row was usable.
__device__ bool normalize_row(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst,
                              int d) {
  __shared__ double s_part[kNormThreads / 32];
  __shared__ int s_bad[kNormThreads / 32];
  __shared__ double s_inv;
  const int n_chunks = d >> 3;
  const uint4* src4 = reinterpret_cast<const uint4*>(src);
  double ss = 0.0;
  int bad = 0;
  for (int c = threadIdx.x; c < n_chunks; c += kNormThreads) {
    uint4 v = __ldg(src4 + c);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float lo = bf16_lo(w[i]), hi = bf16_hi(w[i]);
      bad |= ((w[i] & 0x7f80u) == 0x7f80u) | ((w[i] & 0x7f800000u) == 0x7f800000u);
      ss += (double)lo * (double)lo;
      ss += (double)hi * (double)hi;
    }
  }
#pragma unroll
  for (int m = 16; m; m >>= 1) {
    ss += __shfl_xor_sync(0xffffffffu, ss, m);
    bad |= __shfl_xor_sync(0xffffffffu, bad, m);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { s_part[warp] = ss; s_bad[warp] = bad; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    int b = 0;
    for (int w = 0; w < kNormThreads / 32; ++w) { tot += s_part[w]; b |= s_bad[w]; }
    double nrm = sqrt(tot);
    bool ok = !b && nrm > 0.0 && isfinite(nrm);
    s_inv = ok ? 1.0 / nrm : 0.0;
  }
  __syncthreads();
  const double inv = s_inv;
  uint4* dst4 = reinterpret_cast<uint4*>(dst);
  for (int c = threadIdx.x; c < n_chunks; c += kNormThreads) {
    uint4 v = __ldg(src4 + c);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (inv == 0.0) { o[i] = 0; continue; }
      float lo = __double2float_rn((double)bf16_lo(w[i]) * inv);
      float hi = __double2float_rn((double)bf16_hi(w[i]) * inv);
      o[i] = f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
    }
    dst4[c] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  return inv != 0.0;
}

__global__ void __launch_bounds__(kNormThreads)
append_kernel(const uint16_t* __restrict__ states, const int32_t* __restrict__ tokens, int64_t n,
              int d, uint16_t* __restrict__ keys, int32_t* __restrict__ tok,
              int32_t* __restrict__ trace_id, int64_t row0, int32_t trace,
              int32_t* __restrict__ trace_end, uint64_t* __restrict__ trace_tag, uint64_t tag,
              int set_tag, DeviceStats* stats) {
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    trace_end[trace] = (int32_t)(row0 + n);
    if (set_tag) trace_tag[trace] = tag;
  }
  for (int64_t r = blockIdx.x; r < n; r += gridDim.x) {
    const int64_t row = row0 + r;
    bool ok = normalize_row(states + r * d, keys + row * d, d);
    if (threadIdx.x == 0) {
      tok[row] = tokens[r];
      trace_id[row] = trace;
      if (!ok) atomicAdd(&stats->degenerate_rows, 1ull);  // zero or non-finite input row
    }
    __syncthreads();  // shared scratch of normalize_row is reused by the next row
  }
}

__global__ void __launch_bounds__(kNormThreads)
qnorm_kernel(const uint16_t* __restrict__ q, int nq, int d, uint16_t* __restrict__ qn,
             int32_t* __restrict__ q_valid, DeviceStats* stats) {
  const int r = blockIdx.x;
  if (r < nq) {
    // A query holding NaN/Inf returns no neighbours; an all-zero query is legal and
    // scores 0 against every row.
    __shared__ int s_nonfinite;
    if (threadIdx.x == 0) s_nonfinite = 0;
    __syncthreads();
    const uint4* src4 = reinterpret_cast<const uint4*>(q + (size_t)r * d);
    int bad = 0;
    for (int c = threadIdx.x; c < (d >> 3); c += kNormThreads) {
      uint4 v = __ldg(src4 + c);
      uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
        bad |= ((w[i] & 0x7f80u) == 0x7f80u) | ((w[i] & 0x7f800000u) == 0x7f800000u);
    }
    if (bad) s_nonfinite = 1;
    __syncthreads();
    normalize_row(q + (size_t)r * d, qn + (size_t)r * d, d);
    if (threadIdx.x == 0) {
      q_valid[r] = s_nonfinite ? 0 : 1;
      if (s_nonfinite) atomicAdd(&stats->nonfinite_queries, 1ull);
    }
  } else {
    uint4* dst4 = reinterpret_cast<uint4*>(qn + (size_t)r * d);
    for (int c = threadIdx.x; c < (d >> 3); c += kNormThreads) dst4[c] = make_uint4(0, 0, 0, 0);
  }
}

cudaError_t launch_append(const uint16_t* states, const int32_t* tokens, int64_t n, int32_t d,
                          uint16_t* keys, int32_t* tok, int32_t* trace_id, int64_t row0,
                          int32_t trace, int32_t* trace_end, uint64_t* trace_tag, uint64_t tag,
                          int set_tag, DeviceStats* stats, cudaStream_t st) {
  int64_t grid = n < 1 ? 1 : (n > 65535 * 8 ? 65535 * 8 : n);
  append_kernel<<<(unsigned)grid, kNormThreads, 0, st>>>(states, tokens, n, d, keys, tok, trace_id,
                                                         row0, trace, trace_end, trace_tag, tag,
                                                         set_tag, stats);
  return cudaGetLastError();
}

cudaError_t launch_qnorm(const uint16_t* q, int32_t nq, int32_t nq_pad, int32_t d, uint16_t* qn,
                         int32_t* q_valid, DeviceStats* stats, cudaStream_t st) {
  qnorm_kernel<<<nq_pad, kNormThreads, 0, st>>>(q, nq, d, qn, q_valid, stats);
  return cudaGetLastError();
}

}  // namespace oilbird

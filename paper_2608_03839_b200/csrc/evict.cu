// Eviction for a bounded store: drop the oldest traces and move what remains to the front.
//
// The paper's Limitations section names eviction as one way to keep the store bounded and
// defines no policy; the one here is oldest first, by whole traces, and the result is exactly
// the pool that the remaining traces alone would have built (rows and traces renumbered from
// zero).  Moving the live rows down by `head` rows in place is an overlapping copy, done in
// waves by one cooperative kernel (all blocks resident together, so its grid-wide barriers
// cannot dead-lock).  Two forms:
//   - a large evicted prefix (at least one wave of bytes): waves of `head` rows; a wave's
//     source and destination are disjoint and a wave's source is the next wave's
//     destination, so the whole grid streams one wave and meets at a barrier;
//   - a small prefix (one short trace in front of millions of rows): waves of a fixed size
//     (a few chunks per thread, ~10 MB per wave on a B200) staged through registers: every
//     thread loads its chunks of the NEXT wave, stores the chunks it holds of THIS wave,
//     and the barrier sits between a wave's loads and its stores.  The number of barriers
//     is live bytes / wave bytes whatever `head` is (waves of `head` rows would need
//     live / head barriers: two million for one row in front of a 2M-row pool).
// Bound by HBM: the live bytes are read once and written once.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"

namespace cg = cooperative_groups;

namespace oilbird {

constexpr int kEvictThreads = 512;

constexpr int kWaveChunks = 4;       // elements a thread holds per wave of the staged form

// a[0, n) <- a[shift, shift + n) for any shift >= 1, staged through registers (see above).
// Every thread of the grid calls this with the same arguments.  sub is subtracted from each
// element on the way (trace ids; T = int32_t) when kSub is set.
template <typename T, bool kSub>
__device__ __forceinline__ void shift_down_staged(cg::grid_group& grid, T* a, int64_t shift,
                                                  int64_t n, int32_t sub) {
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
  const int64_t wave = nthreads * kWaveChunks;
  T cur[kWaveChunks], nxt[kWaveChunks];
#pragma unroll
  for (int c = 0; c < kWaveChunks; ++c) {
    const int64_t i = tid + c * nthreads;
    if (i < n) cur[c] = __ldcg(a + shift + i);
  }
  for (int64_t w0 = 0; w0 < n; w0 += wave) {
    // behind this barrier every load of wave w0 has completed (its sources may now be
    // overwritten) and every store of the wave before it has been issued
    grid.sync();
#pragma unroll
    for (int c = 0; c < kWaveChunks; ++c) {
      const int64_t i = w0 + wave + tid + c * nthreads;        // next wave: beyond all of this
      if (i < n) nxt[c] = __ldcg(a + shift + i);               // wave's destinations
    }
#pragma unroll
    for (int c = 0; c < kWaveChunks; ++c) {
      const int64_t i = w0 + tid + c * nthreads;
      if (i < n) {
        if constexpr (kSub) a[i] = cur[c] - sub;
        else a[i] = cur[c];
      }
    }
#pragma unroll
    for (int c = 0; c < kWaveChunks; ++c) cur[c] = nxt[c];
  }
  grid.sync();      // the next array's first loads must not pass these stores (same thread
                    // order would do; the barrier keeps the reasoning per array)
}

// keys: live rows of `row_bytes` bytes each (a multiple of 16); scales: fp32 per row or
// nullptr; tok, trace_id: int32 per row (trace ids drop by n_traces).
__global__ void __launch_bounds__(kEvictThreads)
compact_kernel(unsigned char* keys, float* scales, int32_t* tok, int32_t* trace_id, int64_t head,
               int64_t live, int64_t row_bytes, int32_t n_traces) {
  cg::grid_group grid = cg::this_grid();
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
  const int64_t chunks_per_row = row_bytes >> 4;
  if (head == 0) {
    // only empty traces were dropped: nothing moves, but the traces are renumbered
    for (int64_t i = tid; i < live; i += nthreads) trace_id[i] -= n_traces;
    return;
  }
  if (head * chunks_per_row < nthreads * kWaveChunks) {
    // small evicted prefix: fixed waves through registers
    shift_down_staged<uint4, false>(grid, reinterpret_cast<uint4*>(keys), head * chunks_per_row,
                                    live * chunks_per_row, 0);
    shift_down_staged<int32_t, false>(grid, tok, head, live, 0);
    shift_down_staged<int32_t, true>(grid, trace_id, head, live, n_traces);
    if (scales) shift_down_staged<int32_t, false>(grid, reinterpret_cast<int32_t*>(scales), head, live, 0);
    return;
  }
  for (int64_t w0 = 0; w0 < live; w0 += head) {
    const int64_t rows = live - w0 < head ? live - w0 : head;
    // keys: rows [w0, w0+rows) <- rows [w0+head, ...), 16 bytes per thread and step
    const uint4* src = reinterpret_cast<const uint4*>(keys + (w0 + head) * row_bytes);
    uint4* dst = reinterpret_cast<uint4*>(keys + w0 * row_bytes);
    const int64_t n16 = rows * chunks_per_row;
    int64_t i = tid;
    for (; i + 3 * nthreads < n16; i += 4 * nthreads) {        // four loads in flight per thread
      const uint4 a = __ldcs(src + i), b = __ldcs(src + i + nthreads),
                  c = __ldcs(src + i + 2 * nthreads), e = __ldcs(src + i + 3 * nthreads);
      __stcs(dst + i, a);
      __stcs(dst + i + nthreads, b);
      __stcs(dst + i + 2 * nthreads, c);
      __stcs(dst + i + 3 * nthreads, e);
    }
    for (; i < n16; i += nthreads) __stcs(dst + i, __ldcs(src + i));
    for (int64_t i = tid; i < rows; i += nthreads) {
      tok[w0 + i] = __ldcg(tok + w0 + head + i);
      trace_id[w0 + i] = __ldcg(trace_id + w0 + head + i) - n_traces;
      if (scales) scales[w0 + i] = __ldcg(scales + w0 + head + i);
    }
    grid.sync();
  }
}

cudaError_t launch_compact(unsigned char* keys, float* scales, int32_t* tok, int32_t* trace_id,
                           int64_t head, int64_t live, int64_t row_bytes, int32_t n_traces,
                           int32_t num_sms, cudaStream_t st) {
  if (live <= 0 || head < 0 || n_traces <= 0) return cudaSuccess;
  int per_sm = 0;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compact_kernel,
                                                                kEvictThreads, 0);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  if (per_sm > 2) per_sm = 2;
  const int grid = per_sm * num_sms;            // all blocks resident: required by grid.sync()
  void* args[] = {&keys, &scales, &tok, &trace_id, &head, &live, &row_bytes, &n_traces};
  return cudaLaunchCooperativeKernel((void*)compact_kernel, dim3(grid), dim3(kEvictThreads), args, 0,
                                     st);
}

cudaError_t preload_evict_kernels() { return preload_kernel(compact_kernel); }

}  // namespace oilbird

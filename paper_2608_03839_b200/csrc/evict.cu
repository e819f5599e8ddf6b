// Eviction for a bounded store: drop the oldest traces and move what remains to the front.
//
// The paper's Limitations section names eviction as one way to keep the store bounded and
// defines no policy; the one here is oldest first, by whole traces, and the result is exactly
// the pool that the remaining traces alone would have built (rows and traces renumbered from
// zero).  Moving the live rows down by `head` rows in place is an overlapping copy: it is
// done in waves of `head` rows (a wave's source and destination are disjoint, and a wave's
// source is the next wave's destination), the whole grid working on one wave and a grid-wide
// barrier between waves.  The kernel is launched cooperatively, so all its blocks are
// resident together and the barrier cannot dead-lock.  Bound by HBM: the live bytes are read
// once and written once.
#include <cooperative_groups.h>

#include "common.cuh"
#include "internal.h"

namespace cg = cooperative_groups;

namespace oilbird {

constexpr int kEvictThreads = 512;

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

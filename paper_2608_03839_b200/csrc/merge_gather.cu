// K4/K5: final top-k merge, firing rule, copy depth and continuation gather.
//
// Eq. 2: E_t = arg top-k s_i, with theta a firing condition on the best neighbour
// only.  Eq. 3: each neighbour copies D(s_i) tokens (or a fixed span) starting
// `offset` rows after itself, read out of the trace that holds it.  Algorithm 1
// iterates the neighbours by decreasing s_i; the output keeps that order.
//
// One CTA per query.  The scan leaves one descending candidate list per CTA; 32 warps
// fold them with register-resident bitonic merges (a few microseconds even for hundreds
// of lists); the integer gather that follows is trivial (nq*k*L tokens).
#include "common.cuh"
#include "gather.cuh"
#include "internal.h"

namespace oilbird {

__global__ void __launch_bounds__(kMergeThreads)
merge_gather_kernel(PoolView pv, const u64* __restrict__ partial, int n_lists, int nq, int kk,
                    const int32_t* __restrict__ q_valid, GatherParams gp, oilbird_query_out out) {
  __shared__ u64 scratch[kMergeWarps * OILBIRD_MAX_K];
  __shared__ u64 s_best[OILBIRD_MAX_K];
  __shared__ int32_t s_idx[OILBIRD_MAX_K];
  __shared__ float s_score[OILBIRD_MAX_K];
  __shared__ int32_t s_len[OILBIRD_MAX_K];
  const int q = blockIdx.x;
  const int k = gp.k;
  pdl_enter();   // the scan's candidate lists
  const int valid = q_valid[q];       // consumed after the merge: the load overlaps it
  if (kk == 32) merge_lists<1>(partial, n_lists, nq, q, k, scratch, s_best);
  else if (kk == 64) merge_lists<2>(partial, n_lists, nq, q, k, scratch, s_best);
  else merge_lists<4>(partial, n_lists, nq, q, k, scratch, s_best);
  for (int j = threadIdx.x; j < k; j += kMergeThreads) {
    const u64 key = valid ? s_best[j] : 0;            // NaN/Inf query: no neighbours
    const int idx = key ? candidate_row(key) : -1;
    const float s = key ? candidate_score(key) : -INFINITY;
    s_idx[j] = idx;
    s_score[j] = s;
    out.idx[(size_t)q * k + j] = idx;
    out.score[(size_t)q * k + j] = s;
  }
  __syncthreads();
  fire_depth_copy(pv, gp, q, s_idx, s_score, out, s_len);
}

__global__ void __launch_bounds__(128)
gather_only_kernel(PoolView pv, const int32_t* __restrict__ idx, const float* __restrict__ score,
                   GatherParams gp, oilbird_query_out out) {
  __shared__ int32_t s_idx[OILBIRD_MAX_K];
  __shared__ float s_score[OILBIRD_MAX_K];
  __shared__ int32_t s_len[OILBIRD_MAX_K];
  const int q = blockIdx.x, k = gp.k;
  pdl_enter();
  for (int j = threadIdx.x; j < k; j += blockDim.x) {
    s_idx[j] = idx[(size_t)q * k + j];
    s_score[j] = score[(size_t)q * k + j];
  }
  __syncthreads();
  fire_depth_copy(pv, gp, q, s_idx, s_score, out, s_len);
}

cudaError_t launch_merge_gather(const PoolView& pv, const u64* partial, int32_t n_lists,
                                int32_t nq, int32_t kk, const int32_t* q_valid,
                                const GatherParams& gp, const oilbird_query_out& out,
                                cudaStream_t st) {
  return launch_pdl(merge_gather_kernel, dim3(nq), dim3(kMergeThreads), 0, st, pv, partial, n_lists,
                    nq, kk, q_valid, gp, out);
}

cudaError_t launch_gather_only(const PoolView& pv, const int32_t* idx, const float* score,
                               int32_t nq, const GatherParams& gp, const oilbird_query_out& out,
                               cudaStream_t st) {
  return launch_pdl(gather_only_kernel, dim3(nq), dim3(128), 0, st, pv, idx, score, gp, out);
}

cudaError_t preload_merge_kernels() {
  cudaError_t e = preload_kernel(merge_gather_kernel);
  return e != cudaSuccess ? e : preload_kernel(gather_only_kernel);
}

}  // namespace oilbird

// a4..a6 of the path for one query whose neighbours are known: firing rule (Eq. 2), copy
// depth (Eq. 3; fixed spans in the batch probe) and the continuation gather (Eq. 3), shared
// by the kernels that end a lookup.
#pragma once
#include "common.cuh"
#include "internal.h"

namespace oilbird {

// Eq. 3's D(s): first tier, in the order given, whose floor the score reaches.  By rank (the
// granularity ablation's arm, Section 6): neighbour j copies tier_depth[j], the last entry
// from there on, whatever its score.
__device__ __forceinline__ int depth_of(float s, int j, const GatherParams& gp) {
  if (gp.depth_mode == OILBIRD_DEPTH_FIXED) return gp.cont_len;
  if (gp.depth_mode == OILBIRD_DEPTH_RANKED)
    return gp.n_tiers > 0 ? gp.tier_depth[j < gp.n_tiers ? j : gp.n_tiers - 1] : 0;
  for (int t = 0; t < gp.n_tiers; ++t)
    if (s >= gp.tier_thr[t]) return gp.tier_depth[t];
  return 0;
}

// a4..a6 for one query whose neighbours (best first) are in shared memory.
__device__ __forceinline__ void fire_depth_copy(const PoolView& pv, const GatherParams& gp, int q,
                                const int32_t* s_idx, const float* s_score,
                                const oilbird_query_out& out, int32_t* s_len) {
  const int k = gp.k, L = gp.cont_len;
  // a4: theta gates on the best neighbour only (Eq. 2)
  const bool fired = s_idx[0] >= 0 && s_score[0] >= gp.theta;
  if (threadIdx.x == 0) out.fired[q] = fired ? 1 : 0;
  for (int j = threadIdx.x; j < k; j += blockDim.x) {
    const int idx = s_idx[j];
    int len = 0;
    if (fired && idx >= 0 && idx < pv.n_rows) {
      const int dep = depth_of(s_score[j], j, gp);                    // a5
      const long long start = (long long)idx + gp.offset;
      const long long end = pv.trace_end[pv.trace_id[idx]];           // never leave the trace
      long long m = end - start;
      if (m > dep) m = dep;
      if (m > L) m = L;
      if (m < 0) m = 0;
      len = (int)m;
    }
    s_len[j] = len;
    out.cont_len[(size_t)q * k + j] = len;
  }
  // a6: gamma = x_{idx+offset : idx+offset+len}, padded with -1.  The tokens are fetched
  // before the lengths are known (any row below n_rows may be read) so that this load does
  // not queue behind the trace lookups above; the length then masks them.
  int32_t* dst = out.cont_tok + (size_t)q * k * L;
  constexpr int kSpec = 4;
  const int n_out = k * L;
  int32_t v[kSpec];
#pragma unroll
  for (int u = 0; u < kSpec; ++u) {
    const int e = threadIdx.x + u * blockDim.x;
    v[u] = -1;
    if (e < n_out) {
      const int j = e / L, t = e - j * L;
      const long long row = (long long)s_idx[j] + gp.offset + t;
      if (fired && s_idx[j] >= 0 && row < pv.n_rows) v[u] = pv.tok[row];
    }
  }
  __syncthreads();                               // s_len is complete
#pragma unroll
  for (int u = 0; u < kSpec; ++u) {
    const int e = threadIdx.x + u * blockDim.x;
    if (e < n_out) {
      const int j = e / L, t = e - j * L;
      dst[e] = t < s_len[j] ? v[u] : -1;
    }
  }
  for (int e = threadIdx.x + kSpec * blockDim.x; e < n_out; e += blockDim.x) {
    const int j = e / L, t = e - j * L;
    dst[e] = t < s_len[j] ? pv.tok[(size_t)s_idx[j] + gp.offset + t] : -1;
  }
}

}  // namespace oilbird

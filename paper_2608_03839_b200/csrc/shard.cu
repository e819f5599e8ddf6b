// Row sharding of one logical pool over several GPUs.
//
// The retrieval of the paper scores every stored row, and rows are independent: a pool too
// large (or too hot) for one GPU is split by whole traces, each GPU answers the query on
// its rows, and the per-shard answers are merged.  The result must be what a single pool
// holding all rows in their global order would return (Eq. 2 with the lowest-position tie
// rule; the theta test of Algorithm 1 on the global best).  Each shard therefore
//   1. runs its local query without the theta gate (depths and continuations for every
//      neighbour),
//   2. maps local rows to the caller-assigned global positions (to_global_kernel),
//   3. exchanges its nq*k records with the other shards (one all-gather, done by the
//      caller's communication library), and
//   4. merges the gathered records (merge_shards_kernel): global top-k by (score desc,
//      global position asc), then the firing rule on the merged best.
// Continuations travel with their neighbour, so no token stream is replicated.
#include <math.h>

#include "common.cuh"
#include "internal.h"

namespace oilbird {

__global__ void __launch_bounds__(256)
to_global_kernel(const int32_t* __restrict__ idx, int64_t* __restrict__ out, int64_t n,
                 const int32_t* __restrict__ trace_id, const int32_t* __restrict__ trace_end,
                 const int64_t* __restrict__ trace_gbase, int32_t n_rows) {
  pdl_enter();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int32_t r = idx[i];
  int64_t g = -1;
  if (r >= 0 && r < n_rows) {
    const int32_t t = trace_id[r];
    const int32_t start = t > 0 ? trace_end[t - 1] : 0;     // local traces are contiguous
    g = trace_gbase[t] + (r - start);
  }
  out[i] = g;
}

constexpr int kShardThreads = 1024;

// One CTA per query.  Candidate c = (shard, j); its rank among all candidates is counted
// directly (at most 8 x 128 candidates: a million compares), which keeps the 64-bit
// positions exact.
__global__ void __launch_bounds__(kShardThreads)
merge_shards_kernel(int n_shards, int nq, int k, int L, float theta,
                    const unsigned char* __restrict__ gathered, size_t shard_stride,
                    size_t off_gidx, size_t off_score, size_t off_len, size_t off_tok,
                    int64_t* __restrict__ out_gidx, float* __restrict__ out_score,
                    int32_t* __restrict__ out_fired, int32_t* __restrict__ out_len,
                    int32_t* __restrict__ out_tok) {
  __shared__ float s_score[kShardThreads];
  __shared__ long long s_gidx[kShardThreads];
  __shared__ int s_src[OILBIRD_MAX_K];     // winning candidate of each output rank
  __shared__ int s_fired;
  const int q = blockIdx.x;
  pdl_enter();
  const int n_cand = n_shards * k;         // <= kShardThreads (checked by the host)
  const int c = threadIdx.x;
  float my_s = -INFINITY;
  long long my_g = -1;
  if (c < n_cand) {
    const int s = c / k, j = c - s * k;
    const unsigned char* base = gathered + (size_t)s * shard_stride;
    my_g = reinterpret_cast<const long long*>(base + off_gidx)[(size_t)q * k + j];
    my_s = reinterpret_cast<const float*>(base + off_score)[(size_t)q * k + j];
    if (my_g < 0) my_s = -INFINITY;
  }
  s_score[c] = my_s;
  s_gidx[c] = my_g;
  for (int j = threadIdx.x; j < k; j += kShardThreads) s_src[j] = -1;
  __syncthreads();
  if (c < n_cand && my_g >= 0) {
    int rank = 0;
    for (int o = 0; o < n_cand; ++o) {
      const float os = s_score[o];
      const long long og = s_gidx[o];
      rank += (og >= 0) && (os > my_s || (os == my_s && og < my_g));   // Eq. 2 + tie rule
    }
    if (rank < k) s_src[rank] = c;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int b = s_src[0];
    s_fired = (b >= 0 && s_score[b] >= theta) ? 1 : 0;     // theta on the merged best only
    out_fired[q] = s_fired;
  }
  __syncthreads();
  const bool fired = s_fired != 0;
  for (int j = threadIdx.x; j < k; j += kShardThreads) {
    const int b = s_src[j];
    out_gidx[(size_t)q * k + j] = b >= 0 ? s_gidx[b] : -1;
    out_score[(size_t)q * k + j] = b >= 0 ? s_score[b] : -INFINITY;
    int len = 0;
    if (b >= 0 && fired) {
      const int s = b / k, jj = b - s * k;
      len = reinterpret_cast<const int32_t*>(gathered + (size_t)s * shard_stride + off_len)
          [(size_t)q * k + jj];
    }
    out_len[(size_t)q * k + j] = len;
  }
  for (int e = threadIdx.x; e < k * L; e += kShardThreads) {
    const int j = e / L, t = e - j * L;
    const int b = s_src[j];
    int tok = -1;
    if (b >= 0 && fired) {
      const int s = b / k, jj = b - s * k;
      const unsigned char* base = gathered + (size_t)s * shard_stride;
      const int len = reinterpret_cast<const int32_t*>(base + off_len)[(size_t)q * k + jj];
      if (t < len) tok = reinterpret_cast<const int32_t*>(base + off_tok)[((size_t)q * k + jj) * L + t];
    }
    out_tok[(size_t)q * k * L + e] = tok;
  }
}

cudaError_t launch_to_global(const int32_t* idx, int64_t* out, int64_t n, const int32_t* trace_id,
                             const int32_t* trace_end, const int64_t* trace_gbase, int32_t n_rows,
                             cudaStream_t st) {
  const unsigned grid = (unsigned)((n + 255) / 256);
  return launch_pdl(to_global_kernel, dim3(grid), dim3(256), 0, st, idx, out, n, trace_id,
                    trace_end, trace_gbase, n_rows);
}

cudaError_t preload_shard_kernels() {
  cudaError_t e = preload_kernel(to_global_kernel);
  return e != cudaSuccess ? e : preload_kernel(merge_shards_kernel);
}

}  // namespace oilbird

using namespace oilbird;

extern "C" int oilbird_merge_shards(int32_t n_shards, int32_t nq, int32_t k, int32_t L, float theta,
                                    const void* gathered, size_t shard_stride, size_t off_gidx,
                                    size_t off_score, size_t off_len, size_t off_tok,
                                    int64_t* out_gidx, float* out_score, int32_t* out_fired,
                                    int32_t* out_len, int32_t* out_tok, int32_t device,
                                    void* cuda_stream) {
  if (n_shards < 1 || nq < 1 || k < 1 || k > OILBIRD_MAX_K || L < 1 || L > OILBIRD_MAX_CONT_LEN ||
      (int64_t)n_shards * k > kShardThreads || !gathered || !out_gidx || !out_score || !out_fired ||
      !out_len || !out_tok || theta != theta || (off_gidx % 8) || (shard_stride % 8))
    return OILBIRD_EINVAL;
  if (cudaSetDevice(device) != cudaSuccess) return OILBIRD_ECUDA;
  if (preload_all_kernels() != cudaSuccess) return OILBIRD_ECUDA;
  cudaError_t e = launch_pdl(merge_shards_kernel, dim3(nq), dim3(kShardThreads), 0,
                             (cudaStream_t)cuda_stream, n_shards, nq, k, L, theta,
                             (const unsigned char*)gathered, shard_stride, off_gidx, off_score,
                             off_len, off_tok, out_gidx, out_score, out_fired, out_len, out_tok);
  return e == cudaSuccess ? OILBIRD_OK : OILBIRD_ECUDA;
}

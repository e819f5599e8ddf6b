// Chain post-filter and tree merge (paper Algorithm 1, chain collection and merge lines;
// Section 4 "(iii) Merge"; Eq. 4).
//
// Candidate chains are taken in order (semantic chains by decreasing similarity, then the
// caller's other chains); a semantic chain shorter than min_len and any chain equal to one
// already collected is dropped; the rest re-walk the draft tree from the root: while the
// next token is carried by a child of the current node that child is walked for free,
// otherwise a node is bought, until the retrieval budget is spent.  A chain therefore costs
// its length minus its longest prefix already present as a root path (Eq. 4).
//
// The problem is tiny (at most 64 nodes, a few hundred tokens) and sequential per request,
// so one warp handles one request: the tree lives in shared memory, the child search is one
// ballot over the nodes, chains are staged in shared memory before they are walked.
// Requests of a batch run in parallel (four per CTA).
#include <stdio.h>

#include "common.cuh"
#include "internal.h"

namespace oilbird {

constexpr int kMergeTreeWarps = 4;
constexpr int kMaxNodes = OILBIRD_TREE_MAX_NODES;   // 64: the ancestor mask is one u64

enum { kChainShort = 0, kChainDuplicate = 1, kChainMerged = 2, kChainCut = 3, kChainNotReached = 4 };

struct ChainRef { const int32_t* tok; int len; };

__device__ __forceinline__ ChainRef chain_of(int c, int q, const int32_t* sem_tok,
                                             const int32_t* sem_len, int k, int L,
                                             const int32_t* ex_tok, const int32_t* ex_len, int ne,
                                             int Le) {
  ChainRef r;
  if (c < k) {
    r.tok = sem_tok + ((size_t)q * k + c) * L;
    r.len = sem_len[(size_t)q * k + c];
    r.len = r.len < 0 ? 0 : (r.len > L ? L : r.len);
  } else {
    r.tok = ex_tok + ((size_t)q * ne + (c - k)) * Le;
    r.len = ex_len[(size_t)q * ne + (c - k)];
    r.len = r.len < 0 ? 0 : (r.len > Le ? Le : r.len);
  }
  return r;
}

__global__ void __launch_bounds__(kMergeTreeWarps * 32)
merge_tree_kernel(int nq, const int32_t* __restrict__ sem_tok, const int32_t* __restrict__ sem_len,
                  int k, int L, const int32_t* __restrict__ ex_tok,
                  const int32_t* __restrict__ ex_len, int ne, int Le, int32_t* tree_tok,
                  int32_t* tree_parent, int32_t* n_nodes, int32_t* depth, uint64_t* mask,
                  int32_t* status, int32_t* bought, int32_t* walked, oilbird_merge_params mp) {
  __shared__ int32_t s_tok[kMergeTreeWarps][kMaxNodes];
  __shared__ int32_t s_par[kMergeTreeWarps][kMaxNodes];
  __shared__ int32_t s_chain[kMergeTreeWarps][OILBIRD_MAX_CONT_LEN];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.x * kMergeTreeWarps + warp;
  pdl_enter();
  if (q >= nq) return;
  int32_t* tok = s_tok[warp];
  int32_t* par = s_par[warp];
  int32_t* chain = s_chain[warp];
  const int max_nodes = mp.max_nodes;
  int n = n_nodes[q];
  n = n < 1 ? 1 : (n > max_nodes ? max_nodes : n);
  for (int j = lane; j < kMaxNodes; j += 32) {
    tok[j] = j < n ? tree_tok[(size_t)q * max_nodes + j] : -1;
    // parents come from caller memory and index shared memory below: one that is not
    // another node of the tree detaches its node (parent -1) instead of being followed
    int p = (j >= 1 && j < n) ? tree_parent[(size_t)q * max_nodes + j] : -1;
    par[j] = (p >= 0 && p < n && p != j) ? p : -1;
  }
  __syncwarp();
  int left = mp.budget;
  const int n_chains = k + ne;
  for (int c = 0; c < n_chains; ++c) {
    const ChainRef g = chain_of(c, q, sem_tok, sem_len, k, L, ex_tok, ex_len, ne, Le);
    int st, n_bought = 0, n_walked = 0;
    if (g.len == 0 || (c < k && g.len < mp.min_len)) {
      st = kChainShort;
    } else {
      for (int t = lane; t < g.len; t += 32) chain[t] = g.tok[t];
      __syncwarp();
      // equal to a chain collected earlier?
      bool dup = false;
      for (int e = 0; e < c && !dup; ++e) {
        const int se = status[(size_t)q * n_chains + e];      // written by this warp below
        if (se == kChainShort || se == kChainDuplicate) continue;
        const ChainRef h = chain_of(e, q, sem_tok, sem_len, k, L, ex_tok, ex_len, ne, Le);
        if (h.len != g.len) continue;
        bool same = true;
        for (int t = lane; t < g.len; t += 32) same &= (h.tok[t] == chain[t]);
        dup = __all_sync(0xffffffffu, same);
      }
      if (dup) {
        st = kChainDuplicate;
      } else if (left == 0 || n >= max_nodes) {
        st = kChainNotReached;
      } else {
        int node = 0;
        bool cut = false, walking = mp.root_attached == 0;
        for (int t = 0; t < g.len; ++t) {
          const int want = chain[t];
          int nxt = -1;
          if (walking) {
            // child of `node` carrying `want`: lowest node number wins
            const unsigned lo = __ballot_sync(0xffffffffu, lane >= 1 && lane < n &&
                                                               par[lane] == node && tok[lane] == want);
            const unsigned hi = __ballot_sync(0xffffffffu, lane + 32 < n && par[lane + 32] == node &&
                                                               tok[lane + 32] == want);
            nxt = lo ? __ffs(lo) - 1 : (hi ? 32 + __ffs(hi) - 1 : -1);
          }
          if (nxt >= 0) {
            ++n_walked;
          } else {
            if (left == 0 || n >= max_nodes) { cut = true; break; }
            if (lane == 0) { tok[n] = want; par[n] = node; }
            __syncwarp();
            nxt = n;
            ++n; --left; ++n_bought;
          }
          node = nxt;
        }
        st = cut ? kChainCut : kChainMerged;
      }
      __syncwarp();
    }
    if (lane == 0) {
      status[(size_t)q * n_chains + c] = st;
      bought[(size_t)q * n_chains + c] = n_bought;
      walked[(size_t)q * n_chains + c] = n_walked;
    }
    __syncwarp();
  }
  // a node attends to itself and its ancestors
  for (int j = lane; j < max_nodes; j += 32) {
    unsigned long long m = 0;
    int dpt = 0;
    if (j < n) {
      int a = j;
      for (int hop = 0; a >= 0 && hop < kMaxNodes; ++hop) { m |= 1ull << a; a = par[a]; ++dpt; }
    }
    tree_tok[(size_t)q * max_nodes + j] = j < n ? tok[j] : -1;
    tree_parent[(size_t)q * max_nodes + j] = j < n ? par[j] : -1;
    depth[(size_t)q * max_nodes + j] = j < n ? dpt - 1 : 0;
    mask[(size_t)q * max_nodes + j] = m;
  }
  if (lane == 0) n_nodes[q] = n;
}

cudaError_t preload_merge_tree_kernels() { return preload_kernel(merge_tree_kernel); }

}  // namespace oilbird

using namespace oilbird;

extern "C" {

void oilbird_merge_params_default(oilbird_merge_params* p) {
  if (!p) return;
  p->budget = 16;         // Algorithm 1: B_ret = 16 ...
  p->max_nodes = 60;      // ... of 60 nodes
  p->min_len = 2;         // a chain needs at least two tokens
  p->root_attached = 0;
}

int oilbird_merge_chains(int32_t nq, const int32_t* sem_tok, const int32_t* sem_len, int32_t k,
                         int32_t L, const int32_t* extra_tok, const int32_t* extra_len, int32_t ne,
                         int32_t Le, int32_t* tree_tok, int32_t* tree_parent, int32_t* n_nodes,
                         int32_t* depth, uint64_t* mask, int32_t* status, int32_t* bought,
                         int32_t* walked, const oilbird_merge_params* mp, int32_t device,
                         void* cuda_stream) {
  if (!mp || nq < 1 || k < 0 || ne < 0 || k + ne < 1 || !tree_tok || !tree_parent || !n_nodes ||
      !depth || !mask || !status || !bought || !walked)
    return OILBIRD_EINVAL;
  if ((k > 0 && (!sem_tok || !sem_len || L < 1 || L > OILBIRD_MAX_CONT_LEN)) ||
      (ne > 0 && (!extra_tok || !extra_len || Le < 1 || Le > OILBIRD_MAX_CONT_LEN)))
    return OILBIRD_EINVAL;
  if (mp->max_nodes < 1 || mp->max_nodes > OILBIRD_TREE_MAX_NODES || mp->budget < 0 ||
      mp->min_len < 0)
    return OILBIRD_EINVAL;
  if (cudaSetDevice(device) != cudaSuccess) return OILBIRD_ECUDA;
  if (preload_all_kernels() != cudaSuccess) return OILBIRD_ECUDA;
  const int grid = (nq + kMergeTreeWarps - 1) / kMergeTreeWarps;
  cudaError_t e = launch_pdl(merge_tree_kernel, dim3(grid), dim3(kMergeTreeWarps * 32), 0,
                             (cudaStream_t)cuda_stream, nq, sem_tok, sem_len, k, L, extra_tok,
                             extra_len, ne, Le, tree_tok, tree_parent, n_nodes, depth, mask, status,
                             bought, walked, *mp);
  return e == cudaSuccess ? OILBIRD_OK : OILBIRD_ECUDA;
}

}  // extern "C"

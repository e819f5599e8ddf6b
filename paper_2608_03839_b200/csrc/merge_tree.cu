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
// The problem is tiny (at most 64 nodes, a few hundred tokens) and the chains of a request
// depend on one another through the tree, so one warp handles one request and the kernel is
// bound by latency, not by bandwidth.  What it does about that:
//   - every load that needs no other load's result is issued at once (node count, tree,
//     chain lengths; then all chains' tokens, sixteen loads in flight per lane);
//   - which chains are short or repeat an earlier one is settled for all chains in parallel,
//     one chain per lane, before the tree is touched;
//   - the free walk of a chain is not taken token by token: the node that ends it is found
//     for all nodes at once by pointer jumping over the parent array (six rounds for 64
//     nodes), and so are the depths and the ancestor masks written at the end;
//   - only the bought nodes, at most the budget per request, are added one by one.
// Measured on 64 requests of 15 chains (8 of up to 48 tokens) into a 44-node tree: 57 us for
// the token-by-token form that read its chains from global memory, 14.6 us for this one
// (one request: 33 us -> 14 us; device time of single launches with cold caches).
// Requests of a batch run in parallel (four per CTA).
#include <stdio.h>

#include "common.cuh"
#include "internal.h"

namespace oilbird {

constexpr int kMergeTreeWarps = 4;
constexpr int kMaxNodes = OILBIRD_TREE_MAX_NODES;   // 64: the ancestor mask is one u64
// A request's chains are copied into shared memory once, when they fit: chain c at
// c * stride tokens.  Larger requests read their chains from global memory, chain by chain.
constexpr int kStageTokens = 2048;                  // per request (8 KB)
constexpr int kStageChains = 64;

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

// Pointer jumping over the parent forest of one request, two nodes per lane (lane, lane + 32):
// six rounds of  v[j] = op(v[j], v[anc[j]]); anc[j] = anc[anc[j]]  reach every ancestor of a
// node at depth <= 63.  A root (or a detached node) is its own ancestor and must hold op's
// neutral value.  s_anc / s_v: 64 entries of shared memory of this warp.
template <class T, class Op>
__device__ __forceinline__ void jump_to_root(int& anc0, int& anc1, T& v0, T& v1, int* s_anc, T* s_v,
                                             int lane, Op op) {
#pragma unroll
  for (int r = 0; r < 6; ++r) {
    s_anc[lane] = anc0; s_anc[lane + 32] = anc1;
    s_v[lane] = v0; s_v[lane + 32] = v1;
    __syncwarp();
    const T p0 = s_v[anc0], p1 = s_v[anc1];
    const int a0 = s_anc[anc0], a1 = s_anc[anc1];
    __syncwarp();
    v0 = op(v0, p0); v1 = op(v1, p1);
    anc0 = a0; anc1 = a1;
  }
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
  __shared__ int32_t s_all[kMergeTreeWarps][kStageTokens];
  __shared__ int16_t s_clen[kMergeTreeWarps][kStageChains];
  __shared__ int8_t s_cst[kMergeTreeWarps][kStageChains];
  __shared__ uint32_t s_hash[kMergeTreeWarps][kStageChains];
  __shared__ int s_anc[kMergeTreeWarps][kMaxNodes];
  __shared__ int s_vi[kMergeTreeWarps][kMaxNodes];
  __shared__ unsigned long long s_vm[kMergeTreeWarps][kMaxNodes];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.x * kMergeTreeWarps + warp;
  pdl_enter();
  if (q >= nq) return;
  int32_t* tok = s_tok[warp];
  int32_t* par = s_par[warp];
  const int32_t* chain = s_chain[warp];
  int32_t* chain_w = s_chain[warp];
  const int max_nodes = mp.max_nodes;
  const int n_chains = k + ne;
  const int stride = (L > Le ? L : Le) | 1;      // odd: chains read one per lane hit distinct banks
  const bool staged = n_chains <= kStageChains && n_chains * stride <= kStageTokens;
  // everything that does not depend on another load is asked for at once: the node count,
  // the tree's two arrays and the chain lengths (one round trip instead of three)
  int n = n_nodes[q];
  int ld_tok[2], ld_par[2], ld_len[2] = {0, 0};
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int j = lane + 32 * h;
    ld_tok[h] = j < max_nodes ? tree_tok[(size_t)q * max_nodes + j] : -1;
    ld_par[h] = (j >= 1 && j < max_nodes) ? tree_parent[(size_t)q * max_nodes + j] : -1;
    if (staged && j < n_chains)
      ld_len[h] = chain_of(j, q, sem_tok, sem_len, k, L, ex_tok, ex_len, ne, Le).len;
  }
  n = n < 1 ? 1 : (n > max_nodes ? max_nodes : n);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int j = lane + 32 * h;
    tok[j] = j < n ? ld_tok[h] : -1;
    // parents come from caller memory and index shared memory below: one that is not
    // another node of the tree detaches its node (parent -1) instead of being followed
    const int p = ld_par[h];
    par[j] = (j < n && p >= 0 && p < n && p != j) ? p : -1;
    if (staged && j < n_chains) s_clen[warp][j] = (int16_t)ld_len[h];
  }
  __syncwarp();
  if (staged) {
    // all chains' tokens next, sixteen loads in flight per lane
    for (int g = 0; g * 32 < stride; ++g) {
      const int t = g * 32 + lane;
      for (int c0 = 0; c0 < n_chains; c0 += 16) {
        int v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int c = c0 + u;
          const bool on = c < n_chains && t < s_clen[warp][c < n_chains ? c : 0];
          const int32_t* src = c < k ? sem_tok + ((size_t)q * k + c) * L : ex_tok + ((size_t)q * ne + (c - k)) * Le;
          v[u] = on ? __ldg(src + t) : 0;
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int c = c0 + u;
          if (c < n_chains && t < s_clen[warp][c]) s_all[warp][c * stride + t] = v[u];
        }
      }
    }
  }
  // the tree, two nodes per lane, is kept in registers; shared memory follows along
  int par0 = par[lane], tok0 = tok[lane], par1 = par[lane + 32], tok1 = tok[lane + 32];
  // depth of every node (edges to the root, or to the top of a detached piece)
  int dep0 = par0 >= 0 ? 1 : 0, dep1 = par1 >= 0 ? 1 : 0;
  {
    int a0 = par0 >= 0 ? par0 : lane, a1 = par1 >= 0 ? par1 : lane + 32;
    jump_to_root(a0, a1, dep0, dep1, s_anc[warp], s_vi[warp], lane, [](int a, int b) { return a + b; });
  }
  // a node with a lower-numbered sibling that carries the same token is never walked (the
  // lowest child wins): such nodes are left out of the prefix search below
  bool val0 = lane >= 1 && lane < n, val1 = lane + 32 < n;
  for (int i = 1; i < n; ++i) {
    const int pi = par[i], ti = tok[i];
    if (i < lane && pi == par0 && ti == tok0) val0 = false;
    if (i < lane + 32 && pi == par1 && ti == tok1) val1 = false;
  }
  int left = mp.budget;
  if (staged) {
    __syncwarp();
    // Which chains are too short, and which repeat an earlier chain that is not, does not
    // depend on the tree: settled here for all chains at once, one chain per lane (a hash
    // picks the candidates, a token-by-token comparison decides).
    for (int c = lane; c < n_chains; c += 32) {
      const int len = s_clen[warp][c];
      uint32_t h = 2166136261u;
      for (int t = 0; t < len; ++t) h = (h ^ (uint32_t)s_all[warp][c * stride + t]) * 16777619u;
      s_hash[warp][c] = h;
    }
    __syncwarp();
    for (int c = lane; c < n_chains; c += 32) {
      const int len = s_clen[warp][c];
      const uint32_t h = s_hash[warp][c];
      int pre = (len == 0 || (c < k && len < mp.min_len)) ? kChainShort : -1;
      for (int e = 0; e < c && pre < 0; ++e) {
        if (s_clen[warp][e] != len || s_hash[warp][e] != h || (e < k && len < mp.min_len)) continue;
        bool same = true;
        for (int t = 0; t < len && same; ++t) same = s_all[warp][e * stride + t] == s_all[warp][c * stride + t];
        if (same) pre = kChainDuplicate;
      }
      s_cst[warp][c] = (int8_t)pre;
    }
    __syncwarp();
  }
  for (int c = 0; c < n_chains; ++c) {
    ChainRef g;
    if (staged) { g.tok = nullptr; g.len = s_clen[warp][c]; }
    else g = chain_of(c, q, sem_tok, sem_len, k, L, ex_tok, ex_len, ne, Le);
    if (staged) chain = s_all[warp] + c * stride;
    int st, n_bought = 0, n_walked = 0;
    const int pre = staged ? s_cst[warp][c] : -1;
    if (staged ? pre == kChainShort : (g.len == 0 || (c < k && g.len < mp.min_len))) {
      st = kChainShort;
    } else {
      if (!staged) {
        for (int t = lane; t < g.len; t += 32) chain_w[t] = g.tok[t];
        __syncwarp();
        chain = chain_w;
      }
      // equal to a chain collected earlier?
      bool dup = staged && pre == kChainDuplicate;
      for (int e = 0; !staged && e < c && !dup; ++e) {
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
        int node = 0, node_dep = 0;
        bool cut = false;
        if (mp.root_attached == 0) {
          // pi(chain, T), the longest prefix of the chain that is a root path, for all nodes
          // at once: node j lies on it iff j and every ancestor of j carry the chain's token
          // at their depth; the deepest such node ends the walk.  (Walking token by token,
          // a ballot over the nodes per token, cost ~100 cycles per token of a single warp.)
          int ok0 = (val0 && lane < n && dep0 >= 1 && dep0 <= g.len && tok0 == chain[dep0 - 1]) ? 1 : 0;
          int ok1 = (val1 && lane + 32 < n && dep1 >= 1 && dep1 <= g.len && tok1 == chain[dep1 - 1]) ? 1 : 0;
          if (lane == 0) ok0 = 1;                                    // the root
          int a0 = (lane >= 1 && lane < n && par0 >= 0) ? par0 : lane;
          int a1 = (lane + 32 < n && par1 >= 0) ? par1 : lane + 32;
          jump_to_root(a0, a1, ok0, ok1, s_anc[warp], s_vi[warp], lane, [](int a, int b) { return a & b; });
          // (a node that does not hang from the root ends at itself or in a cycle, not at 0)
          const unsigned k0 = (ok0 && a0 == 0 && lane >= 1) ? ((unsigned)dep0 << 8 | (unsigned)lane) : 0u;
          const unsigned k1 = (ok1 && a1 == 0) ? ((unsigned)dep1 << 8 | (unsigned)(lane + 32)) : 0u;
          const unsigned best = __reduce_max_sync(0xffffffffu, k0 > k1 ? k0 : k1);
          node = (int)(best & 255u);
          node_dep = (int)(best >> 8);
          n_walked = node_dep;
        }
        // from here on every token is bought: a bought node has no children to walk
        for (int t = n_walked; t < g.len; ++t) {
          if (left == 0 || n >= max_nodes) { cut = true; break; }
          const int want = chain[t];
          if (lane == 0) { tok[n] = want; par[n] = node; }
          if (lane == (n & 31)) {
            if (n < 32) { tok0 = want; par0 = node; dep0 = node_dep + 1; val0 = true; }
            else { tok1 = want; par1 = node; dep1 = node_dep + 1; val1 = true; }
          }
          node = n;
          ++node_dep;
          ++n; --left; ++n_bought;
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
  __syncwarp();
  unsigned long long m0 = lane < n ? 1ull << lane : 0ull, m1 = lane + 32 < n ? 1ull << (lane + 32) : 0ull;
  {
    int a0 = (lane < n && par0 >= 0) ? par0 : lane, a1 = (lane + 32 < n && par1 >= 0) ? par1 : lane + 32;
    jump_to_root(a0, a1, m0, m1, s_anc[warp], s_vm[warp], lane,
                 [](unsigned long long a, unsigned long long b) { return a | b; });
  }
  for (int h = 0; h < 2; ++h) {
    const int j = lane + 32 * h;
    if (j < max_nodes) {
      tree_tok[(size_t)q * max_nodes + j] = j < n ? tok[j] : -1;
      tree_parent[(size_t)q * max_nodes + j] = j < n ? par[j] : -1;
      depth[(size_t)q * max_nodes + j] = j < n ? (h ? dep1 : dep0) : 0;
      mask[(size_t)q * max_nodes + j] = j < n ? (h ? m1 : m0) : 0ull;
    }
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

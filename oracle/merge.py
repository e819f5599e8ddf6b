"""CPU oracle for the chain post-filter and the tree merge (test infrastructure).

Follows Algorithm 1 of the paper: candidate chains are collected in order (semantic chains by
decreasing similarity, then the caller's other chains), a semantic chain is kept only if it
has at least two tokens, a chain equal to one already collected is dropped, and the
collected chains are merged into the draft tree from the root until the retrieval budget
B_ret is spent (Section 4 "(iii) Merge").  Re-walking from the root means: while the next
token of the chain is already carried by a child of the current node that child is walked
for free; otherwise a node is bought.  Hence Eq. 4: cost(chain, T) = len(chain) - pi(chain, T)
with pi the longest prefix of the chain that is already a root path of T.  A node attends to
itself and its ancestors only.

Plain Python loops on purpose: the trees have at most 64 nodes.

Readings where the paper is silent:
  * when the budget runs out inside a chain the chain is cut there (its bought prefix stays);
    chains after it are not reached: once nothing is left to spend (or the tree is full)
    every later chain gets status NOT_REACHED without being walked, ALSO a chain whose
    tokens are all in the tree already, which Eq. 4 would price at zero.  The tree is the
    same either way (such a chain adds no node); only its status reads "not reached"
    rather than "merged at cost 0".  The CUDA kernel does the same;
  * a chain that is a duplicate is dropped before merging, whatever its source; the
    minimum length applies to semantic chains only (the algorithm states it on that line);
  * new nodes are numbered in the order they are bought;
  * "root-attached" (the ablation arm that hangs every chain from the root as its own
    branch) buys one node per token and shares nothing.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

PAPER_TREE_NODES = 60     # Algorithm 1: B_ret = 16 of 60 nodes
PAPER_B_RET = 16
PAPER_MIN_CHAIN = 2       # Algorithm 1: |gamma| >= 2

# chain status codes
SHORT, DUPLICATE, MERGED, CUT, NOT_REACHED = 0, 1, 2, 3, 4


@dataclass
class MergeResult:
    tok: np.ndarray        # [max_nodes] int32, -1 beyond n_nodes
    parent: np.ndarray     # [max_nodes] int32, -1 for the root and beyond n_nodes
    depth: np.ndarray      # [max_nodes] int32
    mask: np.ndarray       # [max_nodes] uint64: bit j set iff node j is the node or an ancestor
    n_nodes: int
    status: np.ndarray     # [n_chains] int32
    bought: np.ndarray     # [n_chains] int32: nodes paid for by each chain (Eq. 4)
    walked: np.ndarray     # [n_chains] int32: pi(chain, T) at the time it was merged


def prefix_in_tree(tok, parent, n_nodes, chain) -> int:
    """pi(chain, T): length of the longest prefix of chain that is a root path of T."""
    node, p = 0, 0
    for t in chain:
        nxt = -1
        for j in range(1, n_nodes):
            if parent[j] == node and tok[j] == t:
                nxt = j
                break
        if nxt < 0:
            break
        node, p = nxt, p + 1
    return p


def merge_chains(tree_tok, tree_parent, n_nodes, sem_chains, extra_chains, budget=PAPER_B_RET,
                 max_nodes=64, min_len=PAPER_MIN_CHAIN, root_attached=False) -> MergeResult:
    """One request.  tree_tok / tree_parent: the lexical tree (node 0 = root = the anchor).
    sem_chains: token lists ordered by decreasing similarity; extra_chains: the caller's
    further chains (lexical branches, recycled rollouts), merged after them."""
    tok = np.full(max_nodes, -1, np.int32)
    par = np.full(max_nodes, -1, np.int32)
    tok[:n_nodes] = np.asarray(tree_tok[:n_nodes], np.int32)
    par[:n_nodes] = np.asarray(tree_parent[:n_nodes], np.int32)
    chains = [list(map(int, c)) for c in sem_chains] + [list(map(int, c)) for c in extra_chains]
    n_sem = len(sem_chains)
    status = np.zeros(len(chains), np.int32)
    bought = np.zeros(len(chains), np.int32)
    walked = np.zeros(len(chains), np.int32)
    collected: list[list[int]] = []
    left = int(budget)
    n = int(n_nodes)
    for ci, g in enumerate(chains):
        if ci < n_sem and len(g) < min_len:
            status[ci] = SHORT
            continue
        if len(g) == 0:
            status[ci] = SHORT
            continue
        if any(g == c for c in collected):
            status[ci] = DUPLICATE
            continue
        collected.append(g)
        if left == 0 or n >= max_nodes:
            status[ci] = NOT_REACHED
            continue
        node = 0
        cut = False
        walking = not root_attached
        for t in g:
            nxt = -1
            if walking:
                for j in range(1, n):
                    if par[j] == node and tok[j] == t:
                        nxt = j
                        break
            if nxt >= 0:
                walked[ci] += 1
            else:
                walking = False if root_attached else walking
                if left == 0 or n >= max_nodes:
                    cut = True
                    break
                tok[n], par[n] = t, node
                nxt = n
                n += 1
                left -= 1
                bought[ci] += 1
            node = nxt
        status[ci] = CUT if cut else MERGED
    depth = np.zeros(max_nodes, np.int32)
    mask = np.zeros(max_nodes, np.uint64)
    for j in range(n):
        m, a, dpt = 0, j, 0
        while a >= 0:
            m |= 1 << a
            a = int(par[a])
            dpt += 1
        mask[j] = np.uint64(m)
        depth[j] = dpt - 1
    return MergeResult(tok, par, depth, mask, n, status, bought, walked)

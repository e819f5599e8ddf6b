"""Pins for the merge oracle (Algorithm 1's chain collection; Section 4 (iii); Eq. 4).  CPU only."""
import json
import os

import numpy as np

from oracle import merge as M

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def empty_tree(anchor=7):
    return [anchor], [-1], 1


def test_paper_constants():
    g = json.load(open(os.path.join(GOLD, "paper_constants.json")))
    assert M.PAPER_B_RET == g["b_ret"]["value"] == 16
    assert M.PAPER_TREE_NODES == g["tree_nodes"]["value"] == 60
    assert M.PAPER_MIN_CHAIN == g["min_chain_len"]["value"] == 2


def test_eq4_cost_is_length_minus_shared_prefix():
    # lexical tree: root(7) -> 10 -> 11 -> 12 ; root -> 20
    tok, par, n = [7, 10, 11, 12, 20], [-1, 0, 1, 2, 0], 5
    chain = [10, 11, 30, 31]                       # shares the prefix (10, 11): pi = 2
    assert M.prefix_in_tree(tok, par, n, chain) == 2
    r = M.merge_chains(tok, par, n, [chain], [], budget=16)
    assert r.bought.tolist() == [2] and r.walked.tolist() == [2]       # cost = 4 - 2
    assert r.n_nodes == 7
    assert r.tok[5:7].tolist() == [30, 31] and r.parent[5:7].tolist() == [2, 5]
    assert r.status.tolist() == [M.MERGED]
    # a chain already wholly in the tree is free
    r2 = M.merge_chains(tok, par, n, [[10, 11, 12]], [], budget=16)
    assert r2.bought.tolist() == [0] and r2.n_nodes == 5
    # a chain that diverges at the root pays for every token
    r3 = M.merge_chains(tok, par, n, [[99, 10, 11]], [], budget=16)
    assert r3.bought.tolist() == [3] and r3.walked.tolist() == [0]


def test_token_proposed_by_two_sources_is_paid_once_and_root_attached_pays_twice():
    tok, par, n = empty_tree()
    a, b = [1, 2, 3, 4], [1, 2, 3, 5, 6]
    r = M.merge_chains(tok, par, n, [a, b], [], budget=16)
    assert r.bought.tolist() == [4, 2] and r.n_nodes == 7            # (1,2,3) shared
    ra = M.merge_chains(tok, par, n, [a, b], [], budget=16, root_attached=True)
    assert ra.bought.tolist() == [4, 5] and ra.n_nodes == 10         # nothing shared
    assert ra.parent[1:5].tolist() == [0, 1, 2, 3] and ra.parent[5] == 0


def test_short_and_duplicate_chains_are_dropped_in_order():
    tok, par, n = empty_tree()
    sem = [[5], [1, 2], [1, 2], [], [1, 2, 3]]
    extra = [[9], [1, 2], [9]]                     # extra chains may be one token long
    r = M.merge_chains(tok, par, n, sem, extra, budget=16)
    assert r.status.tolist() == [M.SHORT, M.MERGED, M.DUPLICATE, M.SHORT, M.MERGED,
                                 M.MERGED, M.DUPLICATE, M.DUPLICATE]
    assert r.bought.tolist() == [0, 2, 0, 0, 1, 1, 0, 0]
    assert r.tok[: r.n_nodes].tolist() == [7, 1, 2, 3, 9]


def test_budget_cuts_the_chain_and_later_chains_are_not_reached():
    tok, par, n = empty_tree()
    r = M.merge_chains(tok, par, n, [[1, 2, 3, 4, 5], [1, 2, 8], [6, 7]], [], budget=4)
    assert r.status.tolist() == [M.CUT, M.NOT_REACHED, M.NOT_REACHED]
    assert r.bought.tolist() == [4, 0, 0] and r.n_nodes == 5
    # the paper's sizes: a 44-node lexical spine plus B_ret = 16 gives at most 60 nodes
    spine_tok = [7] + list(range(100, 143))
    spine_par = [-1] + list(range(0, 43))
    long_chain = list(range(500, 548))             # D(s) = 48 tokens, diverges at the root
    r = M.merge_chains(spine_tok, spine_par, 44, [long_chain], [], budget=M.PAPER_B_RET,
                       max_nodes=M.PAPER_TREE_NODES)
    assert r.n_nodes == 60 and r.bought.tolist() == [16] and r.status.tolist() == [M.CUT]
    # max_nodes binds before the budget does
    r = M.merge_chains(spine_tok, spine_par, 44, [long_chain], [], budget=30, max_nodes=50)
    assert r.n_nodes == 50 and r.bought.tolist() == [6]


def test_unbounded_merge_builds_the_trie_of_all_prefixes():
    rng = np.random.default_rng(0)
    for trial in range(50):
        chains = [rng.integers(0, 3, rng.integers(2, 7)).tolist() for _ in range(6)]
        tok, par, n = empty_tree()
        r = M.merge_chains(tok, par, n, chains, [], budget=1000, max_nodes=64)
        prefixes = {tuple(c[:i]) for c in chains for i in range(1, len(c) + 1)}
        assert r.n_nodes == 1 + len(prefixes)                   # the trie of all chains
        assert int(r.bought.sum()) == len(prefixes)
        # every node's root path is one of the prefixes, each exactly once
        paths = set()
        for j in range(1, r.n_nodes):
            p, a = [], j
            while a > 0:
                p.append(int(r.tok[a])); a = int(r.parent[a])
            paths.add(tuple(reversed(p)))
        assert paths == prefixes
        # Eq. 4 chain by chain, recomputed on the tree as it was before each chain
        t2, p2, n2 = list(tok), list(par), n
        seen = []
        for ci, c in enumerate(chains):
            if c in seen:
                assert r.status[ci] == M.DUPLICATE
                continue
            seen.append(c)
            part = M.merge_chains(t2, p2, n2, [c], [], budget=1000, max_nodes=64)
            assert r.bought[ci] == len(c) - M.prefix_in_tree(t2, p2, n2, c)
            t2, p2, n2 = part.tok.tolist(), part.parent.tolist(), part.n_nodes


def test_ancestor_mask_and_depth():
    tok, par, n = [7, 10, 11, 20], [-1, 0, 1, 0], 4
    r = M.merge_chains(tok, par, n, [[10, 11, 5], [20, 6]], [], budget=16)
    # nodes: 0 root, 1:10, 2:11, 3:20, 4:5 (under 2), 5:6 (under 3)
    assert r.parent[:6].tolist() == [-1, 0, 1, 0, 2, 3]
    assert r.depth[:6].tolist() == [0, 1, 2, 1, 3, 2]
    assert [int(m) for m in r.mask[:6]] == [0b1, 0b11, 0b111, 0b1001, 0b10111, 0b101001]
    for j in range(r.n_nodes):                     # a node sees itself and its ancestors only
        seen = {i for i in range(64) if (int(r.mask[j]) >> i) & 1}
        a, want = j, set()
        while a >= 0:
            want.add(a); a = int(r.parent[a])
        assert seen == want

"""GPU parity of the chain post-filter + tree merge against its CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import merge as M
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_both(trees, sems, extras, budget, max_nodes, min_len=2, root_attached=False, L=None,
             Le=None):
    """trees: list of (tok, parent); sems / extras: list (per request) of lists of chains."""
    nq = len(trees)
    k = max(len(s) for s in sems) if sems else 0
    ne = max(len(e) for e in extras) if extras else 0
    L = L or max([len(c) for s in sems for c in s] + [1])
    Le = Le or max([len(c) for e in extras for c in e] + [1])
    t_tok = np.full((nq, max_nodes), -1, np.int32)
    t_par = np.full((nq, max_nodes), -1, np.int32)
    n_nodes = np.zeros(nq, np.int32)
    s_tok = np.full((nq, max(k, 1), L), -1, np.int32)
    s_len = np.zeros((nq, max(k, 1)), np.int32)
    e_tok = np.full((nq, max(ne, 1), Le), -1, np.int32)
    e_len = np.zeros((nq, max(ne, 1)), np.int32)
    for q in range(nq):
        tok, par = trees[q]
        n_nodes[q] = len(tok)
        t_tok[q, : len(tok)], t_par[q, : len(tok)] = tok, par
        for j, c in enumerate(sems[q]):
            s_tok[q, j, : len(c)], s_len[q, j] = c, len(c)
        for j, c in enumerate(extras[q]):
            e_tok[q, j, : len(c)], e_len[q, j] = c, len(c)
    dev = lambda a: torch.from_numpy(a).cuda()
    out = B.merge_chains(dev(t_tok), dev(t_par), dev(n_nodes),
                         dev(s_tok) if k else None, dev(s_len) if k else None,
                         dev(e_tok) if ne else None, dev(e_len) if ne else None,
                         budget=budget, min_len=min_len, root_attached=root_attached)
    torch.cuda.synchronize()
    for q in range(nq):
        sem_q = [list(s_tok[q, j, : s_len[q, j]]) for j in range(k)]
        ext_q = [list(e_tok[q, j, : e_len[q, j]]) for j in range(ne)]
        ref = M.merge_chains(trees[q][0], trees[q][1], len(trees[q][0]), sem_q, ext_q,
                             budget=budget, max_nodes=max_nodes, min_len=min_len,
                             root_attached=root_attached)
        assert int(out.n_nodes[q]) == ref.n_nodes
        assert out.tree_tok[q].cpu().numpy().tolist() == ref.tok.tolist()
        assert out.tree_parent[q].cpu().numpy().tolist() == ref.parent.tolist()
        assert out.depth[q].cpu().numpy().tolist() == ref.depth.tolist()
        assert out.mask[q].cpu().numpy().view(np.uint64).tolist() == ref.mask.tolist()
        assert out.status[q].cpu().numpy().tolist() == ref.status.tolist()
        assert out.bought[q].cpu().numpy().tolist() == ref.bought.tolist()
        assert out.walked[q].cpu().numpy().tolist() == ref.walked.tolist()
    return out


def test_hand_cases():
    spine = ([7, 10, 11, 12, 20], [-1, 0, 1, 2, 0])
    run_both([spine], [[[10, 11, 30, 31], [10, 11, 12], [99, 10, 11]]], [[]], 16, 60)
    root = ([7], [-1])
    run_both([root, root], [[[1, 2, 3, 4], [1, 2, 3, 5, 6]], [[5], [1, 2], [1, 2], [], [1, 2, 3]]],
             [[], [[9], [1, 2], [9]]], 16, 60)
    run_both([root], [[[1, 2, 3, 4], [1, 2, 3, 5, 6]]], [[]], 16, 60, root_attached=True)
    run_both([root], [[[1, 2, 3, 4, 5], [1, 2, 8], [6, 7]]], [[]], 4, 60)
    # the paper's sizes: 44-node lexical spine, D(s) = 48 chain, B_ret = 16 of 60 nodes
    big = ([7] + list(range(100, 143)), [-1] + list(range(0, 43)))
    out = run_both([big], [[list(range(500, 548))]], [[]], 16, 60)
    assert int(out.n_nodes[0]) == 60
    run_both([big], [[list(range(500, 548))]], [[]], 30, 50)


@pytest.mark.parametrize("seed", range(4))
def test_random_batches(seed):
    rng = np.random.default_rng(seed)
    nq = 37
    trees, sems, extras = [], [], []
    for _ in range(nq):
        n = int(rng.integers(1, 30))
        tok = [7] + rng.integers(0, 4, n - 1).tolist()
        par = [-1] + [int(rng.integers(0, j)) for j in range(1, n)]
        trees.append((tok, par))
        sems.append([rng.integers(0, 4, rng.integers(0, 12)).tolist() for _ in range(8)])
        extras.append([rng.integers(0, 4, rng.integers(0, 7)).tolist() for _ in range(5)])
    for budget, max_nodes, ra in ((16, 60, False), (1000, 64, False), (3, 64, False),
                                   (16, 60, True), (0, 60, False)):
        run_both(trees, sems, extras, budget, max_nodes, root_attached=ra, L=12, Le=7)


def test_more_chains_than_the_kernel_stages_on_chip():
    # 70 chains per request: beyond the 64 whose tokens the kernel keeps in shared memory, so
    # it reads them from global memory chain by chain; same results either way
    rng = np.random.default_rng(11)
    trees, sems, extras = [], [], []
    for _ in range(9):
        n = int(rng.integers(1, 30))
        trees.append(([7] + rng.integers(0, 3, n - 1).tolist(),
                      [-1] + [int(rng.integers(0, j)) for j in range(1, n)]))
        sems.append([rng.integers(0, 3, rng.integers(0, 12)).tolist() for _ in range(40)])
        extras.append([rng.integers(0, 3, rng.integers(0, 7)).tolist() for _ in range(30)])
    for budget, ra in ((16, False), (1000, False), (16, True)):
        run_both(trees, sems, extras, budget, 64, root_attached=ra, L=12, Le=7)


def test_query_output_feeds_the_merge():
    """End of the retrieval path: cont_tok / cont_len of a query go straight into the merge."""
    w = W.C3.scaled(n_rows=6000, n_templates=10, d=512, nq=8, k=8, cont_len=12)
    pool = B.Pool(w.d, w.n_rows)
    for st, tk, tag in w.traces("cuda"):
        pool.append(st, tk, tag=tag)
    q, meta = w.queries("cuda")
    res = pool.query(q, B.QueryParams(k=8, theta=-2.0, depth_mode=B.DEPTH_FIXED, cont_len=12))
    nq = 8
    t_tok = torch.full((nq, 60), -1, dtype=torch.int32, device="cuda")
    t_par = torch.full((nq, 60), -1, dtype=torch.int32, device="cuda")
    t_tok[:, 0] = 7
    n_nodes = torch.ones(nq, dtype=torch.int32, device="cuda")
    out = B.merge_chains(t_tok, t_par, n_nodes, res.cont_tok, res.cont_len, budget=16)
    r = res.cpu()
    for qi in range(nq):
        sem = [r.cont_tok[qi, j, : int(r.cont_len[qi, j])].tolist() for j in range(8)]
        ref = M.merge_chains([7], [-1], 1, sem, [], budget=16, max_nodes=60)
        assert int(out.n_nodes[qi]) == ref.n_nodes
        assert out.tree_tok[qi].cpu().numpy().tolist() == ref.tok.tolist()
        assert out.bought[qi].cpu().numpy().tolist() == ref.bought.tolist()
    # neighbours of one (template, position) mostly agree: later chains buy less than the first
    b = out.bought.cpu().numpy()
    assert b[:, 0].sum() >= b[:, 1:].max(axis=1).sum()

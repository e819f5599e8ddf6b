"""Shared machinery of the GPU parity tests: feed the same arrays to the CUDA pool and
to the CPU oracle, and compare the two under the stated acceptance rule.

Acceptance rule for one query (k neighbours):
  scores   |s_gpu - s_oracle(row)| <= SCORE_TOL for every returned row (the benchmark's
           tolerance, 2e-2); additionally <= SCORE_BUG (5e-5), the bound the arithmetic
           gives: both sides multiply identical bf16 operands and differ only in fp32
           accumulation order.
  sets     where the oracle's gap between rank k and k+1 exceeds GAP (1e-3) the index
           sets are identical; at every rank whose oracle gaps to both neighbours exceed
           GAP the row is identical.  Always: every returned row scores >= s_(k) - GAP in
           the oracle, every oracle row scoring > s_(k) + GAP is returned, rows are
           distinct and in range, GPU scores are non-increasing and rows ascend among
           exactly equal GPU scores.
  fired    equal wherever the oracle's best score is further than GAP from theta.
  gather   bit-exact given the GPU's own (idx, score, fired): the expected continuation
           is recomputed by the oracle's copy routine for those neighbours.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W

SCORE_TOL = 2e-2
SCORE_BUG = 5e-5
GAP = 1e-3


def oracle_params(p: B.QueryParams, exclude=None) -> oracle.QueryParams:
    return oracle.QueryParams(k=p.k, theta=p.theta, offset=p.offset, depth_mode=p.depth_mode,
                              cont_len=p.cont_len, tier_thr=tuple(p.tier_thr),
                              tier_depth=tuple(p.tier_depth), exclude_tag=exclude)


def fill_both(w: W.Workload, device="cuda", n_rows=None, chunk_traces=64, **pool_kw):
    """Materialise workload w on `device`, append it to a CUDA pool and to the oracle."""
    n_rows = w.n_rows if n_rows is None else n_rows
    pool = B.Pool(w.d, n_rows + pool_kw.pop("spare_rows", 0), **pool_kw)
    ora = OraclePool(w.d, pool.key_format)
    done = 0
    for st, tk, tag in w.traces(device):
        if done >= n_rows:
            break
        if done + st.shape[0] > n_rows:
            st, tk = st[: n_rows - done].contiguous(), tk[: n_rows - done].contiguous()
        pool.append(st, tk, tag=tag, new_trace=True)
        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=tag, new_trace=True)
        done += st.shape[0]
    torch.cuda.synchronize()
    return pool, ora


def check_query(out: B.QueryOut, ora: OraclePool, q_bits: np.ndarray, params: B.QueryParams,
                exclude: np.ndarray | None = None, strict_scores: bool = True) -> dict:
    """Compare one CUDA query result with the oracle. Returns error statistics."""
    o = out.cpu()
    idx, score, fired = o.idx.numpy(), o.score.numpy(), o.fired.numpy()
    clen, ctok = o.cont_len.numpy(), o.cont_tok.numpy()
    nq, k = idx.shape
    N = len(ora)
    ref = ora.query(q_bits, oracle_params(params, exclude), want_all_scores=True)
    max_err = 0.0
    strict_sets = 0
    for q in range(nq):
        s_all = ref.all_scores[q]
        n_valid = int(np.sum(np.isfinite(s_all)))
        kk = min(k, n_valid)
        got = idx[q]
        # padding
        assert np.all(got[kk:] == -1), (q, got, kk)
        assert np.all(np.isneginf(score[q, kk:]))
        assert np.all(got[:kk] >= 0) and np.all(got[:kk] < N)
        assert len(set(got[:kk].tolist())) == kk, "duplicate rows returned"
        # scores of the returned rows
        if kk:
            err = np.abs(score[q, :kk].astype(np.float64) - s_all[got[:kk]].astype(np.float64))
            max_err = max(max_err, float(err.max()))
            assert err.max() <= SCORE_TOL
            if strict_scores:
                assert err.max() <= SCORE_BUG, f"score error {err.max():.3g} exceeds arithmetic bound"
        # ordering of the GPU's own output
        for j in range(1, kk):
            assert score[q, j - 1] >= score[q, j]
            if score[q, j - 1] == score[q, j]:
                assert got[j - 1] < got[j], "equal scores must list the lower row first"
        # sets
        want = ref.idx[q]
        if kk:
            s_k = float(ref.score[q, kk - 1])
            assert np.all(s_all[got[:kk]] >= s_k - GAP)
            must = np.where(s_all > s_k + GAP)[0]
            assert set(must.tolist()) <= set(got[:kk].tolist())
            srt = np.sort(s_all[np.isfinite(s_all)])[::-1]
            nxt = float(srt[kk]) if n_valid > kk else -np.inf
            if s_k - nxt > GAP:
                strict_sets += 1
                assert set(got[:kk].tolist()) == set(want[:kk].tolist())
            for j in range(kk):
                up = np.inf if j == 0 else float(srt[j - 1]) - float(srt[j])
                dn = np.inf if j + 1 >= n_valid else float(srt[j]) - float(srt[j + 1])
                if up > GAP and dn > GAP:
                    assert got[j] == want[j], (q, j)
        # firing rule
        if kk and abs(float(ref.score[q, 0]) - params.theta) > GAP:
            assert fired[q] == ref.fired[q]
        if kk == 0:
            assert fired[q] == 0
        # gather: bit-exact given the GPU's own neighbours
        for j in range(k):
            dep = 0
            if fired[q] and got[j] >= 0:
                dep = (params.cont_len if params.depth_mode == B.DEPTH_FIXED
                       else oracle.depth_by_rank(j, params.tier_depth) if params.depth_mode == B.DEPTH_RANKED
                       else oracle.depth(float(score[q, j]), params.tier_thr, params.tier_depth))
            exp_tok, exp_len = ora.gather_one(int(got[j]), dep, params.offset, params.cont_len)
            assert clen[q, j] == exp_len, (q, j, got[j], clen[q, j], exp_len)
            assert np.array_equal(ctok[q, j], exp_tok)
    return dict(max_score_err=max_err, strict_sets=strict_sets, oracle=ref)

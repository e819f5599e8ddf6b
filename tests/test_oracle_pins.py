"""Pins for the CPU oracle: it is checked against things other than itself.

Closed forms (+-1 pools whose scores are exact dyadic rationals), the constants the
paper prints (tests/golden), brute force on tiny pools, torch's own bf16 rounding,
and a library restatement (numpy matmul + lexsort).  No GPU, no CUDA library.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import DEPTH_FIXED, DEPTH_TIERED, OraclePool, QueryParams

GOLD = os.path.join(os.path.dirname(__file__), "golden")
P1, M1 = 0x3F80, 0xBF80  # bf16 bit patterns of +1.0 and -1.0


def pm1(rows):
    """Array of +-1 (given as +1/-1 ints) -> bf16 bit patterns."""
    a = np.asarray(rows)
    return np.where(a > 0, P1, M1).astype(np.uint16)


def hamming_row(base, h):
    """`base` (+-1 ints) with its first h entries flipped."""
    r = np.array(base, copy=True)
    r[:h] *= -1
    return r


# --------------------------------------------------------------------- T1 bf16 --

def test_bf16_widen_all_patterns_match_torch():
    bits = np.arange(65536, dtype=np.uint16)
    ours = oracle.bf16_bits_to_f32(bits)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    L = oracle.lib()
    for b in [0, 1, 0x3F80, 0xBF80, 0x7F7F, 0x0080, 0x8000, 0x7F80, 0xFF80]:
        assert np.float32(L.oracle_bf16_to_f32(b)).view(np.uint32) == (np.uint32(b) << 16)


def test_bf16_round_to_nearest_even_matches_torch_and_halfway_cases():
    L = oracle.lib()
    # every bf16 value round-trips
    for b in range(0, 65536, 7):
        f = float(oracle.bf16_bits_to_f32(np.array([b], np.uint16))[0])
        if f != f:
            continue
        assert L.oracle_f32_to_bf16(f) == b
    # halfway cases: 1 + 2^-8 is exactly between 1.0 (even) and 1+2^-7 (odd)
    assert L.oracle_f32_to_bf16(1.0 + 2.0**-8) == 0x3F80
    assert L.oracle_f32_to_bf16(1.0 + 2.0**-7 + 2.0**-8) == 0x3F82
    assert L.oracle_f32_to_bf16(np.float32(1.0 + 2.0**-8 + 2.0**-20)) == 0x3F81
    assert L.oracle_f32_to_bf16(-(1.0 + 2.0**-8)) == 0xBF80
    # against torch's rounding on a wide random sample (incl. tiny and huge values)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32),
                        (rng.standard_normal(2000) * 1e-30).astype(np.float32),
                        (rng.standard_normal(2000) * 1e30).astype(np.float32),
                        rng.integers(0, 2**32, 20000, dtype=np.uint32).view(np.float32)])
    x = x[np.isfinite(x)]
    ours = oracle.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)


# ------------------------------------------------- T2 closed form: Hamming pool --

@pytest.mark.parametrize("d", [16, 64, 256, 1024, 4096])
def test_hamming_pool_scores_order_and_ties_exact(d):
    rng = np.random.default_rng(d)
    base = rng.choice([-1, 1], size=d)
    hs = [0, 3, 1, d // 2, 3, d, 2, 1, 7, 3]           # designed ties: 3,3,3 and 1,1
    pool = OraclePool(d)
    pool.append(pm1([hamming_row(base, h) for h in hs]), np.arange(len(hs)), tag=1)
    s = pool.scores(pm1(base))
    want = np.array([1.0 - 2.0 * h / d for h in hs], dtype=np.float32)
    assert np.array_equal(s, want)                      # exact, not approximate
    # stored keys are exactly +-2^-m
    keys = oracle.bf16_bits_to_f32(pool.keys)
    assert np.array_equal(np.abs(keys), np.full_like(keys, 1.0 / np.sqrt(d)))
    res = pool.query(pm1(base), QueryParams(k=len(hs), theta=-2.0, depth_mode=DEPTH_FIXED,
                                            cont_len=1))
    # order by (h ascending, position ascending): lower position wins a tie
    order = sorted(range(len(hs)), key=lambda i: (hs[i], i))
    assert res.idx[0].tolist() == order
    assert np.array_equal(res.score[0], want[order])


def test_sparse_pm1_pool_each_vector_uses_its_own_norm():
    # supports of size 4^a normalise to exactly 2^-a: s = signed overlap / (|q| |k_i|)
    d = 256
    q = np.zeros(d, np.int64); q[:16] = 1                 # |q| = 4
    k0 = np.zeros(d, np.int64); k0[:4] = 1                 # |k| = 2, overlap 4  -> 4/8
    k1 = np.zeros(d, np.int64); k1[:64] = 1                # |k| = 8, overlap 16 -> 16/32
    k2 = np.zeros(d, np.int64); k2[8:24] = 1; k2[8:12] = -1  # |k| = 4, overlap -4+4 = 0
    k3 = np.zeros(d, np.int64); k3[:16] = -1               # -1
    def bits(v):
        return np.where(v > 0, P1, np.where(v < 0, M1, 0)).astype(np.uint16)
    pool = OraclePool(d)
    pool.append(np.stack([bits(k0), bits(k1), bits(k2), bits(k3)]), [0, 1, 2, 3], tag=1)
    s = pool.scores(bits(q))
    # k2: positions 8..11 are -1 (inside q's support), 12..15 are +1 (inside), 16..23 outside
    assert s.tolist() == [0.5, 0.5, 0.0, -1.0]
    res = pool.query(bits(q), QueryParams(k=4, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=1))
    assert res.idx[0].tolist() == [0, 1, 2, 3]           # 0.5 tie -> lower position first


# ------------------------------------------------------ T3 one-hot, k > N padding --

def test_one_hot_pool_and_padding_when_k_exceeds_rows():
    d, n = 64, 5
    eye = np.zeros((n, d), np.uint16)
    for i in range(n):
        eye[i, 3 * i] = P1
    pool = OraclePool(d)
    pool.append(eye, np.arange(10, 10 + n), tag=9)
    qv = np.zeros(d, np.uint16); qv[6] = 0x4000           # 2.0 * e_6 -> matches row 2
    res = pool.query(qv, QueryParams(k=8, theta=0.8, depth_mode=DEPTH_FIXED, cont_len=2))
    assert res.idx[0].tolist() == [2, 0, 1, 3, 4, -1, -1, -1]
    assert res.score[0, :5].tolist() == [1.0, 0.0, 0.0, 0.0, 0.0]
    assert np.all(np.isneginf(res.score[0, 5:]))
    assert res.fired[0] == 1
    assert res.cont_len[0].tolist() == [1, 2, 2, 0, 0, 0, 0, 0]   # clipped at the trace end (row 5)
    assert res.cont_tok[0, 0].tolist() == [14, -1]
    assert res.cont_tok[0, 1].tolist() == [12, 13]
    assert np.all(res.cont_tok[0, 5:] == -1)


def test_empty_pool():
    pool = OraclePool(32)
    res = pool.query(np.full(32, P1, np.uint16), QueryParams(k=3, cont_len=4))
    assert res.idx.tolist() == [[-1, -1, -1]] and res.fired.tolist() == [0]
    assert np.all(res.cont_tok == -1) and np.all(res.cont_len == 0)


# --------------------------------------------- T4/T5 duplicates, self-similarity --

def test_planted_duplicate_ranks_first_lowest_position_first():
    rng = np.random.default_rng(4)
    d, n = 128, 40
    x = rng.standard_normal((n, d)).astype(np.float32)
    x[19] = x[5]
    bits = oracle.f32_to_bf16_bits(x)
    pool = OraclePool(d)
    pool.append(bits, np.arange(n), tag=1)
    res = pool.query(bits[19], QueryParams(k=4, theta=0.8, depth_mode=DEPTH_FIXED, cont_len=1))
    assert res.idx[0, :2].tolist() == [5, 19]
    assert res.score[0, 0] == res.score[0, 1]
    assert abs(res.score[0, 0] - 1.0) < 1e-3
    assert res.score[0, 2] < 0.6


def test_self_similarity_is_maximal_and_scores_bounded():
    rng = np.random.default_rng(5)
    d, n = 256, 300
    bits = oracle.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32) * 3.0)
    pool = OraclePool(d)
    pool.append(bits, np.arange(n), tag=1)
    for i in (0, 17, 299):
        s = pool.scores(bits[i])
        assert int(np.argmax(s)) == i
        assert abs(s[i] - 1.0) < 1e-3
        assert np.all(np.abs(s) <= 1.0 + 1e-3)


# ------------------------------------------------ T6 theta and D(s) (paper values) --

def test_defaults_are_the_papers_constants():
    g = json.load(open(os.path.join(GOLD, "paper_constants.json")))
    p = QueryParams()
    assert p.k == g["k"]["value"] and p.offset == g["offset"]["value"]
    assert p.theta == g["theta"]["value"]
    assert list(p.tier_thr) == g["depth_tiers"]["thr"]
    assert list(p.tier_depth) == g["depth_tiers"]["depth"]
    assert p.depth_mode == DEPTH_TIERED


def test_theta_and_depth_tiers_on_exact_hamming_scores():
    d = 1024
    rows = [ln.split() for ln in open(os.path.join(GOLD, "hamming_d1024_thresholds.txt"))
            if ln.strip() and not ln.startswith("#")]
    base = np.ones(d, np.int64)
    for h, s, fired, dep in rows:
        h, s, fired, dep = int(h), float(s), int(fired), int(dep)
        pool = OraclePool(d)
        # row 0 is the neighbour; 60 more rows of the same trace supply the continuation
        filler = np.stack([hamming_row(base, d)] * 60)
        pool.append(pm1(np.concatenate([[hamming_row(base, h)], filler])), np.arange(61), tag=1)
        res = pool.query(pm1(base), QueryParams(cont_len=48))     # the paper's defaults
        assert res.score[0, 0] == np.float32(s)
        assert res.fired[0] == fired, (h, s)
        assert res.cont_len[0, 0] == dep, (h, s)
        assert oracle.depth(s) == dep
        if dep:
            assert res.cont_tok[0, 0, :dep].tolist() == list(range(2, 2 + dep))
        # theta is a firing condition on the best, not a floor inside the top-k:
        # the 60 far rows (s=-1) are still returned as neighbours 2..8
        assert np.all(res.idx[0, 1:] >= 1)


def test_theta_gates_on_best_only_and_lower_ranked_get_own_depth():
    d = 1024
    base = np.ones(d, np.int64)
    hs = [40, 60, 95, 200]                      # s = .9219 (48), .8828 (8), .8145 (0), .609 (0)
    body = [hamming_row(base, h) for h in hs] + [hamming_row(base, d)] * 60
    pool = OraclePool(d)
    pool.append(pm1(body), np.arange(len(body)), tag=1)
    res = pool.query(pm1(base), QueryParams(k=4, cont_len=48))
    assert res.idx[0].tolist() == [0, 1, 2, 3] and res.fired[0] == 1
    assert res.cont_len[0].tolist() == [48, 8, 0, 0]
    # best below theta: nothing is copied although neighbours are still reported
    pool2 = OraclePool(d)
    pool2.append(pm1(body[2:]), np.arange(len(body) - 2), tag=1)
    res2 = pool2.query(pm1(base), QueryParams(k=4, theta=0.82, cont_len=48))
    assert res2.fired[0] == 0 and res2.idx[0, 0] == 0 and np.all(res2.cont_len == 0)
    assert np.all(res2.cont_tok == -1)


def test_depth_by_rank_follows_the_table_whatever_the_scores():
    # the granularity ablation's arm: neighbour j copies tier_depth[j], the last entry from
    # there on; the scores only order the neighbours and decide the firing
    d = 1024
    base = np.ones(d, np.int64)
    hs = [200, 40, 95, 60, 300]                 # s = .609, .9219, .8145, .8828, .414 (rows 0..4)
    body = [hamming_row(base, h) for h in hs] + [hamming_row(base, d)] * 60
    pool = OraclePool(d)
    pool.append(pm1(body), np.arange(len(body)), tag=1)
    pr = QueryParams(k=5, cont_len=48, depth_mode=oracle.DEPTH_RANKED)          # the paper's {48, 8}
    res = pool.query(pm1(base), pr)
    assert res.idx[0].tolist() == [1, 3, 2, 0, 4] and res.fired[0] == 1
    assert res.cont_len[0].tolist() == [48, 8, 8, 8, 8]    # by similarity it would be 48, 8, 0, 0, 0
    assert res.cont_tok[0, 0, :3].tolist() == [3, 4, 5] and res.cont_tok[0, 3, :8].tolist() == list(range(2, 10))
    assert pool.query(pm1(base), QueryParams(k=5, cont_len=48)).cont_len[0].tolist() == [48, 8, 0, 0, 0]
    # a longer table, a depth above L (capped at L) and one of zero
    pr = QueryParams(k=5, cont_len=12, depth_mode=oracle.DEPTH_RANKED, tier_thr=(0, 0, 0), tier_depth=(20, 0, 3))
    assert pool.query(pm1(base), pr).cont_len[0].tolist() == [12, 0, 3, 3, 3]
    assert [oracle.depth_by_rank(j, (20, 0, 3)) for j in range(5)] == [20, 0, 3, 3, 3]
    assert oracle.depth_by_rank(0, ()) == 0
    # the firing rule is unchanged: best below theta, nothing is copied
    pr = QueryParams(k=5, theta=0.95, cont_len=48, depth_mode=oracle.DEPTH_RANKED)
    res = pool.query(pm1(base), pr)
    assert res.fired[0] == 0 and np.all(res.cont_len == 0) and np.all(res.cont_tok == -1)
    # clipped at the trace end like every copy: row 64 is the last of 65
    pr = QueryParams(k=1, theta=-2.0, cont_len=48, depth_mode=oracle.DEPTH_RANKED)
    far = pool.query(pm1(-base), pr)
    assert far.idx[0, 0] == 5 and far.cont_len[0, 0] == 48
    tail = OraclePool(d)
    tail.append(pm1(body[:6]), np.arange(6), tag=1)
    assert tail.query(pm1(base), QueryParams(k=2, cont_len=48, depth_mode=oracle.DEPTH_RANKED)
                      ).cont_len[0].tolist() == [3, 1]          # rows 1 and 3 of six


# ------------------------------------------------------------------- T7 gather --

def test_gather_offsets_clipping_and_trace_boundaries():
    d = 16
    pool = OraclePool(d)
    one = np.full((1, d), P1, np.uint16)
    pool.append(np.repeat(one, 10, 0), np.arange(100, 110), tag=1)        # rows 0..9
    pool.append(np.repeat(one, 6, 0), np.arange(200, 206), tag=2)         # rows 10..15
    pool.append(np.repeat(one, 3, 0), np.arange(206, 209), tag=2, new_trace=False)  # 16..18
    assert pool.trace_starts.tolist() == [0, 10] and pool.trace_ends.tolist() == [10, 19]
    assert pool.trace_ids.tolist() == [0] * 10 + [1] * 9
    L = 4
    cases = {  # (idx, dep, offset) -> tokens
        (0, 4, 2): [102, 103, 104, 105],
        (0, 4, 1): [101, 102, 103, 104],
        (5, 4, 2): [107, 108, 109],          # clipped at the end of trace 0
        (7, 4, 2): [109],
        (8, 4, 2): [],                       # idx+2 == trace end
        (9, 4, 2): [],                       # last row of trace 0: never leaks into trace 1
        (9, 4, 1): [],
        (10, 4, 2): [202, 203, 204, 205],
        (14, 4, 2): [206, 207, 208],         # continues through the extension of the open trace
        (18, 4, 2): [],
        (3, 0, 2): [],                       # depth 0
        (3, 2, 2): [105, 106],               # depth below L
        (3, 9, 2): [105, 106, 107, 108],     # depth above L is capped at L
    }
    for (i, dep, off), want in cases.items():
        out, n = pool.gather_one(i, dep, off, L)
        assert n == len(want), (i, dep, off)
        assert out.tolist() == want + [-1] * (L - len(want))


# ---------------------------------------------------------------- T8 exclusion --

def test_exclusion_tag_removes_exactly_the_tagged_traces():
    rng = np.random.default_rng(8)
    d = 64
    bits = oracle.f32_to_bf16_bits(rng.standard_normal((30, d)).astype(np.float32))
    pool = OraclePool(d)
    pool.append(bits[:10], np.arange(10), tag=7)
    pool.append(bits[10:20], np.arange(10, 20), tag=8)
    pool.append(bits[20:], np.arange(20, 30), tag=7)
    s_all = pool.scores(bits[3])
    s_ex = pool.scores(bits[3], exclude_tag=7)
    assert np.all(np.isneginf(s_ex[:10])) and np.all(np.isneginf(s_ex[20:]))
    assert np.array_equal(s_ex[10:20], s_all[10:20])
    res = pool.query(np.stack([bits[3], bits[3]]),
                     QueryParams(k=12, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=2,
                                 exclude_tag=np.array([7, 0], np.uint64)))
    assert set(res.idx[0, :10].tolist()) == set(range(10, 20))
    assert res.idx[0, 10:].tolist() == [-1, -1]
    assert res.idx[1, 0] == 3


# ------------------------------------------------------- T9 chunked append ≡ one --

def test_chunked_append_gives_identical_pool():
    rng = np.random.default_rng(9)
    d, n = 96, 50
    bits = oracle.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    toks = rng.integers(0, 1000, n).astype(np.int32)
    a, b = OraclePool(d), OraclePool(d)
    a.append(bits, toks, tag=3)
    b.append(bits[:7], toks[:7], tag=3)
    b.append(bits[7:8], toks[7:8], new_trace=False)
    b.append(bits[8:], toks[8:], new_trace=False)
    assert np.array_equal(a.keys, b.keys) and np.array_equal(a.tokens, b.tokens)
    assert np.array_equal(a.trace_ids, b.trace_ids)
    assert a.trace_starts.tolist() == b.trace_starts.tolist() == [0]
    assert a.trace_ends.tolist() == b.trace_ends.tolist() == [n]
    a.reset()
    assert len(a) == 0 and a.num_traces == 0


# ------------------------------------------- T10 library restatement (numpy) -----

def _numpy_topk(keys_bits, q_bits, k):
    """Textbook GEMV + sort on the stored operands: K @ q in float64, lexsort."""
    K = oracle.bf16_bits_to_f32(keys_bits).astype(np.float64)
    q = oracle.bf16_bits_to_f32(q_bits).astype(np.float64)
    s = (K @ q).astype(np.float32)
    order = np.lexsort((np.arange(len(s)), -s.astype(np.float64)))
    return order[:k], s


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_matches_numpy_matmul_and_sort_on_clustered_pool(seed):
    from paper_2608_03839_b200 import workloads as W
    w = W.C1.scaled(n_rows=1024, seed=100 + seed)
    pool = OraclePool(w.d)
    for st, tk, tag in w.traces():
        pool.append(W.to_bits(st), tk.numpy(), tag=tag)
    q, meta = w.queries()
    qb = W.to_bits(q)[0]
    res = pool.query(qb, QueryParams(k=w.k, theta=-2.0, depth_mode=DEPTH_FIXED,
                                     cont_len=w.cont_len), want_all_scores=True)
    # torch normalises the query independently (float64, then torch's own bf16 rounding)
    qn = (q[0].double() / q[0].double().norm()).float().to(torch.bfloat16)
    idx, s = _numpy_topk(pool.keys, W.to_bits(qn), w.k)
    assert np.allclose(res.all_scores[0], s, atol=2e-6)
    # identical ranking wherever the numpy scores are separated by more than rounding noise
    assert res.idx[0, 0] == meta["planted_row"] == idx[0]
    srt = np.sort(s)[::-1]
    for j in range(w.k):
        if (j == 0 or srt[j - 1] - srt[j] > 1e-5) and srt[j] - srt[j + 1] > 1e-5:
            assert res.idx[0, j] == idx[j]
    # keys themselves: torch's normalisation + rounding agrees bit for bit
    st0, _, _ = w.trace(0)
    kn = (st0.double() / st0.double().norm(dim=1, keepdim=True)).float().to(torch.bfloat16)
    assert np.array_equal(W.to_bits(kn), pool.keys[: st0.shape[0]])


def test_brute_force_tiny_pools_all_k():
    """Pure-Python definition on tiny pools: every k from 1 to N+3, with exact ties."""
    rng = np.random.default_rng(11)
    d = 16
    for n in (1, 2, 7, 33):
        # small-integer rows, many duplicates -> many exact ties
        x = rng.integers(-2, 3, size=(n, d)).astype(np.float32)
        x[x.sum(1) == 0, 0] = 1.0
        bits = oracle.f32_to_bf16_bits(x)
        pool = OraclePool(d)
        pool.append(bits, np.arange(n), tag=1)
        qb = oracle.f32_to_bf16_bits(rng.integers(-2, 3, size=d).astype(np.float32) + 0.5)
        keys = oracle.bf16_bits_to_f32(pool.keys).astype(np.float64)
        qn, _ = oracle.normalize_bf16(qb)
        qf = oracle.bf16_bits_to_f32(qn).astype(np.float64)
        sc = [np.float32(sum(float(qf[j]) * float(keys[i, j]) for j in range(d)))
              for i in range(n)]
        for k in range(1, n + 4):
            want = sorted(range(n), key=lambda i: (-float(sc[i]), i))[:k]
            res = pool.query(qb, QueryParams(k=k, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=1))
            assert res.idx[0, : len(want)].tolist() == want
            assert res.idx[0, len(want):].tolist() == [-1] * (k - len(want))
            assert res.score[0, : len(want)].tolist() == [float(sc[i]) for i in want]


# ------------------------------------------------------ T11 degenerate inputs ----

def test_zero_and_nonfinite_rows_and_queries_never_produce_nan():
    d = 32
    rng = np.random.default_rng(12)
    bits = oracle.f32_to_bf16_bits(rng.standard_normal((6, d)).astype(np.float32))
    bits[1, :] = 0                     # zero row
    bits[2, 5] = 0x7F80                # +inf
    bits[4, 0] = 0x7FC0                # NaN
    pool = OraclePool(d)
    pool.append(bits, np.arange(6), tag=1)
    assert pool.degenerate_rows == 3
    assert np.all(pool.keys[[1, 2, 4]] == 0)
    res = pool.query(bits[0], QueryParams(k=6, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=1))
    assert not np.any(np.isnan(res.score)) and res.idx[0, 0] == 0
    assert sorted(res.idx[0][res.score[0] == 0.0].tolist()) == [1, 2, 4]   # zero keys score 0
    # zero query: every score is 0, ties resolve to the lowest positions
    z = pool.query(np.zeros(d, np.uint16), QueryParams(k=3, theta=0.8, depth_mode=DEPTH_FIXED,
                                                       cont_len=1))
    assert z.idx[0].tolist() == [0, 1, 2] and z.score[0].tolist() == [0.0, 0.0, 0.0]
    assert z.fired[0] == 0
    # NaN query: no neighbours at all
    bad = bits[0].copy(); bad[3] = 0x7FC0
    r = pool.query(bad, QueryParams(k=3, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=1))
    assert r.idx[0].tolist() == [-1, -1, -1] and r.fired[0] == 0
    assert np.all(np.isneginf(r.score))


# ---------------------------------------------------------- metamorphic invariants --

def test_query_scale_invariance_and_row_permutation():
    rng = np.random.default_rng(13)
    d, n = 128, 200
    x = rng.standard_normal((n, d)).astype(np.float32)
    bits = oracle.f32_to_bf16_bits(x)
    qb = oracle.f32_to_bf16_bits(rng.standard_normal(d).astype(np.float32))
    q8 = oracle.f32_to_bf16_bits(oracle.bf16_bits_to_f32(qb) * 8.0)    # exact power of two
    pool = OraclePool(d)
    pool.append(bits, np.arange(n), tag=1)
    pr = QueryParams(k=10, theta=-2.0, depth_mode=DEPTH_FIXED, cont_len=1)
    a, b = pool.query(qb, pr, True), pool.query(q8, pr, True)
    assert np.array_equal(a.idx, b.idx) and np.array_equal(a.all_scores, b.all_scores)
    perm = rng.permutation(n)
    pool2 = OraclePool(d)
    pool2.append(bits[perm], np.arange(n), tag=1)
    c = pool2.query(qb, pr, True)
    assert np.array_equal(c.all_scores[0], a.all_scores[0][perm])
    assert np.array_equal(perm[c.idx[0]], a.idx[0])     # no exact ties in random data

"""Pins for the coarse-index oracle (oracle/index.py), all on the CPU.

The index answers with the brute-force result restricted to the rows of the probed lists
plus the tail, so it is pinned (1) against brute force where every list is probed, (2) by a
pool built by hand whose lists, probes and answers can be written down, (3) by the
properties any inverted file has: candidates only grow with n_probe, the tail is always
scanned, ties between centroids go to the lower one.
"""
import numpy as np
import pytest

import oracle
from oracle import OraclePool
from oracle.index import OracleIndex

f2b = oracle.f32_to_bf16_bits


def fixed(k, L=2, theta=-np.inf, **kw):
    return oracle.QueryParams(k=k, theta=theta, depth_mode=oracle.DEPTH_FIXED, cont_len=L, **kw)


def random_pool(rng, n, d, n_traces=4, key_format="bf16"):
    pool = OraclePool(d, key_format)
    rows = rng.standard_normal((n, d)).astype(np.float32)
    bits = f2b(rows)
    per = n // n_traces
    for t in range(n_traces):
        lo, hi = t * per, n if t == n_traces - 1 else (t + 1) * per
        pool.append(bits[lo:hi], np.arange(lo, hi, dtype=np.int32) + 100, tag=t + 1)
    return pool, bits


@pytest.mark.parametrize("key_format", ["bf16", "e4m3"])
@pytest.mark.parametrize("n_lists", [1, 3, 16])
def test_all_lists_probed_is_brute_force(n_lists, key_format):
    rng = np.random.default_rng(n_lists)
    pool, bits = random_pool(rng, 300, 32, key_format=key_format)
    idx = OracleIndex(pool, f2b(rng.standard_normal((n_lists, 32)).astype(np.float32)))
    idx.refresh()
    assert idx.n_indexed == 300 and sum(len(l) for l in idx.lists()) == 300
    q = f2b(rng.standard_normal((5, 32)).astype(np.float32))
    for k in (1, 7, 40):
        pr = fixed(k, L=3, theta=0.1)
        a, b = idx.query(q, n_lists, pr), pool.query(q, pr)
        assert np.array_equal(a.idx, b.idx) and np.array_equal(a.score, b.score)
        assert np.array_equal(a.fired, b.fired) and np.array_equal(a.cont_len, b.cont_len)
        assert np.array_equal(a.cont_tok, b.cont_tok)
        # more probes than lists change nothing
        c = idx.query(q, n_lists + 5, pr)
        assert np.array_equal(c.idx, b.idx)


def hand_pool():
    """d = 4, three centroids e0, e1, e2; seven rows whose lists can be read off:
         row 0 = (1, .1, 0, 0) -> list 0      row 1 = (.2, 1, 0, 0) -> list 1
         row 2 = (.9, .3, 0, 0) -> list 0     row 3 = (0, .1, 1, 0) -> list 2
         row 4 = (.6, .8, 0, 0) -> list 1     row 5 = (.5, .5, 0, 0) -> tie 0/1 -> list 0
         row 6 = (0, 0, .3, 1)  -> list 2 (its best centroid, however poor)"""
    rows = np.array([[1, .1, 0, 0], [.2, 1, 0, 0], [.9, .3, 0, 0], [0, .1, 1, 0],
                     [.6, .8, 0, 0], [.5, .5, 0, 0], [0, 0, .3, 1]], dtype=np.float32)
    pool = OraclePool(4)
    pool.append(f2b(rows), np.arange(7, dtype=np.int32) + 10, tag=1)
    cent = f2b(np.eye(4, dtype=np.float32)[:3])
    return pool, OracleIndex(pool, cent), rows


def test_hand_built_lists_probes_and_answers():
    pool, idx, rows = hand_pool()
    idx.refresh()
    assert idx.assign.tolist() == [0, 1, 0, 2, 1, 0, 2]
    assert [l.tolist() for l in idx.lists()] == [[0, 2, 5], [1, 4], [3, 6]]
    q = f2b(np.array([[1.0, 0.45, 0.0, 0.0]], dtype=np.float32))
    assert idx.probes(q, 2).tolist() == [[0, 1]] and idx.probes(q, 5).tolist() == [[0, 1, 2, -1, -1]]
    # cosines with q, by hand: rows 0..6 = .951, .567, .999(2), .041, .875, .933, 0
    # one probe (list 0 = rows 0, 2, 5): the best three are 2, 0, 5 and row 4 (.875) is missed
    r1 = idx.query(q, 1, fixed(4))
    assert r1.idx.tolist() == [[2, 0, 5, -1]]
    # copies start two rows on (tokens are 10 + row) and stop at the end of the trace (row 7)
    assert np.isneginf(r1.score[0, 3]) and r1.cont_len[0].tolist() == [2, 2, 0, 0]
    assert r1.cont_tok[0].tolist() == [[14, 15], [12, 13], [-1, -1], [-1, -1]]
    # two probes add list 1 (rows 1, 4): row 4 now ranks fourth
    r2 = idx.query(q, 2, fixed(4))
    assert r2.idx.tolist() == [[2, 0, 5, 4]]
    # all three: identical to brute force
    assert np.array_equal(idx.query(q, 3, fixed(7)).idx, pool.query(q, fixed(7)).idx)
    # theta applies to the best candidate
    assert idx.query(q, 1, fixed(2, theta=0.9995)).fired.tolist() == [0]
    assert idx.query(q, 1, fixed(2, theta=0.99)).fired.tolist() == [1]


def test_tail_rows_are_always_candidates_and_refresh_moves_them_into_lists():
    pool, idx, rows = hand_pool()
    idx.refresh()
    # a new row in the direction of e2, appended after the refresh: no list holds it yet
    new = f2b(np.array([[0.05, 0.0, 1.0, 0.1]], dtype=np.float32))
    pool.append(new, np.array([99], dtype=np.int32), tag=2)
    q = f2b(np.array([[0.0, 0.0, 1.0, 0.05]], dtype=np.float32))
    # probing list 0 only (nothing there is close): the tail row is still found, and first
    far = f2b(np.array([[1.0, 0.0, 0.0, 0.0]], dtype=np.float32))
    assert idx.probes(far, 1).tolist() == [[0]]
    got = idx.query(q, 1, fixed(2))
    assert got.idx[0].tolist() == [7, 3]            # list 2 probed: tail row 7, then row 3
    # list 0 probed (rows 0, 2, 5): the tail row is a candidate all the same, here the last
    assert idx.query(far, 1, fixed(5)).idx[0].tolist() == [0, 2, 5, 7, -1]
    assert idx.n_indexed == 7
    idx.refresh()
    assert idx.n_indexed == 8 and idx.assign[7] == 2
    assert idx.query(far, 1, fixed(2)).idx[0].tolist() == [0, 2]     # no tail any more


def test_duplicate_centroids_tie_to_the_lower_and_empty_lists_are_harmless():
    rng = np.random.default_rng(7)
    pool, bits = random_pool(rng, 120, 16)
    c = rng.standard_normal((4, 16)).astype(np.float32)
    c[3] = c[1]                                              # list 3 can never win a tie
    idx = OracleIndex(pool, f2b(c))
    idx.refresh()
    assert len(idx.lists()[3]) == 0
    q = f2b(rng.standard_normal((3, 16)).astype(np.float32))
    pr = fixed(5)
    # probing the empty list adds nothing
    p = idx.probes(q, 4)
    assert all(3 in row for row in p.tolist())
    assert np.array_equal(idx.query(q, 4, pr).idx, pool.query(q, pr).idx)


def test_candidates_grow_with_n_probe_and_so_does_recall():
    rng = np.random.default_rng(11)
    pool, bits = random_pool(rng, 2000, 24, n_traces=10)
    idx = OracleIndex(pool, bits[rng.choice(2000, 32, replace=False)])   # 32 stored rows as centroids
    idx.refresh()
    q = f2b(rng.standard_normal((6, 24)).astype(np.float32))
    pr = fixed(10)
    exact = pool.query(q, pr)
    prev_mask = [np.zeros(2000, bool)] * 6
    prev_hits = [0] * 6
    for n_probe in (1, 2, 4, 8, 16, 32):
        res = idx.query(q, n_probe, pr, want_all_scores=True)
        probes = idx.probes(q, n_probe)
        for i in range(6):
            mask = idx.candidates(probes[i])
            assert np.all(mask[prev_mask[i]])                    # nothing ever leaves
            prev_mask[i] = mask
            hits = len(set(res.idx[i].tolist()) & set(exact.idx[i].tolist()))
            assert hits >= prev_hits[i]
            prev_hits[i] = hits
            # what is returned is the best of the candidates, nothing else
            assert np.all(mask[res.idx[i][res.idx[i] >= 0]])
            kth = res.score[i, -1]
            assert np.all(res.all_scores[i][mask] <= res.score[i, 0])
            assert np.sum(res.all_scores[i] > kth) <= 10
    assert prev_hits == [10] * 6


def test_exclusion_and_reset():
    rng = np.random.default_rng(13)
    pool, bits = random_pool(rng, 200, 16, n_traces=4)        # tags 1..4, 50 rows each
    idx = OracleIndex(pool, f2b(rng.standard_normal((5, 16)).astype(np.float32)))
    idx.refresh()
    q = bits[[60]].copy()                                     # a stored row of trace 2 (tag 2)
    plain = idx.query(q, 5, fixed(3))
    assert plain.idx[0, 0] == 60
    ex = idx.query(q, 5, fixed(3, exclude_tag=np.array([2], dtype=np.uint64)))
    assert np.all((ex.idx[0] < 50) | (ex.idx[0] >= 100))
    idx.reset()
    assert idx.n_indexed == 0
    # with nothing indexed every row is tail: brute force whatever is probed
    assert np.array_equal(idx.query(q, 1, fixed(3)).idx, pool.query(q, fixed(3)).idx)


# ---- training (Lloyd's iterations) ------------------------------------------------------

def pm1_pool(rows):
    """Rows of +-1 with d = 16 normalise to +-0.25 exactly, so means can be written down."""
    pool = OraclePool(16)
    pool.append(f2b(np.asarray(rows, dtype=np.float32)), np.arange(len(rows), dtype=np.int32), tag=1)
    return pool


# ------------------------------------------------------------------ 8-bit pools ----

def test_8bit_rows_along_axes_and_diagonals_fall_into_the_lists_read_off_by_hand():
    # A row along an axis keeps one non-zero code, so whatever its scale it dequantises to a
    # multiple of that axis and, as a query, normalises to the axis exactly; a row with two
    # equal entries keeps two equal codes and so ties between the two axes, to the lower one.
    r = np.float32(1.0)
    rows = np.array([[r, 0, 0, 0], [0, 3 * r, 0, 0], [-r, 0, 0, 0], [0, 0, 0.5 * r, 0],
                     [r, r, 0, 0], [0, r, r, 0], [0, 0, -2 * r, 0]], dtype=np.float32)
    pool = OraclePool(4, "e4m3")
    pool.append(f2b(rows), np.arange(7, dtype=np.int32) + 10, tag=1)
    idx = OracleIndex(pool, f2b(np.eye(4, dtype=np.float32)[:3]))
    idx.refresh()
    #   e0 -> 0, 3 e1 -> 1, -e0 -> scores (-1, 0, 0): tie of lists 1 and 2 -> 1, e2/2 -> 2,
    #   e0+e1 -> tie 0/1 -> 0, e1+e2 -> tie 1/2 -> 1, -2 e2 -> scores (0, 0, -1) -> tie 0/1 -> 0
    assert idx.assign.tolist() == [0, 1, 1, 2, 0, 1, 0]
    # the rows as the index sees them: element = fp32(value(code) * scale), one rounding
    got = idx._stored_f32(0, 7)
    codes, scales = pool.codes, pool.scales
    for i in range(7):
        for j in range(4):
            want = np.float32(np.float64(oracle.e4m3_decode(int(codes[i, j]))) * np.float64(scales[i]))
            assert got[i, j] == want
        assert np.count_nonzero(got[i]) == np.count_nonzero(rows[i])
    assert got[4, 0] == got[4, 1] and got[5, 1] == got[5, 2]
    # and as queries: bf16 of those elements
    assert np.array_equal(idx._stored_as_queries(0, 7), f2b(got))
    # a lookup probes by the query, scores by the 8-bit pool's own rule
    q = f2b(np.array([[1.0, 0.2, 0.0, 0.0]], dtype=np.float32))
    assert idx.probes(q, 2).tolist() == [[0, 1]]
    one = idx.query(q, 1, fixed(3))
    assert one.idx[0].tolist() == [0, 4, 6]                 # list 0 = rows 0, 4, 6: cos .98, .83, 0
    full = pool.query(q, fixed(3))
    assert np.array_equal(one.score[0, :2], full.score[0, :2])


def test_8bit_training_takes_the_means_of_the_dequantised_elements():
    rng = np.random.default_rng(5)
    d, n = 8, 120
    rows = (rng.standard_normal((n, d)) * np.exp(rng.uniform(-4, 0, size=(n, d)))).astype(np.float32)
    pool = OraclePool(d, "e4m3")
    pool.append(f2b(rows), np.arange(n, dtype=np.int32), tag=1)
    idx = OracleIndex(pool, f2b(np.ones((1, d), dtype=np.float32)))
    idx.train(1)                                            # one list: the mean of every row
    from fractions import Fraction
    codes, scales = pool.codes, pool.scales
    for j in range(d):
        total = 0
        for i in reversed(range(n)):                        # Python ints, another order
            x = np.float32(np.float64(oracle.e4m3_decode(int(codes[i, j]))) * np.float64(scales[i]))
            total += int(np.trunc(np.float64(x) * 2.0 ** 30))
        want = f2b(np.array([np.float32(float(Fraction(total, n * 2 ** 30)))]))[0]
        assert idx.cent_raw[0, j] == want
    assert idx.n_indexed == n and idx.assign.tolist() == [0] * n


def test_one_iteration_by_hand():
    a = [1.0] * 16
    b = [1.0] * 12 + [-1.0] * 4          # cos(a, b) = 0.5
    c = [-1.0] * 16
    e = [-1.0] * 8 + [1.0] * 8           # cos(c, e) = 0, cos(a, e) = 0
    pool = pm1_pool([a, b, c, e, a])
    # centroid 0 near a, centroid 1 near c, centroid 2 = e exactly (but rows tie towards lower
    # centroids only when scores are equal: e scores 1 against centroid 2)
    c0 = [1.0] * 15 + [0.5]
    c1 = [-1.0] * 15 + [-0.5]
    idx = OracleIndex(pool, f2b(np.array([c0, c1, e, [0.0] * 15 + [1.0]], dtype=np.float32)))
    idx.train(1)
    # lists after the iteration's own assignment: {a, b, a} -> 0, {c} -> 1, {e} -> 2, none -> 3
    got = oracle.bf16_bits_to_f32(idx.cent_raw)
    mean0 = (2 * np.array(a) * 0.25 + np.array(b) * 0.25) / 3        # 0.25 x 12, 0.25/3 x 4
    assert np.array_equal(got[0], oracle.bf16_bits_to_f32(f2b(mean0.astype(np.float32))))
    assert np.array_equal(got[0][:12], np.full(12, 0.25, dtype=np.float32))
    assert np.array_equal(got[0][12:], oracle.bf16_bits_to_f32(f2b(np.full(4, 0.25 / 3, np.float32))))
    assert np.array_equal(got[1], np.full(16, -0.25, dtype=np.float32))     # the one row itself
    assert np.array_equal(got[2], np.array(e, dtype=np.float32) * 0.25)
    assert np.array_equal(idx.cent_raw[3], f2b(np.array([0.0] * 15 + [1.0], dtype=np.float32)))  # kept
    assert idx.n_indexed == 5
    assert [l.tolist() for l in idx.lists()] == [[0, 1, 4], [2], [3], []]


def test_fixed_point_sum_is_exact_and_order_free():
    # many rows whose elements differ wildly in size: the integer sum is the same whatever
    # the order, and equals the exact rational sum of the truncated terms
    rng = np.random.default_rng(3)
    d, n = 8, 200
    rows = (rng.standard_normal((n, d)) * np.exp(rng.uniform(-12, 0, size=(n, d)))).astype(np.float32)
    pool = OraclePool(d)
    pool.append(f2b(rows), np.arange(n, dtype=np.int32), tag=1)
    idx = OracleIndex(pool, f2b(np.ones((1, d), dtype=np.float32)))
    idx.train(1)
    x = oracle.bf16_bits_to_f32(pool.keys).astype(np.float64)
    from fractions import Fraction
    for j in range(d):
        total = sum(int(np.trunc(v * 2.0 ** 30)) for v in x[::-1, j])          # Python ints, reversed
        mean = Fraction(total, n * 2 ** 30)
        want = f2b(np.array([np.float32(float(mean))]))[0]                      # float(Fraction) is correctly rounded
        assert idx.cent_raw[0, j] == want


def test_training_is_a_fixed_point_once_converged_and_never_lowers_the_objective():
    rng = np.random.default_rng(11)
    d, n, n_lists = 32, 600, 12
    cent = rng.standard_normal((n_lists, d))
    rows = cent[rng.integers(0, n_lists, n)] + 0.3 * rng.standard_normal((n, d))
    pool = OraclePool(d)
    pool.append(f2b(rows.astype(np.float32)), np.arange(n, dtype=np.int32), tag=1)
    start = f2b(rows[:n_lists].astype(np.float32))                 # twelve rows as first centroids
    idx = OracleIndex(pool, start)
    one = fixed(1)

    def objective(ix):
        return float(ix.cent.query(pool.keys, one).score[:, 0].astype(np.float64).sum())

    idx.refresh()
    obj = [objective(idx)]
    for _ in range(6):
        idx.train(1)
        obj.append(objective(idx))
    assert all(b >= a - 1e-3 for a, b in zip(obj, obj[1:])) and obj[-1] > obj[0] + 1.0
    # several single iterations equal one call with that many
    again = OracleIndex(pool, start)
    again.train(6)
    assert np.array_equal(again.cent_raw, idx.cent_raw) and np.array_equal(again.assign, idx.assign)
    # converged: further iterations change nothing
    for _ in range(20):
        before = idx.cent_raw.copy()
        idx.train(1)
        if np.array_equal(before, idx.cent_raw):
            break
    before, lists = idx.cent_raw.copy(), [l.tolist() for l in idx.lists()]
    idx.train(2)
    assert np.array_equal(before, idx.cent_raw) and lists == [l.tolist() for l in idx.lists()]
    # and the answers with every list probed are still brute force
    q = f2b(rng.standard_normal((4, d)).astype(np.float32))
    a, b = idx.query(q, n_lists, fixed(9)), pool.query(q, fixed(9))
    assert np.array_equal(a.idx, b.idx) and np.array_equal(a.score, b.score)


def test_training_raises_recall_at_one_probe():
    rng = np.random.default_rng(5)
    d, n, n_clusters = 48, 3000, 30
    cent = rng.standard_normal((n_clusters, d))
    who = rng.integers(0, n_clusters, n)
    rows = cent[who] + 0.25 * rng.standard_normal((n, d))
    pool = OraclePool(d)
    pool.append(f2b(rows.astype(np.float32)), np.arange(n, dtype=np.int32), tag=1)
    idx = OracleIndex(pool, f2b(rows[:n_clusters].astype(np.float32)))   # a poor start: the first rows
    q = f2b((cent[rng.integers(0, n_clusters, 40)] + 0.25 * rng.standard_normal((40, d))).astype(np.float32))
    exact = pool.query(q, fixed(10)).idx

    def recall(ix):
        got = ix.query(q, 1, fixed(10)).idx
        return np.mean([len(set(got[i]) & set(exact[i])) / 10 for i in range(40)])

    idx.refresh()
    r0 = recall(idx)
    idx.train(5)
    assert recall(idx) > r0 + 0.1

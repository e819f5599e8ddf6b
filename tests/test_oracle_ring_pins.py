"""Pins for the recycled-pool oracle (Section 4 (i b); Algorithm 1's recycled-pool line):
closed-form +-1 pools, the constants the paper prints, ring-buffer semantics by hand, and a
numpy restatement.  CPU only."""
import json
import os

import numpy as np

import oracle
from oracle import OracleRing

GOLD = os.path.join(os.path.dirname(__file__), "golden")
P1, M1 = 0x3F80, 0xBF80


def pm1(a):
    return np.where(np.asarray(a) > 0, P1, M1).astype(np.uint16)


def flipped(base, h):
    r = np.array(base, copy=True)
    r[:h] *= -1
    return r


def test_paper_constants_of_the_recycled_pool():
    g = json.load(open(os.path.join(GOLD, "paper_constants.json")))
    assert oracle.PAPER_RING_M == g["ring_max_results"]["value"] == 4
    assert oracle.PAPER_RING_FLOOR == g["ring_cos_floor"]["value"] == 0.8
    assert oracle.PAPER_ROLLOUT == g["ring_rollout_depth"]["value"] == 6


def test_anchor_equality_floor_order_and_cap_on_exact_scores():
    d = 1024                                   # s = 1 - 2h/1024 exactly
    base = np.ones(d, np.int64)
    #            h    anchor
    recs = [(102, 7),    # 0.80078  anchor 7  -> qualifies (just above the floor)
            (103, 7),    # 0.79883  anchor 7  -> below the floor: filtered out
            (10, 9),     # 0.98     anchor 9  -> other anchor: never returned
            (40, 7),     # 0.92188
            (40, 7),     # tie with the previous: lower slot first
            (0, 7),      # 1.0
            (60, 7),     # 0.88281
            (80, 7)]     # 0.84375  -> sixth qualifying record, cut by m = 4
    ring = OracleRing(d, 16)
    roll = np.full((len(recs), 6), -1, np.int32)
    for i in range(len(recs)):
        roll[i, : (i % 6) + 1] = np.arange(100 * i, 100 * i + (i % 6) + 1)
    ring.append(pm1([flipped(base, h) for h, _ in recs]), [a for _, a in recs], roll)
    res = ring.query(pm1(base), [7])           # the paper's m = 4, floor = 0.8
    assert res.slot[0].tolist() == [5, 3, 4, 6]
    assert res.score[0].tolist() == [1.0, 1 - 80 / 1024, 1 - 80 / 1024, 1 - 120 / 1024]
    assert res.count[0] == 4
    for j, s in enumerate(res.slot[0]):
        n = (s % 6) + 1
        assert res.rollout_len[0, j] == n
        assert res.rollout[0, j].tolist() == list(range(100 * s, 100 * s + n)) + [-1] * (6 - n)
    # all qualifying records when m is large: the floor is a per-record filter
    big = ring.query(pm1(base), [7], m=8)
    assert big.slot[0].tolist() == [5, 3, 4, 6, 7, 0, -1, -1] and big.count[0] == 6
    assert big.score[0, 5] == np.float32(1 - 204 / 1024) and np.isneginf(big.score[0, 6])
    assert np.all(big.rollout[0, 6:] == -1) and np.all(big.rollout_len[0, 6:] == 0)
    # an anchor nobody stored
    none = ring.query(pm1(base), [12345])
    assert none.count[0] == 0 and np.all(none.slot == -1)
    # two queries at once, each with its own anchor
    two = ring.query(np.stack([pm1(base), pm1(base)]), [9, 7], m=2)
    assert two.slot.tolist() == [[2, -1], [5, 3]] and two.count.tolist() == [1, 2]


def test_ring_overwrites_the_oldest_records():
    d, cap = 64, 5
    rng = np.random.default_rng(1)
    x = rng.standard_normal((12, d)).astype(np.float32)
    bits = oracle.f32_to_bf16_bits(x)
    roll = np.tile(np.arange(12, dtype=np.int32)[:, None], (1, 6))
    ring = OracleRing(d, cap)
    ring.append(bits[:3], [1, 1, 1], roll[:3])
    assert len(ring) == 3 and ring.total == 3
    ring.append(bits[3:7], [1, 1, 1, 1], roll[3:7])      # records 5, 6 overwrite slots 0, 1
    assert len(ring) == 5 and ring.total == 7
    assert ring.rollouts[:, 0].tolist() == [5, 6, 2, 3, 4]
    # record 0 is gone: its own state no longer finds it; record 6 is found in slot 1
    r0 = ring.query(bits[0], [1], m=1, floor=0.99)
    assert r0.count[0] == 0
    r6 = ring.query(bits[6], [1], m=1, floor=0.99)
    assert r6.slot[0, 0] == 1 and r6.rollout[0, 0, 0] == 6
    ring.append(bits[7:12], [2] * 5, roll[7:12])         # a whole lap
    assert ring.rollouts[:, 0].tolist() == [10, 11, 7, 8, 9] and set(ring.anchors) == {2}
    ring.reset()
    assert len(ring) == 0 and ring.query(bits[8], [2]).count[0] == 0


def test_matches_numpy_restatement_on_random_ring():
    rng = np.random.default_rng(2)
    d, cap, n = 128, 300, 420                     # wraps once
    cent = rng.standard_normal((6, d)).astype(np.float32)
    x = cent[rng.integers(0, 6, n)] + 0.4 * rng.standard_normal((n, d)).astype(np.float32)
    bits = oracle.f32_to_bf16_bits(x)
    anchors = rng.integers(0, 5, n).astype(np.int32)
    roll = rng.integers(0, 1000, (n, 6)).astype(np.int32)
    roll[rng.random((n, 6)) < 0.2] = -1
    ring = OracleRing(d, cap)
    for lo in range(0, n, 50):
        ring.append(bits[lo:lo + 50], anchors[lo:lo + 50], roll[lo:lo + 50])
    # what the ring must hold: record i lives in slot i % cap, the newest wins
    keep = {i % cap: i for i in range(n)}
    q = oracle.f32_to_bf16_bits(cent[:3] + 0.4 * rng.standard_normal((3, d)).astype(np.float32))
    qa = np.array([0, 3, 4], np.int32)
    res = ring.query(q, qa, m=6, floor=0.5)
    K = oracle.bf16_bits_to_f32(ring.keys).astype(np.float64)
    for qi in range(3):
        qn, _ = oracle.normalize_bf16(q[qi])
        s = (K @ oracle.bf16_bits_to_f32(qn).astype(np.float64)).astype(np.float32)
        ok = [sl for sl in range(cap) if anchors[keep[sl]] == qa[qi] and s[sl] >= np.float32(0.5)]
        want = sorted(ok, key=lambda sl: (-float(s[sl]), sl))[:6]
        assert res.slot[qi, : len(want)].tolist() == want
        assert res.count[qi] == len(want)
        for j, sl in enumerate(want):
            r = roll[keep[sl]]
            neg = np.where(r < 0)[0]
            ln = int(neg[0]) if len(neg) else 6
            assert res.rollout_len[qi, j] == ln
            assert res.rollout[qi, j, :ln].tolist() == r[:ln].tolist()
            assert np.all(res.rollout[qi, j, ln:] == -1)

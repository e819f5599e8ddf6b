"""GPU parity of the recycled pool (rejected-branch ring buffer) against its CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OracleRing
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W

pytestmark = pytest.mark.gpu
P1, M1 = 0x3F80, 0xBF80
GAP, SCORE_BUG = 1e-3, 5e-5


def dev_bits(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def ring_inputs(n, d, vocab, seed, n_cent=16, sigma=0.3, R=6):
    g = torch.Generator(device="cuda").manual_seed(seed)
    cent = torch.randn(n_cent, d, generator=g, device="cuda")
    c = torch.randint(0, n_cent, (n,), generator=g, device="cuda")
    st = (cent[c] + sigma * torch.randn(n, d, generator=g, device="cuda")).to(torch.bfloat16)
    anc = torch.randint(0, vocab, (n,), generator=g, device="cuda", dtype=torch.int32)
    roll = torch.randint(0, 50000, (n, R), generator=g, device="cuda", dtype=torch.int32)
    ln = torch.randint(0, R + 1, (n,), generator=g, device="cuda")
    roll[torch.arange(R, device="cuda")[None, :] >= ln[:, None]] = -1
    return cent, st, anc, roll


def check(out, ref_ring, q_bits, q_anchor, m, floor):
    o = out.cpu()
    ref = ref_ring.query(q_bits, q_anchor, m=m, floor=floor)
    # full information: every stored slot's score, from a wide-open oracle query
    allr = ref_ring.query(q_bits, q_anchor, m=min(len(ref_ring), 4096) or 1, floor=-2.0)
    for qi in range(o.slot.shape[0]):
        got = o.slot[qi].numpy()
        cnt = int(o.count[qi])
        assert np.all(got[cnt:] == -1) and np.all(np.isneginf(o.score[qi, cnt:].numpy()))
        assert np.all(got[:cnt] >= 0) and len(set(got[:cnt].tolist())) == cnt
        s_of = {int(s): float(v) for s, v in zip(allr.slot[qi], allr.score[qi]) if s >= 0}
        for j in range(cnt):
            assert int(got[j]) in s_of, "returned a slot whose anchor does not match"
            assert abs(float(o.score[qi, j]) - s_of[int(got[j])]) < SCORE_BUG
            assert o.score[qi, j] >= np.float32(floor)
            if j:
                assert o.score[qi, j - 1] >= o.score[qi, j]
                if o.score[qi, j - 1] == o.score[qi, j]:
                    assert got[j - 1] < got[j]
        # records clearly above the floor and clearly inside the top m must be there
        want = [int(s) for s in ref.slot[qi] if s >= 0]
        kth = float(ref.score[qi, m - 1]) if len(want) == m else floor
        must = [s for s, v in s_of.items() if v > max(kth, floor) + GAP]
        assert set(must) <= set(got[:cnt].tolist())
        assert cnt >= len([s for s, v in s_of.items() if v >= floor + GAP][:m]) or cnt == m
        # continuation: bit-exact given the slots
        rolls = ref_ring.rollouts
        for j in range(cnt):
            r = rolls[int(got[j])]
            neg = np.where(r < 0)[0]
            ln = int(neg[0]) if len(neg) else len(r)
            assert o.rollout_len[qi, j] == ln
            assert o.rollout[qi, j].tolist() == r[:ln].tolist() + [-1] * (len(r) - ln)
        assert torch.all(o.rollout[qi, cnt:] == -1) and torch.all(o.rollout_len[qi, cnt:] == 0)


def test_exact_scores_floor_ties_and_cap():
    d = 1024
    base = np.ones(d, np.int64)
    recs = [(102, 7), (103, 7), (10, 9), (40, 7), (40, 7), (0, 7), (60, 7), (80, 7)]
    rows = np.stack([np.where(np.arange(d) < h, -base, base) for h, _ in recs])
    bits = np.where(rows > 0, P1, M1).astype(np.uint16)
    anc = np.array([a for _, a in recs], np.int32)
    roll = np.full((len(recs), 6), -1, np.int32)
    for i in range(len(recs)):
        roll[i, : (i % 6) + 1] = np.arange(100 * i, 100 * i + (i % 6) + 1)
    ring, ora = B.Ring(d, 16), OracleRing(d, 16)
    ring.append(dev_bits(bits), torch.from_numpy(anc).cuda(), torch.from_numpy(roll).cuda())
    ora.append(bits, anc, roll)
    q = dev_bits(np.full((2, d), P1, np.uint16))
    qa = torch.tensor([7, 9], dtype=torch.int32, device="cuda")
    for m in (4, 8, 1):
        out = ring.query(q, qa, m=m).cpu()
        ref = ora.query(np.full((2, d), P1, np.uint16), [7, 9], m=m)
        assert out.slot.numpy().tolist() == ref.slot.tolist()
        assert np.array_equal(out.score.numpy(), ref.score)
        assert out.count.tolist() == ref.count.tolist()
        assert np.array_equal(out.rollout.numpy(), ref.rollout)
        assert np.array_equal(out.rollout_len.numpy(), ref.rollout_len)
    assert ring.query(q, qa, m=4).cpu().slot[0].tolist() == [5, 3, 4, 6]


@pytest.mark.parametrize("d,cap,n,vocab", [(256, 1000, 700, 5), (4096, 4096, 6000, 40),
                                            (512, 257, 2000, 3)])
def test_random_ring_with_wraparound(d, cap, n, vocab):
    cent, st, anc, roll = ring_inputs(n, d, vocab, seed=d + cap)
    ring, ora = B.Ring(d, cap), OracleRing(d, cap)
    for lo in range(0, n, 333):
        ring.append(st[lo:lo + 333].contiguous(), anc[lo:lo + 333].contiguous(),
                    roll[lo:lo + 333].contiguous())
        ora.append(W.to_bits(st[lo:lo + 333]), anc[lo:lo + 333].cpu().numpy(),
                   roll[lo:lo + 333].cpu().numpy())
    assert len(ring) == len(ora) == min(n, cap) and ring.total == n
    keys, a2, r2 = ring.read()
    assert np.array_equal(keys, ora.keys) and np.array_equal(a2, ora.anchors)
    assert np.array_equal(r2, ora.rollouts)
    g = torch.Generator(device="cuda").manual_seed(9)
    nq = 5
    q = (cent[:nq] + 0.3 * torch.randn(nq, d, generator=g, device="cuda")).to(torch.bfloat16)
    qa = torch.randint(0, vocab, (nq,), generator=g, device="cuda", dtype=torch.int32)
    for m, floor in ((4, 0.8), (32, 0.5), (2, -2.0)):
        out = ring.query(q, qa, m=m, floor=floor)
        check(out, ora, W.to_bits(q), qa.cpu().numpy(), m, floor)


def test_more_records_than_slots_in_one_append_and_reset():
    d, cap = 64, 50
    _, st, anc, roll = ring_inputs(180, d, 2, seed=3)
    ring, ora = B.Ring(d, cap), OracleRing(d, cap)
    ring.append(st, anc, roll)
    ora.append(W.to_bits(st), anc.cpu().numpy(), roll.cpu().numpy())
    for a, b in zip(ring.read(), (ora.keys, ora.anchors, ora.rollouts)):
        assert np.array_equal(a, b)
    ring.reset()
    assert len(ring) == 0
    out = ring.query(st[:1].contiguous(), anc[:1].contiguous()).cpu()
    assert out.count[0] == 0 and torch.all(out.slot == -1)
    bad = st[:1].clone(); bad[0, 3] = float("nan")
    ring.append(st[:10].contiguous(), anc[:10].contiguous(), roll[:10].contiguous())
    out = ring.query(bad, anc[:1].contiguous(), floor=-2.0).cpu()
    assert out.count[0] == 0                      # a NaN query finds nothing
    with pytest.raises(B.OilbirdError):
        ring.query(st[:1].contiguous(), anc[:1].contiguous(), m=33)


@pytest.mark.parametrize("d,cap,vocab,nq", [(256, 1000, 5, 1), (4096, 8192, 40, 1), (512, 257, 3, 4),
                                             (1024, 90000, 6, 1), (128, 40000, 4, 8)])
def test_steps_that_store_and_look_up_in_one_call(d, cap, vocab, nq):
    """oilbird_ring_step = append + query: the stored ring and every answer equal the oracle's
    after the same append; the query of a step looks for one of the step's own records (it
    must come back first); rings that wrap, steps of 0, 1, 64 and more records than blocks, and
    a lookup that needs more blocks than fit at once (its append then gets a launch of its own)."""
    ring, ora = B.Ring(d, cap), OracleRing(d, cap)
    cent, st, anc, roll = ring_inputs(cap + 1500, d, vocab, seed=7 + d + nq)
    # most of the ring first, in bulk; then steps across the wrap-around
    bulk = max(0, cap - 300)
    ring.append(st[:bulk].contiguous(), anc[:bulk].contiguous(), roll[:bulk].contiguous())
    ora.append(W.to_bits(st[:bulk]), anc[:bulk].cpu().numpy(), roll[:bulk].cpu().numpy())
    g = torch.Generator(device="cuda").manual_seed(5)
    pos = bulk
    for n in (64, 0, 1, 64, 333, 64, 7, 64, 700):
        s_, a_, r_ = st[pos:pos + n].contiguous(), anc[pos:pos + n].contiguous(), roll[pos:pos + n].contiguous()
        q = (cent[:nq] + 0.3 * torch.randn(nq, d, generator=g, device="cuda")).to(torch.bfloat16)
        qa = torch.randint(0, vocab, (nq,), generator=g, device="cuda", dtype=torch.int32)
        if n:
            q[0] = s_[n - 1]                      # a record stored by this very call
            qa[0] = a_[n - 1]
        out = ring.step(s_, a_, r_, q, qa, m=4, floor=0.5)
        ora.append(W.to_bits(s_), a_.cpu().numpy(), r_.cpu().numpy())
        pos += n
        assert len(ring) == len(ora) and ring.total == pos
        check(out, ora, W.to_bits(q), qa.cpu().numpy(), 4, 0.5)
        if n:
            assert int(out.slot[0, 0]) == (pos - 1) % cap
    keys, a2, r2 = ring.read()
    assert np.array_equal(keys, ora.keys) and np.array_equal(a2, ora.anchors)
    assert np.array_equal(r2, ora.rollouts)
    # a plain lookup afterwards sees the same ring
    q = (cent[:nq] + 0.3 * torch.randn(nq, d, generator=g, device="cuda")).to(torch.bfloat16)
    qa = torch.randint(0, vocab, (nq,), generator=g, device="cuda", dtype=torch.int32)
    check(ring.query(q, qa, m=8, floor=-2.0), ora, W.to_bits(q), qa.cpu().numpy(), 8, -2.0)

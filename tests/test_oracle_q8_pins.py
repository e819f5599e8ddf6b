"""Pins for the oracle's 8-bit (E4M3) store, against things other than the oracle:
PyTorch's own float8_e4m3fn conversion (an independent implementation of the format), the
format's published constants, a closed form on +-1 pools, the mathematical error bound of
the quantiser, and a numpy restatement of the score that decodes with PyTorch."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OraclePool


def torch_decode(codes: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(codes, dtype=np.uint8)).view(torch.float8_e4m3fn)
    return t.to(torch.float32).numpy().astype(np.float64)


def bits(x: np.ndarray) -> np.ndarray:
    return oracle.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_decode_table_matches_pytorch_and_format_constants():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch_decode(codes)
    for c in range(256):
        v = oracle.e4m3_decode(c)
        if c in (0x7F, 0xFF):
            assert np.isnan(v) and np.isnan(ref[c])
        else:
            assert v == ref[c], (c, v, ref[c])
    # constants of the format: largest finite 448, smallest normal 2^-6, smallest
    # subnormal 2^-9, one, negative zero
    assert oracle.e4m3_decode(0x7E) == 448.0
    assert oracle.e4m3_decode(0x08) == 2.0 ** -6
    assert oracle.e4m3_decode(0x01) == 2.0 ** -9
    assert oracle.e4m3_decode(0x38) == 1.0
    assert oracle.e4m3_decode(0x80) == 0.0 and np.signbit(oracle.e4m3_decode(0x80))
    pos = [oracle.e4m3_decode(c) for c in range(0x7F)]
    assert all(a < b for a, b in zip(pos, pos[1:]))          # monotone in the code


def test_encode_matches_pytorch_round_to_nearest_even():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.uniform(-448, 448, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 2000),
        np.array([0.0, 1.0, 1.0625, 1.1875, 2.0 ** -10, 2.0 ** -9, 3 * 2.0 ** -10, 447.9, 448.0,
                  -448.0, 15.5, 0.0175])]).astype(np.float32)
    ref = torch.from_numpy(xs).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for x, r in zip(xs, ref):
        c = oracle.e4m3_encode(float(x))
        if float(x) == 0.0:
            assert c & 0x7F == 0
        else:
            assert c == int(r), (float(x), c, int(r))
    # every finite code is a fixed point; midpoints go to the even code
    for c in list(range(0x7F)) + list(range(0x80, 0xFF)):
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) & 0x7F == c & 0x7F
    for c in range(0x7E):
        mid = 0.5 * (oracle.e4m3_decode(c) + oracle.e4m3_decode(c + 1))
        assert oracle.e4m3_encode(mid) == (c if c % 2 == 0 else c + 1)
    # saturation, not NaN, above the largest finite value
    assert oracle.e4m3_encode(1e6) == 0x7E and oracle.e4m3_encode(-465.0) == 0xFE


@pytest.mark.parametrize("d", [16, 64, 1024])
def test_quantise_row_properties_and_error_bound(d):
    rng = np.random.default_rng(d)
    x = bits(rng.normal(0, 2.0, d) * (rng.random(d) < 0.7))          # some exact zeros
    codes, scale, ok = oracle.quantize_e4m3(x)
    assert ok
    xv = oracle.bf16_bits_to_f32(x).astype(np.float64)
    v = xv / np.sqrt(np.sum(xv * xv))
    dec = torch_decode(codes)
    assert np.max(np.abs(dec)) == 448.0                              # the row's peak maps to +-448
    assert abs(scale * 448.0 - np.max(np.abs(v))) <= 2.0 ** -23 * np.max(np.abs(v))
    # nearest-value property: half a unit in the last place of each element
    err = np.abs(v - scale * dec)
    ulp = np.where(np.abs(dec) >= 2.0 ** -6, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(dec), 1e-300))) - 3),
                   2.0 ** -9)
    assert np.all(err <= scale * ulp * 0.5 * (1 + 1e-6) + 1e-300)
    assert np.all(codes[xv == 0] & 0x7F == 0)


def test_unusable_rows_are_stored_as_zero():
    d = 32
    for row in (np.zeros(d, np.float32), np.r_[np.inf, np.ones(d - 1)].astype(np.float32),
                np.r_[np.nan, np.ones(d - 1)].astype(np.float32)):
        codes, scale, ok = oracle.quantize_e4m3(bits(row))
        assert not ok and scale == 0.0 and not codes.any()
    p = OraclePool(d, "e4m3")
    p.append(bits(np.stack([np.zeros(d), np.ones(d)])), np.array([1, 2]))
    r = p.query(bits(np.ones((1, d))), oracle.QueryParams(k=2, theta=-2.0, depth_mode=oracle.DEPTH_FIXED,
                                                          cont_len=1), want_all_scores=True)
    assert r.all_scores[0, 0] == 0.0
    assert abs(r.all_scores[0, 1] - 1.0) < 2.0 ** -8      # the bf16 query carries the only rounding


@pytest.mark.parametrize("d", [16, 64, 256, 1024])
def test_closed_form_on_plus_minus_one_pools(d):
    # rows and query in {+-1}^d: every normalised entry is +-2^-m (d a power of 4), the row's
    # peak is every entry, so every code is +-448 and s = (1 - 2 Hamming / d) * (scale*448*2^m)
    rng = np.random.default_rng(d)
    n = 40
    rows = rng.choice([-1.0, 1.0], size=(n, d))
    q = rng.choice([-1.0, 1.0], size=(1, d))
    rows[7] = q[0]                                   # an exact copy
    rows[9] = q[0]                                   # and a tie with it
    rows[11] = -q[0]
    p = OraclePool(d, "e4m3")
    p.append(bits(rows), np.arange(n, dtype=np.int32))
    assert set(np.unique(p.codes)) <= {0x7E, 0xFE}
    m = int(round(np.log2(d) / 2))
    assert 4 ** m == d
    scale = float(np.float32((2.0 ** -m) / 448.0))
    assert np.all(p.scales == np.float32(scale))
    ham = np.sum(rows != q, axis=1)
    expect = ((1.0 - 2.0 * ham / d) * (scale * 448.0 * 2.0 ** m)).astype(np.float32)
    r = p.query(bits(q), oracle.QueryParams(k=3, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=1),
                want_all_scores=True)
    assert np.array_equal(r.all_scores[0], expect)
    assert r.idx[0].tolist()[:2] == [7, 9]           # equal scores: lower position first
    assert r.all_scores[0, 11] == -expect[7]


def test_score_equals_numpy_restatement_with_pytorch_decode():
    rng = np.random.default_rng(5)
    d, n = 96, 50
    rows = bits(rng.normal(0, 1, (n, d)))
    q = bits(rng.normal(0, 1, (2, d)))
    p = OraclePool(d, "e4m3")
    p.append(rows, np.arange(n, dtype=np.int32))
    r = p.query(q, oracle.QueryParams(k=5, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=2),
                want_all_scores=True)
    dec = torch_decode(p.codes)                                    # [n,d], decoded by PyTorch
    for i in range(2):
        qn, _ = oracle.normalize_bf16(q[i])
        qv = oracle.bf16_bits_to_f32(qn).astype(np.float64)
        s = (dec @ qv) * p.scales.astype(np.float64)
        assert np.allclose(r.all_scores[i], s.astype(np.float32), rtol=0, atol=1e-7)
        order = sorted(range(n), key=lambda j: (-r.all_scores[i][j], j))
        assert r.idx[i].tolist() == order[:5]


def test_quantisation_error_of_a_score_is_within_its_bound():
    # |s8 - s16| <= |q| * |v - v8| + (bf16 rounding of the 16-bit key), with
    # |v - v8| <= 2^-4 |v| + sqrt(d) * scale * 2^-10   (normals: half an ulp of a 3-bit
    # mantissa; subnormals: half the subnormal spacing)
    rng = np.random.default_rng(9)
    d, n = 512, 300
    cent = rng.normal(0, 1, (8, d))
    rows = bits(cent[rng.integers(0, 8, n)] + 0.2 * rng.normal(0, 1, (n, d)))
    q = bits(cent[:4] + 0.2 * rng.normal(0, 1, (4, d)))
    p8, p16 = OraclePool(d, "e4m3"), OraclePool(d)
    tok = np.arange(n, dtype=np.int32)
    p8.append(rows, tok)
    p16.append(rows, tok)
    pr = oracle.QueryParams(k=8, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=1)
    a = p8.query(q, pr, want_all_scores=True).all_scores
    b = p16.query(q, pr, want_all_scores=True).all_scores
    bound = 2.0 ** -4 + np.sqrt(d) * p8.scales.max() * 2.0 ** -10 + 2.0 ** -8
    assert np.max(np.abs(a - b)) <= bound
    assert np.max(np.abs(a - b)) < 0.02              # and in practice far below it


# ---------------------------------------------------------------- eviction ----
# Oldest-first eviction by whole traces must leave exactly the pool that the remaining
# traces alone would have built (the append and query paths are pinned elsewhere).

def _traces(rng, d, lens):
    return [(bits(rng.normal(0, 1, (n, d))), rng.integers(0, 1000, n).astype(np.int32), 100 + i)
            for i, n in enumerate(lens)]


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
@pytest.mark.parametrize("drop", [0, 1, 3, 6, 9])
def test_evict_oldest_equals_rebuild_from_remaining_traces(fmt, drop):
    rng = np.random.default_rng(31)
    d = 32
    lens = [5, 1, 17, 4, 9, 2]
    tr = _traces(rng, d, lens)
    a, b = OraclePool(d, fmt), OraclePool(d, fmt)
    for st, tk, tag in tr:
        a.append(st, tk, tag=tag)
    dropped = a.evict_oldest(drop)
    keep = tr[min(drop, len(tr)):]
    for st, tk, tag in keep:
        b.append(st, tk, tag=tag)
    assert dropped == sum(lens[:min(drop, len(lens))])
    assert len(a) == len(b) and a.num_traces == b.num_traces
    if fmt == "bf16":
        assert np.array_equal(a.keys, b.keys)
    else:
        assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)
    assert np.array_equal(a.tokens, b.tokens) and np.array_equal(a.trace_ids, b.trace_ids)
    assert np.array_equal(a.trace_starts, b.trace_starts)
    assert np.array_equal(a.trace_ends, b.trace_ends) and np.array_equal(a.trace_tags, b.trace_tags)
    if len(a):
        q = bits(rng.normal(0, 1, (2, d)))
        pr = oracle.QueryParams(k=4, theta=-2.0, depth_mode=oracle.DEPTH_FIXED, cont_len=6)
        ra, rb = a.query(q, pr), b.query(q, pr)
        for f in ("idx", "score", "fired", "cont_len", "cont_tok"):
            assert np.array_equal(getattr(ra, f), getattr(rb, f))
    # the pool keeps working: an append after the eviction extends / opens traces as usual
    st, tk, tag = _traces(rng, d, [3])[0]
    a.append(st, tk, tag=7, new_trace=False)
    b.append(st, tk, tag=7, new_trace=False)
    assert np.array_equal(a.trace_ends, b.trace_ends) and np.array_equal(a.tokens, b.tokens)


def test_evicted_rows_by_hand():
    d = 16
    p = OraclePool(d)
    e = np.eye(d, dtype=np.float32)
    p.append(bits(e[0:2]), np.array([10, 11]), tag=1)        # rows 0,1
    p.append(bits(e[2:5]), np.array([20, 21, 22]), tag=2)    # rows 2,3,4
    p.append(bits(e[5:6]), np.array([30]), tag=3)            # row 5
    assert p.evict_oldest(1) == 2
    assert p.tokens.tolist() == [20, 21, 22, 30]
    assert p.trace_ids.tolist() == [0, 0, 0, 1]
    assert p.trace_starts.tolist() == [0, 3] and p.trace_ends.tolist() == [3, 4]
    assert p.trace_tags.tolist() == [2, 3]
    r = p.query(bits(e[2:3]), oracle.QueryParams(k=1, theta=0.5, offset=1, depth_mode=oracle.DEPTH_FIXED,
                                                 cont_len=4))
    assert r.idx[0, 0] == 0 and r.cont_tok[0, 0].tolist() == [21, 22, -1, -1]   # clipped at the trace end

"""Boundary hardening on the GPU: what the library refuses before it launches anything, the
give-up path of its bounded device-side waits, and the guard zones the other GPU tests run
under.  Nothing here faults, traps or hangs a GPU: refusals are host-side, and the wait that
runs out is a bounded wait on something that never happens, which returns by itself.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import OraclePool
from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both

pytestmark = pytest.mark.gpu


def fixed(k, L, theta=-2.0, **kw):
    return B.QueryParams(k=k, theta=theta, depth_mode=B.DEPTH_FIXED, cont_len=L, **kw)


def odd_view(t: torch.Tensor) -> torch.Tensor:
    """The same values at an address two bytes (bf16) or four bytes (int32) further on:
    contiguous, right dtype and shape, but no longer on a 16-byte boundary."""
    buf = torch.empty(t.numel() + 8, dtype=t.dtype, device=t.device)
    v = buf[1:1 + t.numel()].view(t.shape)
    v.copy_(t)
    assert v.is_contiguous() and v.data_ptr() % 16 != 0
    return v


def test_misaligned_pointers_are_refused_before_any_launch():
    d = 256
    g = torch.Generator(device="cuda").manual_seed(5)
    st = torch.randn(40, d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(40, dtype=torch.int32, device="cuda")
    pool = B.Pool(d, 200)
    pool.append(st, tk, tag=1)
    launches, rows, traces = pool.launch_count, len(pool), pool.num_traces
    q = st[3:5].contiguous()
    for call in (lambda: pool.append(odd_view(st), tk, tag=2),
                 lambda: pool.query(odd_view(q), fixed(4, 4)),
                 lambda: pool.step(odd_view(st[:8].contiguous()), tk[:8].contiguous(), q, fixed(4, 4)),
                 lambda: pool.step(st[:8].contiguous(), tk[:8].contiguous(), odd_view(q), fixed(4, 4))):
        with pytest.raises(B.OilbirdError) as e:
            call()
        assert e.value.code == B.EINVAL and "aligned" in str(e.value)
    assert (pool.launch_count, len(pool), pool.num_traces) == (launches, rows, traces)
    # the entry point that allocates nothing checks the same
    keys, tok, tid = pool.read_rows()
    keys_t = torch.from_numpy(keys.view(np.int16)).view(torch.bfloat16).cuda()
    end = torch.tensor([40], dtype=torch.int32, device="cuda")
    tid_t = torch.from_numpy(tid).cuda()
    for kk, qq in ((odd_view(keys_t), q), (keys_t, odd_view(q))):
        with pytest.raises(B.OilbirdError) as e:
            B.query_static(kk, tk, tid_t, end, qq, fixed(4, 4))
        assert e.value.code == B.EINVAL and "misaligned" in str(e.value)
    # and the pool still answers
    out = pool.query(q, fixed(4, 4)).cpu()
    assert out.idx[:, 0].tolist() == [3, 4]


@pytest.mark.parametrize("fmt,path,d,k", [("e4m3", B.PATH_MMA, 384, 8),       # 8-bit warp-level scan: d a multiple of 256
                                          ("bf16", B.PATH_MMA, 200, 8),       # d not a multiple of 128
                                          ("bf16", B.PATH_MMA, 256, 100)])    # k beyond the warp-level scan
def test_a_refused_step_appends_nothing(fmt, path, d, k):
    g = torch.Generator(device="cuda").manual_seed(6)
    pool = B.Pool(d, 400, key_format=fmt, max_k=128)
    st = torch.randn(64, d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(64, dtype=torch.int32, device="cuda")
    pool.append(st, tk, tag=1)
    before = (len(pool), pool.num_traces, pool.launch_count)
    q = st[:4].contiguous()
    for n in (8, 100):                       # a step that would fuse its append, and one that would not
        with pytest.raises(B.OilbirdError) as e:
            pool.step(st[:n].contiguous() if n <= 64 else torch.cat([st, st])[:n].contiguous(),
                      torch.arange(n, dtype=torch.int32, device="cuda"), q,
                      fixed(k, 4, path=path), tag=2)
        assert e.value.code == B.EINVAL
        assert (len(pool), pool.num_traces, pool.launch_count) == before
    st_, en_, _ = pool.traces()
    assert st_.tolist() == [0] and en_.tolist() == [64]


def test_a_wait_that_runs_out_is_reported_cleared_and_leaves_the_pool_usable():
    w = W.C1.scaled(n_rows=2048, nq=2, seed=9)
    pool, ora = fill_both(w, spare_rows=64)
    assert pool.status() == B.OK
    pool.set_wait_limit(1_000_000)           # one millisecond
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    pool.stall_selftest()                    # a counter nobody advances, a barrier nobody arrives at
    t1.record()
    assert pool.status() == B.ESTALL         # synchronises: the kernel has returned by itself
    assert pool.stats()["stalled"] == 1
    assert 0.5 < t0.elapsed_time(t1) < 500.0   # gave up after about the limit, not after seconds
    # sticky until reset, which clears the counters but keeps the rows' owner honest: the pool
    # is emptied, so it is refilled before it is asked again
    assert pool.status() == B.ESTALL
    pool.reset()
    assert pool.status() == B.OK and pool.stats()["stalled"] == 0 and len(pool) == 0
    pool.set_wait_limit(0)                   # back to the default (two seconds)
    for st, tk, tag in w.traces("cuda"):
        pool.append(st, tk, tag=tag)
    q, _ = w.queries("cuda")
    for path in (B.PATH_GEMV, B.PATH_TENSOR, B.PATH_MMA):
        pr = fixed(w.k, w.cont_len, path=path)
        check_query(pool.query(q, pr), ora, W.to_bits(q), pr)
    # the fused step, whose scanning warps do wait for the appending ones, still completes
    g = torch.Generator(device="cuda").manual_seed(1)
    st = torch.randn(8, w.d, generator=g, device="cuda").to(torch.bfloat16)
    tk = torch.arange(8, dtype=torch.int32, device="cuda")
    out = pool.step(st, tk, st[6:7].contiguous(), fixed(4, 4), tag=77)
    assert int(out.idx[0, 0]) == len(pool) - 2
    assert pool.status() == B.OK


def test_guard_zones_catch_a_write_behind_an_array():
    d, cap = 64, 128
    pool = B.Pool(d, cap, use_torch_arena=True, debug_guards=True)
    g = torch.Generator(device="cuda").manual_seed(3)
    st = torch.randn(cap, d, generator=g, device="cuda").to(torch.bfloat16)
    pool.append(st, torch.arange(cap, dtype=torch.int32, device="cuda"), tag=1)   # a full pool
    pool.query(st[:16].contiguous(), fixed(8, 4))
    pool.check_guards()                                   # untouched after a full append + query
    # the first byte behind the keys (the arena starts on a 256-byte boundary, keys first)
    assert pool._arena.data_ptr() % 256 == 0
    pool._arena[cap * d * 2] = 0
    with pytest.raises(B.OilbirdError) as e:
        pool.check_guards()
    assert e.value.code == B.EGUARD and "keys" in str(e.value)
    pool._arena[cap * d * 2] = 0xA5                        # put it back: close() checks again
    pool.check_guards()
    plain = B.Pool(d, cap, debug_guards=False)
    with pytest.raises(B.OilbirdError) as e:
        plain.check_guards()
    assert e.value.code == B.EINVAL


def test_tree_merge_ignores_parents_that_name_no_node():
    # parent entries are caller memory: out-of-range values detach their node, nothing else
    t_tok = torch.full((2, 60), -1, dtype=torch.int32, device="cuda")
    t_par = torch.full((2, 60), -1, dtype=torch.int32, device="cuda")
    t_tok[:, :4] = torch.tensor([7, 1, 2, 3], dtype=torch.int32)
    t_par[0, :4] = torch.tensor([-1, 0, 1, 2], dtype=torch.int32)            # a sound chain
    t_par[1, :4] = torch.tensor([55, 0, 1_000_000, -9], dtype=torch.int32)   # junk at 0, 2, 3
    n = torch.tensor([4, 4], dtype=torch.int32, device="cuda")
    sem = torch.tensor([[[1, 2, 3, 4]], [[1, 2, 3, 4]]], dtype=torch.int32, device="cuda")
    slen = torch.tensor([[4], [4]], dtype=torch.int32, device="cuda")
    mo = B.merge_chains(t_tok, t_par, n, sem, slen)
    torch.cuda.synchronize()
    assert mo.n_nodes.tolist() == [5, 7]          # request 1: only node 1 hangs off the root
    assert mo.tree_parent[1, :7].tolist() == [-1, 0, -1, -1, 1, 4, 5]
    assert mo.bought[:, 0].tolist() == [1, 3] and mo.walked[:, 0].tolist() == [3, 1]
    assert mo.mask[1, 2].item() == 1 << 2 and mo.depth[1, 2].item() == 0


@pytest.mark.gpu
def test_tree_merge_returns_on_parents_that_form_a_cycle():
    # nodes 2 and 3 name each other: neither hangs off the root, so neither is walked, and
    # the call still returns with the sound part of the tree extended
    t_tok = torch.full((1, 60), -1, dtype=torch.int32, device="cuda")
    t_par = torch.full((1, 60), -1, dtype=torch.int32, device="cuda")
    t_tok[0, :4] = torch.tensor([7, 1, 2, 3], dtype=torch.int32)
    t_par[0, :4] = torch.tensor([-1, 0, 3, 2], dtype=torch.int32)
    n = torch.tensor([4], dtype=torch.int32, device="cuda")
    sem = torch.tensor([[[1, 2, 3, 4]]], dtype=torch.int32, device="cuda")
    slen = torch.tensor([[4]], dtype=torch.int32, device="cuda")
    mo = B.merge_chains(t_tok, t_par, n, sem, slen)
    torch.cuda.synchronize()
    assert mo.n_nodes.tolist() == [7]
    assert mo.tree_parent[0, :7].tolist() == [-1, 0, 3, 2, 1, 4, 5]
    assert mo.bought[0, 0].item() == 3 and mo.walked[0, 0].item() == 1
    assert mo.depth[0, 4:7].tolist() == [2, 3, 4]
    assert mo.mask[0, 6].item() == (1 << 6) | (1 << 5) | (1 << 4) | (1 << 1) | 1

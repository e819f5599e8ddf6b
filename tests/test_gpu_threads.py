"""Two pools driven by two host threads on two streams at the same time.

The boundary promises one host thread per pool at a time, and says nothing is shared between
pools: the per-thread error text, the per-call launch policy and the per-pool caches are what
make that true.  Each thread checks every answer against its own oracle; the two pools use
different scan paths so that different kernels overlap on the device."""
import threading

import pytest
import torch

from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import workloads as W
from parity import check_query, fill_both

pytestmark = pytest.mark.gpu


def test_two_pools_two_threads_two_streams():
    specs = [dict(n_rows=40000, d=256, nq=1, k=8, seed=91, paths=(B.PATH_GEMV, B.PATH_TENSOR)),
             dict(n_rows=77000, d=128, nq=130, k=16, seed=92, paths=(B.PATH_TENSOR,)),
             dict(n_rows=9000, d=512, nq=8, k=8, seed=93, paths=(B.PATH_MMA, B.PATH_GEMV))]
    jobs = []
    for sp in specs:
        w = W.C1.scaled(n_rows=sp["n_rows"], d=sp["d"], nq=sp["nq"], k=sp["k"], cont_len=4,
                        rows_per_trace=500, seed=sp["seed"])
        pool, ora = fill_both(w, max_nq=256, spare_rows=256)
        jobs.append((w, pool, ora, sp["paths"]))
    torch.cuda.synchronize()
    errors = []
    start = threading.Barrier(len(jobs))

    def run(w, pool, ora, paths):
        try:
            stream = torch.cuda.Stream()
            start.wait()
            with torch.cuda.stream(stream):
                for it in range(6):
                    q, _ = w.queries("cuda", step=it)
                    for path in paths:
                        pr = B.QueryParams(k=w.k, theta=-2.0, depth_mode=B.DEPTH_FIXED, cont_len=4,
                                           path=path)
                        out = pool.query(q, pr, stream=stream)
                        stream.synchronize()
                        check_query(out, ora, W.to_bits(q), pr)
                    # a refused call in between: its text belongs to this thread
                    odd = torch.zeros(w.d + 8, dtype=torch.bfloat16, device="cuda")[1:1 + w.d].view(1, w.d)
                    with pytest.raises(B.OilbirdError) as e:
                        pool.query(odd, pr, stream=stream)
                    assert e.value.code == B.EINVAL and "aligned" in str(e.value)
                    if it % 2 == 0:              # and the pool grows while the others scan
                        g = torch.Generator(device="cuda").manual_seed(1000 * w.seed + it)
                        st = torch.randn(64, w.d, generator=g, device="cuda").to(torch.bfloat16)
                        tk = torch.randint(0, 1000, (64,), generator=g, device="cuda", dtype=torch.int32)
                        pool.append(st, tk, tag=5000 + it, stream=stream)
                        stream.synchronize()
                        ora.append(W.to_bits(st), tk.cpu().numpy(), tag=5000 + it)
                stream.synchronize()
                assert pool.stats(stream=stream)["stalled"] == 0
        except BaseException as ex:              # noqa: BLE001 - reported in the main thread
            errors.append(ex)
            try:
                start.abort()
            except Exception:
                pass

    threads = [threading.Thread(target=run, args=j) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    if errors:
        raise errors[0]

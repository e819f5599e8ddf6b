"""Seeded synthetic pools and queries for the five benchmark configurations.

This module only draws random numbers and lays them out; it contains none of the
retrieval arithmetic (no normalisation, no scoring, no selection).  Both the CUDA
library and the CPU checker are fed the arrays produced here: a workload is
materialised once on one device and the *same* bf16 bit patterns are handed to
both sides (torch's CPU and CUDA generators give different streams for the same
seed, so a workload's contents depend on the device it was drawn on).

The pools stand in for the hidden states of the paper's tool-calling, code and
chat traffic, which cannot be reproduced here: raw states are bf16, one row per
generated token, grouped into traces (one per finished request).  Shapes follow
the paper's sizes (8 KB per token at 8B width, i.e. d=4096 bf16; 33k to 317k rows
per benchmark store) and extend to serving scale.

Kinds of pool
  clustered   rows = centroid[c] + sigma * N(0,1): many near-duplicates per query
  template    tool-calling shape: requests replay one of a few hundred templates
              and differ only at a few "slot" positions holding freshly minted ids
  separated   unclustered N(0,1) background plus a few planted neighbours of each
              query at well separated similarities (parity-only variant)
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from functools import lru_cache

import torch

BASE_SEED = 0x0B11B12D


def _gen(device, *parts: int) -> torch.Generator:
    seed = BASE_SEED
    for p in parts:
        seed = (seed * 1000003 + int(p) + 0x9E3779B9) % (2**62)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str                 # "clustered" | "template" | "separated"
    d: int
    n_rows: int
    rows_per_trace: int
    vocab: int
    nq: int
    k: int
    cont_len: int
    seed: int
    n_centroids: int = 0
    sigma: float = 0.2
    # template pools
    n_templates: int = 0
    slot_frac: float = 0.05
    sigma_slot: float = 0.5
    # separated pools
    n_planted: int = 0
    # a planted query: pool row + this noise (clustered pools)
    query_noise: float = 0.05

    # ---- structure -----------------------------------------------------------
    @property
    def num_traces(self) -> int:
        return (self.n_rows + self.rows_per_trace - 1) // self.rows_per_trace

    def trace_rows(self, t: int) -> int:
        return min(self.rows_per_trace, self.n_rows - t * self.rows_per_trace)

    def trace_tag(self, t: int) -> int:
        if self.kind == "template":
            return 1 + (t % self.n_templates)     # same "prompt" = same template
        return 1 + t

    def key_bytes(self, n_rows: int | None = None) -> int:
        return (self.n_rows if n_rows is None else n_rows) * self.d * 2

    # ---- centroids -----------------------------------------------------------
    def _centroids(self, device) -> torch.Tensor:
        g = _gen(device, self.seed, 1)
        return torch.randn(self.n_centroids, self.d, generator=g, device=device,
                           dtype=torch.float32)

    def _template(self, m: int, device):
        """Centroids [P,d], tokens [P] and slot mask [P] of template m."""
        P = self.rows_per_trace
        g = _gen(device, self.seed, 2, m)
        cent = torch.randn(P, self.d, generator=g, device=device, dtype=torch.float32)
        toks = torch.randint(0, self.vocab, (P,), generator=g, device=device, dtype=torch.int32)
        n_slots = max(1, int(round(self.slot_frac * P)))
        perm = torch.randperm(P, generator=g, device=device)
        slot = torch.zeros(P, dtype=torch.bool, device=device)
        slot[perm[:n_slots]] = True
        return cent, toks, slot

    # ---- pool contents -------------------------------------------------------
    def trace(self, t: int, device="cpu", centroids: torch.Tensor | None = None):
        """Raw states bf16 [n,d], tokens int32 [n] and the tag of trace t."""
        n = self.trace_rows(t)
        g = _gen(device, self.seed, 3, t)
        if self.kind == "clustered":
            C = self._centroids(device) if centroids is None else centroids
            assign = torch.randint(0, self.n_centroids, (n,), generator=g, device=device)
            noise = torch.randn(n, self.d, generator=g, device=device, dtype=torch.float32)
            states = C[assign] + self.sigma * noise
            toks = torch.randint(0, self.vocab, (n,), generator=g, device=device,
                                 dtype=torch.int32)
        elif self.kind == "template":
            cent, ttoks, slot = self._template(t % self.n_templates, device)
            noise = torch.randn(n, self.d, generator=g, device=device, dtype=torch.float32)
            sig = torch.where(slot[:n], self.sigma_slot, self.sigma).unsqueeze(1)
            states = cent[:n] + sig * noise
            fresh = torch.randint(0, self.vocab, (n,), generator=g, device=device,
                                  dtype=torch.int32)
            toks = torch.where(slot[:n], fresh, ttoks[:n])
        elif self.kind == "separated":
            states = torch.randn(n, self.d, generator=g, device=device, dtype=torch.float32)
            toks = torch.randint(0, self.vocab, (n,), generator=g, device=device,
                                 dtype=torch.int32)
            # planted neighbours overwrite background rows that fall in this trace
            q_raw, _, sig, where = _separated_plan(self)
            lo = t * self.rows_per_trace
            for r in range(lo, lo + n):
                if r in where:
                    qi, j = where[r]
                    gp = _gen(device, self.seed, 5, qi, j)
                    nz = torch.randn(self.d, generator=gp, device=device, dtype=torch.float32)
                    states[r - lo] = q_raw[qi].to(device) + sig[j] * nz
        else:
            raise ValueError(self.kind)
        return states.to(torch.bfloat16), toks, self.trace_tag(t)

    def trace_assign(self, t: int, device="cpu") -> torch.Tensor:
        """Clustered pools: the centroid each row of trace t was drawn around (the labels
        only, without materialising the states: the trace generator's first draw)."""
        if self.kind != "clustered":
            raise ValueError("only clustered pools have centroid labels")
        g = _gen(device, self.seed, 3, t)
        return torch.randint(0, self.n_centroids, (self.trace_rows(t),), generator=g, device=device)

    def traces(self, device="cpu"):
        C = self._centroids(device) if self.kind == "clustered" else None
        for t in range(self.num_traces):
            yield self.trace(t, device, C)

    # ---- queries -------------------------------------------------------------
    def queries(self, device="cpu", nq: int | None = None, step: int = 0):
        """Raw query states bf16 [nq,d] plus a dict describing what was planted.

        clustered: query 0 is a pool row plus small noise (it must retrieve that
        row first); the rest are fresh draws around random centroids.
        template:  new instances of random (template, position) pairs; the rows
        holding the same pair in earlier traces are returned as ``planted_rows``.
        separated: the queries whose neighbours were planted in the pool.
        """
        nq = self.nq if nq is None else nq
        g = _gen(device, self.seed, 6, step)
        meta: dict = {}
        if self.kind == "clustered":
            C = self._centroids(device)
            c = torch.randint(0, self.n_centroids, (nq,), generator=g, device=device)
            noise = torch.randn(nq, self.d, generator=g, device=device, dtype=torch.float32)
            q = C[c] + self.sigma * noise
            gi = _gen("cpu", self.seed, 7, step)
            row = int(torch.randint(0, self.n_rows, (1,), generator=gi))
            t, r = divmod(row, self.rows_per_trace)
            st, _, _ = self.trace(t, device, C)
            q[0] = st[r].float() + self.query_noise * noise[0]
            meta["planted_row"] = row
            cl = c.tolist()
            cl[0] = int(self.trace_assign(t, device)[r])
            meta["centroid"] = cl              # the centroid each query was drawn around
        elif self.kind == "template":
            gi = _gen("cpu", self.seed, 7, step)
            P = self.rows_per_trace
            tm = torch.randint(0, self.n_templates, (nq,), generator=gi).tolist()
            pos = torch.randint(0, max(1, P - self.cont_len - 2), (nq,), generator=gi).tolist()
            # force one query onto a slot position and one right after a slot
            _, _, slot0 = self._template(tm[0], device)
            slots = torch.nonzero(slot0[: P - self.cont_len - 3]).flatten().tolist()
            if slots:
                pos[0] = slots[0]
            if nq > 1:
                _, _, slot1 = self._template(tm[1], device)
                slots1 = torch.nonzero(slot1[: P - self.cont_len - 3]).flatten().tolist()
                if slots1:
                    pos[1] = slots1[0] + 1
            qs, planted, conts, is_slot = [], [], [], []
            for i in range(nq):
                cent, ttoks, slot = self._template(tm[i], device)
                sg = self.sigma_slot if bool(slot[pos[i]]) else self.sigma
                nz = torch.randn(self.d, generator=g, device=device, dtype=torch.float32)
                qs.append(cent[pos[i]] + sg * nz)
                rows = [t * P + pos[i] for t in range(self.num_traces)
                        if t % self.n_templates == tm[i] and pos[i] < self.trace_rows(t)]
                planted.append(rows)
                conts.append((ttoks.cpu(), slot.cpu()))
                is_slot.append(bool(slot[pos[i]]))
            q = torch.stack(qs)
            meta.update(template=tm, pos=pos, planted_rows=planted, template_tokens=conts,
                        is_slot=is_slot)
        elif self.kind == "separated":
            q_raw, rows, sig, _ = _separated_plan(self)
            q = q_raw[:nq].to(device)
            meta.update(planted_rows=rows[:nq], planted_sigma=sig)
        else:
            raise ValueError(self.kind)
        return q.to(torch.bfloat16), meta

    def scaled(self, **kw) -> "Workload":
        """The same recipe at other sizes (CPU-sized test cases, sweeps)."""
        return replace(self, **kw)

    def separated(self) -> "Workload":
        """Parity-only variant: same sizes, unclustered background, k+4 planted rows."""
        return replace(self, name=self.name + "S", kind="separated", n_planted=self.k + 4)


@lru_cache(maxsize=16)
def _separated_plan(w: Workload):
    """Queries (drawn on the CPU), planted row numbers, their noise levels, row -> (q, j)."""
    g = _gen("cpu", w.seed, 4)
    q_raw = torch.randn(w.nq, w.d, generator=g, dtype=torch.float32)
    rows = torch.randperm(w.n_rows, generator=g)[: w.nq * w.n_planted]
    rows = rows.reshape(w.nq, w.n_planted).tolist()
    sig = [0.05 * (j + 1.0) for j in range(w.n_planted)]
    where = {r: (qi, j) for qi, rr in enumerate(rows) for j, r in enumerate(rr)}
    return q_raw, rows, sig, where


# The five benchmark configurations (sizes as the benchmark definition gives them).
C1 = Workload("C1", "clustered", d=256, n_rows=4096, rows_per_trace=256, vocab=32000,
              nq=1, k=8, cont_len=8, seed=1, n_centroids=64, sigma=0.3)
C2 = Workload("C2", "clustered", d=4096, n_rows=65536, rows_per_trace=512, vocab=128256,
              nq=1, k=16, cont_len=16, seed=2, n_centroids=512, sigma=0.2)
C3 = Workload("C3", "template", d=5120, n_rows=262144, rows_per_trace=300, vocab=152064,
              nq=8, k=8, cont_len=32, seed=3, n_templates=200, sigma=0.1, sigma_slot=0.5)
C4 = Workload("C4", "clustered", d=4096, n_rows=1048576, rows_per_trace=1024, vocab=128256,
              nq=64, k=32, cont_len=16, seed=4, n_centroids=4096, sigma=0.2)
# C5 starts at 2^20 rows and grows to 2^21 by 256-row appends; n_rows is the final size.
C5 = Workload("C5", "clustered", d=8192, n_rows=2097152, rows_per_trace=256, vocab=128256,
              nq=64, k=64, cont_len=16, seed=5, n_centroids=8192, sigma=0.2)
C5_START_ROWS = 1048576
C5_NQ_SWEEP = (1, 8, 64, 256)

CONFIGS = {w.name: w for w in (C1, C2, C3, C4, C5)}


def to_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns on the host (for the CPU checker)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")

"""One logical pool sharded by whole traces over the GPUs of a process group.

Every rank owns a local :class:`~paper_2608_03839_b200.binding.Pool` holding the traces that
were routed to it, at caller-assigned global positions.  A query is answered by all ranks
together: local query (no theta gate) -> local rows to global positions -> ONE all-gather of
the ranks' records -> merge kernel (global top-k, theta on the merged best).  The result is
replicated on every rank and equals what a single pool with all rows would return.

The record of a rank (its nq*k neighbours with scores, lengths, continuations and global
positions) is one contiguous int32 buffer; the query's output tensors are views into it, so
nothing is packed or copied before the all-gather.  torch.distributed supplies the
collective (NCCL over NVLink on GPUs); all arithmetic runs in the CUDA library.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import torch
import torch.distributed as dist

from . import binding as B


@dataclass(frozen=True)
class RecordLayout:
    """Byte offsets of one rank's record for (nq, k, L).  The int64 part comes first so that
    it is 8-byte aligned whatever nq, k and L are."""
    nq: int
    k: int
    L: int

    @property
    def off_gidx(self) -> int:
        return 0

    @property
    def off_score(self) -> int:
        return self.nq * self.k * 8

    @property
    def off_len(self) -> int:
        return self.off_score + self.nq * self.k * 4

    @property
    def off_tok(self) -> int:
        return self.off_len + self.nq * self.k * 4

    @property
    def off_idx(self) -> int:                  # local rows: scratch, not used by the merge
        return self.off_tok + self.nq * self.k * self.L * 4

    @property
    def off_fired(self) -> int:
        return self.off_idx + self.nq * self.k * 4

    @property
    def nbytes(self) -> int:
        n = self.off_fired + self.nq * 4
        return (n + 7) // 8 * 8

    def views(self, buf: torch.Tensor):
        """(gidx int64 [nq,k], QueryOut with tensors viewing `buf`) for a uint8 buffer."""
        nq, k, L = self.nq, self.k, self.L

        def v(off, count, dtype, shape):
            size = torch.empty((), dtype=dtype).element_size()
            return buf[off: off + count * size].view(dtype).view(shape)

        gidx = v(self.off_gidx, nq * k, torch.int64, (nq, k))
        out = B.QueryOut(v(self.off_idx, nq * k, torch.int32, (nq, k)),
                         v(self.off_score, nq * k, torch.float32, (nq, k)),
                         v(self.off_fired, nq, torch.int32, (nq,)),
                         v(self.off_len, nq * k, torch.int32, (nq, k)),
                         v(self.off_tok, nq * k * L, torch.int32, (nq, k, L)))
        out._c = B.CQueryOut(out.idx.data_ptr(), out.score.data_ptr(), out.fired.data_ptr(),
                             out.cont_len.data_ptr(), out.cont_tok.data_ptr())
        return gidx, out


def all_gather_records(send: torch.Tensor, group=None) -> torch.Tensor:
    """[nbytes] uint8 on every rank -> [world, nbytes] with rank r's record in row r."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    recv = torch.empty((world, send.numel()), dtype=send.dtype, device=send.device)
    if world == 1:
        recv[0].copy_(send)
    else:
        dist.all_gather_into_tensor(recv.view(-1), send, group=group)
    return recv


@dataclass
class ShardedOut:
    gidx: torch.Tensor       # [nq,k] int64 global positions, -1 padded
    score: torch.Tensor      # [nq,k] float32
    fired: torch.Tensor      # [nq] int32
    cont_len: torch.Tensor   # [nq,k] int32
    cont_tok: torch.Tensor   # [nq,k,L] int32


def merge_gathered(gathered: torch.Tensor, lay: RecordLayout, theta: float, stream=None
                   ) -> ShardedOut:
    """oilbird_merge_shards on a [n_shards, nbytes] uint8 CUDA buffer of records."""
    n_shards = gathered.shape[0]
    dev = gathered.device
    nq, k, L = lay.nq, lay.k, lay.L
    out = ShardedOut(B.ALLOC((nq, k), torch.int64, dev),
                     B.ALLOC((nq, k), torch.float32, dev),
                     B.ALLOC((nq,), torch.int32, dev),
                     B.ALLOC((nq, k), torch.int32, dev),
                     B.ALLOC((nq, k, L), torch.int32, dev))
    B._check(B.lib().oilbird_merge_shards(
        n_shards, nq, k, L, float(theta), gathered.data_ptr(), gathered.stride(0), lay.off_gidx,
        lay.off_score, lay.off_len, lay.off_tok, out.gidx.data_ptr(), out.score.data_ptr(),
        out.fired.data_ptr(), out.cont_len.data_ptr(), out.cont_tok.data_ptr(), dev.index or 0,
        B._stream_ptr(stream)), "oilbird_merge_shards")
    return out


class ShardedPool:
    """This rank's shard of a pool that spans the process group."""

    def __init__(self, d: int, capacity_rows: int, group=None, **pool_kw):
        self.group = group
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.pool = B.Pool(d, capacity_rows, **pool_kw)
        self._bufs: dict = {}

    def append(self, states, tokens, global_row: int, tag: int = 0, new_trace: bool = True):
        """Called on the owning rank only, with the global position of the first row."""
        self.pool.append_global(states, tokens, global_row, tag=tag, new_trace=new_trace)

    def local_record(self, q: torch.Tensor, params: B.QueryParams):
        """Steps 1 and 2: this rank's record (a uint8 buffer) and its layout."""
        if params.depth_mode == B.DEPTH_RANKED:
            # a neighbour's depth would be set by its rank on its own shard, not in the merged
            # answer, and the merge only carries continuations along
            raise ValueError("copy depth by rank is not offered on a sharded pool")
        q = q.reshape(-1, self.pool.d)
        lay = RecordLayout(q.shape[0], params.k, params.cont_len)
        buf = self._bufs.get(lay)
        if buf is None:
            buf = torch.empty(lay.nbytes, dtype=torch.uint8, device=q.device)
            self._bufs[lay] = buf
        gidx, out = lay.views(buf)
        local = B.QueryParams(k=params.k, theta=float("-inf"), offset=params.offset,
                              depth_mode=params.depth_mode, cont_len=params.cont_len,
                              tier_thr=params.tier_thr, tier_depth=params.tier_depth,
                              exclude_tag=params.exclude_tag, path=params.path)
        self.pool.query(q, local, out=out)
        self.pool.to_global(out.idx, out=gidx)
        return buf, lay

    def query(self, q: torch.Tensor, params: B.QueryParams) -> ShardedOut:
        """Same query on every rank (replicated q); the answer is replicated too."""
        buf, lay = self.local_record(q, params)
        gathered = all_gather_records(buf, self.group)           # step 3: one collective
        return merge_gathered(gathered, lay, params.theta)       # step 4

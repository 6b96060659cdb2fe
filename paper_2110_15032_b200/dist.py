"""The k logical shards of a placement mapped onto the ranks of a torch.distributed job, one
process per GPU (Section 3.1: a placement is the set of devices a tensor lives on; Section 3.2:
a boxing op between them stands for a collective).

Every rank owns a contiguous block of k / world_size shards.  A boxing op then runs as
`sbp_boxing_shard` calls: each rank produces the destination shards it owns, reading the source
local tensors it needs straight out of its peers' memory (peer-mapped buffers, plain loads over
NVLink; no multicast of any kind), with a host barrier before (sources complete everywhere) and
after (nobody still reads a source that its owner is about to overwrite).  Nothing in a kernel
waits for another rank.

`ShardMap` and `sources_read` are plain host logic.  `PeerShards` and `boxing_over_ranks` need one
GPU per rank; on a single-GPU job (world_size 1) they reduce to the local calls.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as _b


class ShardMap:
    """Block mapping of k shards onto world_size ranks: shard r lives on rank r // (k / world_size)."""

    def __init__(self, k: int, world_size: int):
        if k < 1 or world_size < 1 or k % world_size != 0:
            raise ValueError(f"k = {k} shards do not divide evenly over {world_size} ranks")
        self.k, self.world_size, self.per_rank = int(k), int(world_size), k // world_size

    def owner(self, shard: int) -> int:
        if not 0 <= shard < self.k:
            raise IndexError(shard)
        return shard // self.per_rank

    def shards(self, rank: int) -> range:
        if not 0 <= rank < self.world_size:
            raise IndexError(rank)
        return range(rank * self.per_rank, (rank + 1) * self.per_rank)


def _split_range(n: int, k: int, r: int):
    """(start, length) of shard r's piece of an axis of length n split k ways.  The split rule lives
    in the library alone: the lengths are asked from sbp_local_shape, the start is their running sum."""
    lens = [_b.sbp_local_shape((n,), _b.S(0), k, i)[0] for i in range(r + 1)]
    return sum(lens[:-1]), lens[-1]


def sources_read(src_sig: _b.Sig, dst_sig: _b.Sig, p: int, q: int, dst_shard: int, shape: Sequence[int]) -> List[int]:
    """Source shards whose local tensors `sbp_boxing_shard(..., dst_shard)` reads, for a tensor of
    logical `shape` going from `src_sig` on p shards to `dst_sig` on q shards (p == q: the same
    placement).  What a rank must be able to reach in its peers' memory before it makes the call."""
    split, bcast = _b.SBP_SPLIT, _b.SBP_BROADCAST
    src_p = src_sig.kind not in (split, bcast)
    dst_p = dst_sig.kind not in (split, bcast)
    if any(int(n) == 0 for n in shape):
        return []
    if dst_sig.kind == split and _split_range(int(shape[dst_sig.axis]), q, dst_shard)[1] == 0:
        return []                                     # an empty destination shard reads nothing
    if src_p and dst_p:                               # partial r goes to shard r mod q
        return list(range(dst_shard, p, q))
    if src_p:                                         # every partial is reduced
        return list(range(p))
    if src_sig.kind == bcast:
        if dst_p:                                     # shard 0 receives the tensor, the others zeros
            return [0] if dst_shard == 0 else []
        return [dst_shard % p]                        # any replica serves: the shard's own on one placement
    # split source: the shards whose range on the source axis overlaps what the destination shard holds
    ax = src_sig.axis
    n = int(shape[ax])
    lo, hi = 0, n
    if dst_p or (dst_sig.kind == split and dst_sig.axis == ax):
        start, ln = _split_range(n, q, dst_shard)     # S(i) -> S(i), or the q-way piece kept in partial d
        lo, hi = start, start + ln
    out = []
    for s in range(p):
        start, ln = _split_range(n, p, s)
        if ln > 0 and max(start, lo) < min(start + ln, hi):
            out.append(s)
    return out


class PeerShards:
    """The local tensors of one global tensor across the ranks of a process group: this rank's
    shards live in a peer-mappable allocation, the others are views of the peers' allocations.
    `.tensor` is an SbpTensor whose locals can all be read from this rank's GPU."""

    def __init__(self, shape, dtype, sig: _b.Sig, smap: ShardMap, group=None, device=None):
        import torch.distributed as dist
        self.shape, self.dtype, self.sig, self.smap = tuple(shape), dtype, sig, smap
        self.group = group if group is not None else dist.group.WORLD
        self.rank = dist.get_rank(self.group)
        if dist.get_world_size(self.group) != smap.world_size:
            raise ValueError("process group and shard map differ in size")
        device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        shapes = [tuple(_b.sbp_local_shape(self.shape, sig, smap.k, r, dtype)) for r in range(smap.k)]
        numels = [int(torch.Size(s).numel()) for s in shapes]
        # one slab per rank, every shard at a 256-byte aligned offset; all ranks allocate the same size
        esz = torch.empty((), dtype=dtype).element_size()
        pad = lambda n: (n * esz + 255) // 256 * 256 // esz
        slab = max(sum(pad(numels[r]) for r in smap.shards(rk)) for rk in range(smap.world_size))
        if smap.world_size == 1:
            self._slab = torch.empty(max(slab, 1), dtype=dtype, device=device)
            slabs = [self._slab]
        else:
            import torch.distributed._symmetric_memory as symm
            self._slab = symm.empty(max(slab, 1), dtype=dtype, device=device)
            self._handle = symm.rendezvous(self._slab, self.group)
            slabs = [self._slab if rk == self.rank else self._handle.get_buffer(rk, (max(slab, 1),), dtype)
                     for rk in range(smap.world_size)]
        locals_: List[torch.Tensor] = []
        for rk in range(smap.world_size):
            off = 0
            for r in smap.shards(rk):
                locals_.append(slabs[rk][off:off + numels[r]].view(shapes[r]))
                off += pad(numels[r])
        self.tensor = _b.SbpTensor(self.shape, dtype, sig, locals_)

    def own(self) -> List[torch.Tensor]:
        """This rank's local tensors (the ones it may write)."""
        return [self.tensor.locals[r] for r in self.smap.shards(self.rank)]


def boxing_over_ranks(src: PeerShards, dst: PeerShards, stream: Optional[torch.cuda.Stream] = None) -> None:
    """src -> dst across the ranks: every rank produces the destination shards it owns."""
    import torch.distributed as dist
    stream = stream if stream is not None else torch.cuda.current_stream()
    stream.synchronize()
    if src.smap.world_size > 1:
        dist.barrier(src.group)                       # every rank's sources are complete
    for d in dst.smap.shards(dst.rank):
        _b.sbp_boxing_shard(src.tensor, dst.tensor, d, stream)
    stream.synchronize()
    if src.smap.world_size > 1:
        dist.barrier(src.group)                       # nobody still reads a source

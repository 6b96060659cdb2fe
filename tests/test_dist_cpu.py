"""Host logic of the shards-on-ranks mapping, on CPU.  `sources_read` is checked against the
oracle by perturbation (a destination shard reads a source shard exactly when changing that source
changes it); the division of work between ranks is run as two gloo processes, each producing
the destination shards it owns from only the sources `sources_read` names."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp
from helpers import osig

import paper_2110_15032_b200 as sbp
from paper_2110_15032_b200.dist import ShardMap, sources_read
import sbp_datagen as dg
from oracle import sbp_oracle as O

SIGS = [sbp.S(0), sbp.S(1), sbp.B, sbp.P_SUM]


def _oracle(src, src_sig, dst_sig, p, q):
    if p == q:
        return O.boxing(src, osig(src_sig), osig(dst_sig))
    return O.boxing_disjoint(src, osig(src_sig), osig(dst_sig), q)


def test_shard_map_blocks():
    m = ShardMap(8, 2)
    assert list(m.shards(0)) == [0, 1, 2, 3] and list(m.shards(1)) == [4, 5, 6, 7]
    assert [m.owner(r) for r in range(8)] == [0, 0, 0, 0, 1, 1, 1, 1]
    assert sorted(r for rk in range(2) for r in m.shards(rk)) == list(range(8))
    with pytest.raises(ValueError):
        ShardMap(6, 4)
    with pytest.raises(IndexError):
        m.owner(8)


@pytest.mark.parametrize("shape", [(6, 8), (5, 3), (2, 7)])
@pytest.mark.parametrize("p,q", [(2, 2), (4, 4), (3, 3), (2, 3), (4, 2), (3, 5), (5, 1)])
def test_sources_read_is_the_data_dependence(shape, p, q):
    T = np.arange(1, 1 + shape[0] * shape[1], dtype=np.float32).reshape(shape)
    for src_sig in SIGS:
        if src_sig.kind == 1:
            continue                                  # replicas are equal by definition: see the next test
        parts = [dg.small_integers(41, r, shape, 1, 9).numpy().astype(np.float32) for r in range(p)]
        src = parts if src_sig == sbp.P_SUM else O.to_locals(T, osig(src_sig), p)
        for dst_sig in SIGS:
            base = _oracle(src, src_sig, dst_sig, p, q)
            for d in range(q):
                deps = set()
                for s in range(p):
                    if src[s].size == 0:
                        continue
                    bumped = [a.copy() for a in src]
                    bumped[s] = bumped[s] + 1000.0
                    if not np.array_equal(_oracle(bumped, src_sig, dst_sig, p, q)[d], base[d]):
                        deps.add(s)
                assert set(sources_read(src_sig, dst_sig, p, q, d, shape)) == deps, (src_sig, dst_sig, p, q, d)


def test_sources_read_broadcast_source_convention():
    """A broadcast source: the shard's own replica on one placement, replica d mod p otherwise;
    B -> P(sum) moves the tensor to shard 0 only."""
    for p, q in [(4, 4), (2, 5), (6, 3)]:
        for d in range(q):
            assert sources_read(sbp.B, sbp.S(1), p, q, d, (8, 12)) == [d % p]
            assert sources_read(sbp.B, sbp.B, p, q, d, (8, 12)) == [d % p]
            assert sources_read(sbp.B, sbp.P_SUM, p, q, d, (8, 12)) == ([0] if d == 0 else [])
    assert sources_read(sbp.B, sbp.S(0), 2, 4, 3, (2, 12)) == []          # an empty destination shard
    assert sources_read(sbp.S(0), sbp.B, 2, 2, 0, (0, 12)) == []


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


CASES = [(sbp.S(0), sbp.S(1), 4, 4), (sbp.S(1), sbp.B, 4, 4), (sbp.P_SUM, sbp.S(0), 4, 4), (sbp.P_SUM, sbp.B, 2, 2),
         (sbp.S(0), sbp.S(0), 4, 6), (sbp.P_SUM, sbp.P_SUM, 6, 4), (sbp.S(1), sbp.P_SUM, 2, 4), (sbp.S(0), sbp.B, 6, 2)]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shape = (12, 10)
        results = []
        for ci, (src_sig, dst_sig, p, q) in enumerate(CASES):
            smap_s, smap_d = ShardMap(p, world), ShardMap(q, world)
            # every rank creates only the source shards it owns ...
            if src_sig == sbp.P_SUM:
                full = [dg.small_integers(50 + ci, r, shape, -5, 6).numpy().astype(np.float32) for r in range(p)]
            else:
                T = dg.normal(50 + ci, 0, shape, 0, 1).numpy()
                full = O.to_locals(T, osig(src_sig), p)
            own = {r: torch.from_numpy(np.ascontiguousarray(full[r])) for r in smap_s.shards(rank)}
            # ... and what it can "reach in its peers' memory" is an all-gather of the owned shards
            gathered = [None] * world
            dist.all_gather_object(gathered, {r: t.numpy() for r, t in own.items()})
            reach = {}
            for g in gathered:
                reach.update(g)
            mine = {}
            for d in smap_d.shards(rank):
                need = sources_read(src_sig, dst_sig, p, q, d, shape)
                # sources it does not name are poisoned: the shard must not depend on them
                src = [reach[s] if s in need else np.full_like(reach[s], np.nan) for s in range(p)]
                o = O.boxing(src, osig(src_sig), osig(dst_sig)) if p == q else \
                    O.boxing_disjoint(src, osig(src_sig), osig(dst_sig), q)
                mine[d] = o[d]
            dist.barrier()
            results.append(mine)
        out.put((rank, results))
    finally:
        dist.destroy_process_group()


def test_two_ranks_produce_their_own_destination_shards_gloo():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    qout = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, qout)) for r in range(world)]
    for pr in procs:
        pr.start()
    res = dict(qout.get(timeout=180) for _ in range(world))
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    shape = (12, 10)
    for ci, (src_sig, dst_sig, p, q) in enumerate(CASES):
        if src_sig == sbp.P_SUM:
            full = [dg.small_integers(50 + ci, r, shape, -5, 6).numpy().astype(np.float32) for r in range(p)]
        else:
            full = O.to_locals(dg.normal(50 + ci, 0, shape, 0, 1).numpy(), osig(src_sig), p)
        want = _oracle(full, src_sig, dst_sig, p, q)
        got = {}
        for rank in range(world):
            assert sorted(res[rank][ci]) == list(ShardMap(q, world).shards(rank))     # each rank: exactly its shards
            got.update(res[rank][ci])
        assert sorted(got) == list(range(q))
        for d in range(q):
            assert np.array_equal(got[d], want[d]), (ci, d)

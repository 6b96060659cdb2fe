"""sbp_boxing_shard: the part of a boxing op that one device of the destination placement executes.
Each call writes one destination local tensor and nothing else; the k calls together must give,
bit for bit, what the oracle gives for the whole transform (same and different shard counts)."""
import numpy as np
import pytest
import torch
from helpers import bits, make_global, np_bits, osig, split_cpu, storage_of, to_np

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16, I64 = torch.float32, torch.bfloat16, torch.int64


def _source_locals(shape, dtype, sig, p, seed):
    if sig.kind in (2, 3):
        return [dg.normal(seed, r, shape, 0.0, 1.0, dtype) for r in range(p)]
    T = dg.integers(seed, 0, shape, -(1 << 40), 1 << 40) if dtype == I64 else dg.normal(seed, 0, shape, 0.0, 1.0, dtype)
    return split_cpu(T, sig, p)


def _run(shape, dtype, src_sig, dst_sig, p, q, seed=5, dst_dtype=None):
    dst_dtype = dst_dtype or dtype
    src_cpu = _source_locals(shape, dtype, src_sig, p, seed)
    arrs = [t.numpy() if dtype == I64 else to_np(t) for t in src_cpu]
    storage = storage_of(dtype) if dtype != I64 else "f32"
    if dst_dtype != dtype:
        want = O.boxing_cast(arrs, osig(src_sig), osig(dst_sig), storage_of(dst_dtype))
    elif p == q:
        want = O.boxing(arrs, osig(src_sig), osig(dst_sig), storage)
    else:
        want = O.boxing_disjoint(arrs, osig(src_sig), osig(dst_sig), q, storage)
    src = make_global(src_cpu, shape, dtype, src_sig)
    full = sbp.empty_global(shape, dst_dtype, dst_sig, q)
    for d in range(q):
        # a guard band around the shard's buffer shows that nothing else is written
        n = full.locals[d].numel()
        buf = torch.empty(n + 64, dtype=dst_dtype, device="cuda")
        buf.view(torch.uint8).fill_(0xAB)
        mine = buf[32:32 + n].view(full.locals[d].shape)
        locs = [None] * q
        locs[d] = mine
        dst = sbp.SbpTensor(shape, dst_dtype, dst_sig, locs)
        sbp.sbp_boxing_shard(src, dst, d)
        torch.cuda.synchronize()
        sbp.sbp_check_device_errors()
        assert tuple(mine.shape) == tuple(want[d].shape)
        assert np.array_equal(bits(mine), np_bits(want[d], dst_dtype)), f"shard {d} differs"
        guard = torch.cat([buf[:32], buf[32 + n:]]).view(torch.uint8)
        assert bool((guard == 0xAB).all()), f"shard {d}: wrote outside its local tensor"


ALL = [(sbp.S(0), sbp.B), (sbp.S(1), sbp.B), (sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0)), (sbp.S(0), sbp.S(0)),
       (sbp.B, sbp.S(0)), (sbp.B, sbp.S(1)), (sbp.B, sbp.B), (sbp.S(0), sbp.P_SUM), (sbp.S(1), sbp.P_SUM),
       (sbp.B, sbp.P_SUM), (sbp.P_SUM, sbp.B), (sbp.P_SUM, sbp.S(0)), (sbp.P_SUM, sbp.S(1)), (sbp.P_SUM, sbp.P_SUM),
       (sbp.P_MAX, sbp.B), (sbp.P_MAX, sbp.S(1))]


@pytest.mark.parametrize("src_sig,dst_sig", ALL)
@pytest.mark.parametrize("k", [1, 3, 4, 8])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_shard_calls_same_placement(src_sig, dst_sig, k, dtype):
    _run((96, 320), dtype, src_sig, dst_sig, k, k)       # wide vectors, bulk-copy engine where it applies
    _run((37, 53), dtype, src_sig, dst_sig, k, k)        # ragged


@pytest.mark.parametrize("src_sig,dst_sig", ALL)
@pytest.mark.parametrize("p,q", [(2, 3), (4, 2), (3, 8), (5, 1)])
def test_shard_calls_different_placements(src_sig, dst_sig, p, q):
    _run((96, 320), BF16, src_sig, dst_sig, p, q)
    _run((37, 53), F32, src_sig, dst_sig, p, q)


@pytest.mark.parametrize("src_sig,dst_sig", [(sbp.S(0), sbp.S(2)), (sbp.S(2), sbp.S(1)), (sbp.S(1), sbp.B),
                                             (sbp.P_SUM, sbp.S(1)), (sbp.S(2), sbp.P_SUM)])
def test_shard_calls_3d_and_int64(src_sig, dst_sig):
    _run((5, 24, 40), F32, src_sig, dst_sig, 4, 4)
    _run((3, 7, 9), BF16, src_sig, dst_sig, 3, 5)
    if src_sig.kind not in (2, 3):
        _run((5, 24, 40), I64, src_sig, dst_sig, 2, 2)


def test_shard_calls_cast_gather_and_many_tiles():
    _run((256, 384), F32, sbp.S(0), sbp.B, 4, 4, dst_dtype=BF16)
    _run((1536, 2048), BF16, sbp.S(0), sbp.S(1), 4, 4)
    _run((1536, 2048), BF16, sbp.P_SUM, sbp.S(0), 4, 4)
    _run((1536, 2048), BF16, sbp.S(1), sbp.B, 4, 4)


def test_shard_argument_errors():
    src = make_global(_source_locals((8, 8), F32, sbp.S(0), 2, 1), (8, 8), F32, sbp.S(0))
    dst = sbp.SbpTensor((8, 8), F32, sbp.B, [None, None])
    with pytest.raises(sbp.SbpError):
        sbp.sbp_boxing_shard(src, dst, 0)                 # the shard asked for has no buffer
    with pytest.raises(sbp.SbpError):
        sbp.sbp_boxing_shard(src, sbp.empty_global((8, 8), F32, sbp.B, 2), 2)   # outside the placement
    with pytest.raises(sbp.SbpError):
        sbp.sbp_boxing_shard(src, sbp.empty_global((8, 8), F32, sbp.B, 2), -1)


def test_boxing_over_ranks_on_a_one_rank_job():
    """The rank-level driver with world_size 1 (one GPU): allocation, shard ownership and the
    per-shard calls; the peer mapping itself needs more than one GPU."""
    import socket
    import torch.distributed as dist
    from paper_2110_15032_b200.dist import PeerShards, ShardMap, boxing_over_ranks
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        shape, k = (96, 160), 4
        smap = ShardMap(k, 1)
        for src_sig, dst_sig in [(sbp.S(0), sbp.S(1)), (sbp.P_SUM, sbp.B), (sbp.S(1), sbp.B), (sbp.B, sbp.S(0))]:
            src_cpu = _source_locals(shape, BF16, src_sig, k, 9)
            src = PeerShards(shape, BF16, src_sig, smap)
            dst = PeerShards(shape, BF16, dst_sig, smap)
            assert len(src.own()) == k
            for t, c in zip(src.own(), src_cpu):
                t.copy_(c)
            boxing_over_ranks(src, dst)
            want = O.boxing([to_np(t) for t in src_cpu], osig(src_sig), osig(dst_sig), "bf16")
            for r in range(k):
                assert np.array_equal(bits(dst.tensor.locals[r]), np_bits(want[r], BF16))
    finally:
        dist.destroy_process_group()

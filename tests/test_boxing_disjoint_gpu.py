"""Parity of boxing between two different placements (Table 2, column "disjoint": p source
shards, q destination shards) against the CPU oracle.  Data movement is bit-exact; the
reductions follow the same fixed-order fp32 rule on both sides and are compared bit for bit."""
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


def _run(shape, dtype, src_sig, dst_sig, p, q, seed=3, alias=False, host=False):
    src_cpu = _source_locals(shape, dtype, src_sig, p, seed)
    arrs = [t.numpy() if dtype == I64 else to_np(t) for t in src_cpu]
    want = O.boxing_disjoint(arrs, osig(src_sig), osig(dst_sig), q, storage_of(dtype) if dtype != I64 else "f32")
    assert len(want) == q
    if host:
        src = sbp.SbpTensor(shape, dtype, src_sig, [t.contiguous().pin_memory() for t in src_cpu])
        dst = sbp.empty_global(shape, dtype, dst_sig, q, device="cpu")
        dst = sbp.SbpTensor(shape, dtype, dst_sig, [t.pin_memory() for t in dst.locals])
        ws = torch.empty(sbp.sbp_boxing_host_workspace_bytes(src, dst) + 256, dtype=torch.uint8, device="cuda")
        sbp.sbp_boxing_host(src, dst, ws)
    else:
        src = make_global(src_cpu, shape, dtype, src_sig)
        dst = sbp.empty_global(shape, dtype, dst_sig, q, alias_replicas=alias)
        for t in dst.locals:
            t.view(torch.uint8).fill_(0xAB)
        sbp.sbp_boxing(src, dst)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    for r in range(q):
        got = dst.locals[r]
        assert tuple(got.shape) == tuple(want[r].shape), (r, got.shape, want[r].shape)
        assert np.array_equal(bits(got), np_bits(want[r], dtype)), f"shard {r} differs"


PQ = [(2, 3), (4, 2), (3, 8), (8, 3), (1, 4), (5, 1), (16, 7)]
MOVES = [(sbp.S(0), sbp.S(0)), (sbp.S(1), sbp.S(1)), (sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0)),
         (sbp.S(0), sbp.B), (sbp.S(1), sbp.B), (sbp.B, sbp.S(0)), (sbp.B, sbp.S(1)), (sbp.B, sbp.B),
         (sbp.S(0), sbp.P_SUM), (sbp.S(1), sbp.P_SUM), (sbp.B, sbp.P_SUM)]
REDUCES = [(sbp.P_SUM, sbp.B), (sbp.P_SUM, sbp.S(0)), (sbp.P_SUM, sbp.S(1)), (sbp.P_SUM, sbp.P_SUM),
           (sbp.P_MAX, sbp.B), (sbp.P_MAX, sbp.S(1))]


@pytest.mark.parametrize("src_sig,dst_sig", MOVES + REDUCES)
@pytest.mark.parametrize("p,q", PQ)
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_disjoint_2d_aligned_and_ragged(src_sig, dst_sig, p, q, dtype):
    _run((96, 320), dtype, src_sig, dst_sig, p, q)        # every piece boundary 16-byte aligned for most p, q
    _run((37, 53), dtype, src_sig, dst_sig, p, q)         # ragged: narrow vectors, uneven pieces


@pytest.mark.parametrize("src_sig,dst_sig", [(sbp.S(0), sbp.S(2)), (sbp.S(2), sbp.S(0)), (sbp.S(1), sbp.S(1)),
                                             (sbp.S(2), sbp.S(1)), (sbp.S(1), sbp.B), (sbp.B, sbp.S(2)),
                                             (sbp.P_SUM, sbp.S(1)), (sbp.S(1), sbp.P_SUM), (sbp.S(2), sbp.P_SUM)])
@pytest.mark.parametrize("p,q", [(2, 3), (4, 6), (7, 2)])
def test_disjoint_3d(src_sig, dst_sig, p, q):
    _run((5, 24, 40), F32, src_sig, dst_sig, p, q)
    _run((3, 7, 9), BF16, src_sig, dst_sig, p, q)


@pytest.mark.parametrize("src_sig,dst_sig", [(sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(1)), (sbp.B, sbp.S(0)),
                                             (sbp.S(0), sbp.B), (sbp.S(1), sbp.P_SUM)])
def test_disjoint_int64_moves_bits(src_sig, dst_sig):
    _run((33, 20), I64, src_sig, dst_sig, 3, 5)


@pytest.mark.parametrize("p,q", [(2, 5), (6, 3)])
def test_disjoint_more_shards_than_rows_and_empty(p, q):
    """Shards of length zero on either side, and an empty tensor."""
    for src_sig, dst_sig in [(sbp.S(0), sbp.S(0)), (sbp.S(0), sbp.S(1)), (sbp.S(0), sbp.B), (sbp.B, sbp.S(0)),
                             (sbp.P_SUM, sbp.S(0)), (sbp.S(0), sbp.P_SUM)]:
        _run((2, 16), F32, src_sig, dst_sig, p, q)
        _run((0, 16), F32, src_sig, dst_sig, p, q)


def test_disjoint_pmax_onto_more_shards_is_refused_and_fewer_is_exact():
    _run((64, 48), BF16, sbp.P_MAX, sbp.P_MAX, 5, 2)
    src = make_global(_source_locals((8, 8), F32, sbp.P_MAX, 2, 1), (8, 8), F32, sbp.P_MAX)
    dst = sbp.empty_global((8, 8), F32, sbp.P_MAX, 3)
    with pytest.raises(sbp.SbpError):
        sbp.sbp_boxing(src, dst)
    with pytest.raises(sbp.SbpError):                     # the cast-fused gather stays on one placement
        sbp.sbp_boxing(make_global(_source_locals((8, 8), F32, sbp.S(0), 2, 1), (8, 8), F32, sbp.S(0)),
                       sbp.empty_global((8, 8), BF16, sbp.B, 3))


def test_disjoint_replicas_aliased_and_through_host_buffers():
    _run((128, 96), BF16, sbp.S(1), sbp.B, 3, 4, alias=True)
    _run((128, 96), BF16, sbp.P_SUM, sbp.B, 3, 4, alias=True)
    _run((61, 96), F32, sbp.S(0), sbp.S(1), 2, 3, host=True)
    _run((61, 96), BF16, sbp.P_SUM, sbp.S(0), 4, 3, host=True)


def test_disjoint_spans_many_tiles():
    """Several megabytes per shard: many tiles per task, full-width vectors."""
    _run((1536, 2048), BF16, sbp.S(0), sbp.S(1), 4, 8)
    _run((1536, 2048), BF16, sbp.S(0), sbp.S(0), 4, 6)
    _run((1536, 2048), BF16, sbp.P_SUM, sbp.S(1), 4, 8)
    _run((1536, 2048), F32, sbp.P_SUM, sbp.P_SUM, 5, 2)

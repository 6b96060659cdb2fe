"""Parity of the CUDA boxing kernels against the CPU oracle (Section 3.2, Table 2).

Pure data movement must be bit-exact.  P(sum) reductions follow the same fixed-order fp32
rule on both sides and are expected bit-equal; the asserted bar is 1e-6 relative plus an
fp64 cross-check that is safe under cancellation.  P(max) is exact."""
import numpy as np
import pytest
import torch
from helpers import bits, check_guards, make_global, np_bits, osig, split_cpu, storage_of, to_np

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16, I64 = torch.float32, torch.bfloat16, torch.int64


def _source_locals(shape, dtype, sig, k, seed):
    """CPU local tensors of a seeded global tensor under `sig`."""
    if sig.kind in (2, 3):      # P: k independent shards
        return [dg.normal(seed, r, shape, 0.0, 1.0, dtype) for r in range(k)]
    if dtype == I64:
        T = dg.integers(seed, 0, shape, -(1 << 40), 1 << 40)
    else:
        T = dg.normal(seed, 0, shape, 0.0, 1.0, dtype)
    return split_cpu(T, sig, k)


def _oracle_boxing(src_cpu, dtype, src_sig, dst_sig):
    if dtype == I64:
        arrs = [t.numpy() for t in src_cpu]
    else:
        arrs = [to_np(t) for t in src_cpu]
    return O.boxing(arrs, osig(src_sig), osig(dst_sig), storage_of(dtype) if dtype != I64 else "f32")


def _run(shape, dtype, src_sig, dst_sig, k, seed=1, engine=0, alias=False, offset_elems=0):
    src_cpu = _source_locals(shape, dtype, src_sig, k, seed)
    want = _oracle_boxing(src_cpu, dtype, src_sig, dst_sig)
    if offset_elems:
        # place every local tensor at an odd element offset inside a larger buffer
        def shifted(t):
            buf = torch.zeros(t.numel() + offset_elems + 8, dtype=t.dtype, device="cuda")
            v = buf[offset_elems:offset_elems + t.numel()].view(t.shape)
            v.copy_(t)
            return v
        src = sbp.SbpTensor(shape, dtype, src_sig, [shifted(t) for t in src_cpu])
    else:
        src = make_global(src_cpu, shape, dtype, src_sig)
    dst = sbp.empty_global(shape, dtype, dst_sig, k, alias_replicas=alias)
    for t in dst.locals:
        t.view(torch.uint8).fill_(0xAB)
    sbp.sbp_boxing_set_copy_engine(engine)
    try:
        sbp.sbp_boxing(src, dst)
        torch.cuda.synchronize()
        sbp.sbp_check_device_errors()
    finally:
        sbp.sbp_boxing_set_copy_engine(0)
    check_guards()                                   # nothing was stored outside a destination shard
    assert len(want) == k
    for r in range(k):
        got = dst.locals[r]
        assert tuple(got.shape) == tuple(want[r].shape), (r, got.shape, want[r].shape)
        assert np.array_equal(bits(got), np_bits(want[r], dtype)), f"shard {r} differs"
    return src_cpu, dst


MOVES = [(sbp.S(0), sbp.B), (sbp.S(1), sbp.B), (sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0)),
         (sbp.B, sbp.S(0)), (sbp.B, sbp.S(1)), (sbp.S(0), sbp.S(0)), (sbp.B, sbp.B)]
TO_PARTIAL = [(sbp.S(0), sbp.P_SUM), (sbp.S(1), sbp.P_SUM), (sbp.B, sbp.P_SUM)]
REDUCES = [(sbp.P_SUM, sbp.B), (sbp.P_SUM, sbp.S(0)), (sbp.P_SUM, sbp.S(1)),
           (sbp.P_MAX, sbp.B), (sbp.P_MAX, sbp.S(1)), (sbp.P_SUM, sbp.P_SUM)]


@pytest.mark.parametrize("src_sig,dst_sig", MOVES + REDUCES + TO_PARTIAL)
@pytest.mark.parametrize("k", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_boxing_2d_aligned_and_ragged(src_sig, dst_sig, k, dtype):
    _run((64, 96), dtype, src_sig, dst_sig, k)           # config-1 result shape, aligned
    _run((67, 101), dtype, src_sig, dst_sig, k)          # nothing divides: element-wise path
    _run((130, 520), dtype, src_sig, dst_sig, k)         # several tiles and a ragged tail


@pytest.mark.parametrize("src_sig,dst_sig", MOVES)
def test_boxing_int64_moves(src_sig, dst_sig):
    _run((33, 40), I64, src_sig, dst_sig, 4)


@pytest.mark.parametrize("shape", [(6, 10, 16), (3, 5, 7, 8), (4, 9, 10), (40,)])
@pytest.mark.parametrize("k", [2, 3, 4])
def test_boxing_nd_every_axis_pair(shape, k):
    nd = len(shape)
    for i in range(nd):
        _run(shape, F32, sbp.S(i), sbp.B, k)
        _run(shape, BF16, sbp.B, sbp.S(i), k)
        _run(shape, F32, sbp.P_SUM, sbp.S(i), k)
        for j in range(nd):
            if i != j:
                _run(shape, F32, sbp.S(i), sbp.S(j), k)


@pytest.mark.parametrize("src_sig,dst_sig", MOVES[:6])
@pytest.mark.parametrize("k", [2, 4])
def test_bulk_copy_engine_matches(src_sig, dst_sig, k):
    _run((512, 1024), BF16, src_sig, dst_sig, k, engine=2)     # 512 B .. 2 KiB segments
    _run((384, 8192), F32, src_sig, dst_sig, k, engine=2)      # segments above one stage
    _run((250, 1000), F32, src_sig, dst_sig, k, engine=2)      # uneven shards where k = 4 leaves a tail
    _run((67, 101), F32, src_sig, dst_sig, k, engine=2)        # unaligned: falls back to load/store


def test_boxing_to_partial_sum_nd_and_round_trip():
    for shape in [(6, 10, 16), (3, 5, 7, 8), (40,)]:
        for i in range(len(shape)):
            _run(shape, F32, sbp.S(i), sbp.P_SUM, 3)
        _run(shape, BF16, sbp.B, sbp.P_SUM, 4)
    _run((33, 40), I64, sbp.S(1), sbp.P_SUM, 4)
    # S(0) -> P(sum) -> B returns the logical tensor (x + 0 is exact)
    k, shape = 4, (96, 160)
    T = dg.normal(6, 0, shape, 0, 1, BF16)
    s0 = make_global(split_cpu(T, sbp.S(0), k), shape, BF16, sbp.S(0))
    part = sbp.empty_global(shape, BF16, sbp.P_SUM, k)
    rep = sbp.empty_global(shape, BF16, sbp.B, k)
    sbp.sbp_boxing(s0, part)
    sbp.sbp_boxing(part, rep)
    torch.cuda.synchronize()
    assert all(np.array_equal(bits(r), bits(T)) for r in rep.locals)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(s0, sbp.empty_global(shape, BF16, sbp.P_MAX, k))
    assert e.value.name == "SBP_ERR_UNSUPPORTED"


def test_boxing_larger_than_one_wave():
    _run((2048, 3072), BF16, sbp.S(1), sbp.P_SUM, 4)
    _run((2048, 3072), BF16, sbp.P_SUM, sbp.B, 4)
    _run((2048, 3072), BF16, sbp.S(0), sbp.S(1), 4)
    _run((2048, 3072), BF16, sbp.S(0), sbp.S(1), 4, engine=2)
    _run((2048, 3072), BF16, sbp.S(0), sbp.B, 4, engine=2)


def test_boxing_unaligned_pointers_and_aliased_replicas():
    _run((64, 96), F32, sbp.S(0), sbp.B, 2, offset_elems=1)
    _run((64, 96), BF16, sbp.P_SUM, sbp.B, 4, offset_elems=3)
    _run((64, 96), BF16, sbp.S(0), sbp.S(1), 4, offset_elems=1)
    _, dst = _run((64, 96), F32, sbp.P_SUM, sbp.B, 4, alias=True)
    assert all(t.data_ptr() == dst.locals[0].data_ptr() for t in dst.locals)
    _run((64, 96), BF16, sbp.S(1), sbp.B, 4, alias=True)


def test_boxing_degenerate_shapes():
    _run((3, 96), F32, sbp.S(0), sbp.B, 4)          # a shard with no rows
    _run((3, 96), F32, sbp.S(0), sbp.S(1), 4)
    _run((3, 5), F32, sbp.P_SUM, sbp.S(0), 8)
    _run((0, 16), F32, sbp.S(0), sbp.B, 2)          # empty tensor: nothing launched
    _run((1, 1), BF16, sbp.P_MAX, sbp.B, 2)


def test_psum_tolerance_and_fp64_cross_check():
    """The stated bar: fixed-order fp32 reductions within 1e-6 relative of the oracle's, and
    within one storage ulp / 1e-6 * sum|in| of the fp64 sum."""
    k, shape = 4, (256, 512)
    for dtype in (F32, BF16):
        src_cpu = [dg.normal(77, r, shape, 0.0, 1.0, dtype) for r in range(k)]
        src = make_global(src_cpu, shape, dtype, sbp.P_SUM)
        dst = sbp.empty_global(shape, dtype, sbp.B, k)
        sbp.sbp_boxing(src, dst)
        torch.cuda.synchronize()
        arrs = [to_np(t) for t in src_cpu]
        ref32 = O.reduce_sum_fixed_order(arrs, storage_of(dtype)).astype(np.float64)
        ref64 = O.reduce_sum_fp64(arrs)
        mag = sum(np.abs(a.astype(np.float64)) for a in arrs)
        for t in dst.locals:
            got = to_np(t).astype(np.float64)
            assert np.all(np.abs(got - ref32) <= 1e-6 * np.abs(ref32))
            ulp = 2.0 ** -8 * np.maximum(np.abs(ref64), 2.0 ** -126) if dtype == BF16 else 0.0
            assert np.all(np.abs(got - ref64) <= 1e-6 * mag + ulp)


def test_pmax_sign_of_zero_and_ties():
    a = torch.tensor([[0.0, -0.0, 1.0, -2.0]], dtype=F32)
    b = torch.tensor([[-0.0, 0.0, 1.0, -1.0]], dtype=F32)
    src = make_global([a, b], (1, 4), F32, sbp.P_MAX)
    dst = sbp.empty_global((1, 4), F32, sbp.B, 2)
    sbp.sbp_boxing(src, dst)
    torch.cuda.synchronize()
    want = O.reduce_max_fixed_order([a.numpy(), b.numpy()])
    assert np.array_equal(bits(dst.locals[0]), np_bits(want, F32))
    assert np.signbit(want[0, 1]) and not np.signbit(want[0, 0])


def test_round_trips_on_device():
    """S(0)->S(1)->S(0), S(i)->B->S(i) and B->S(i)->B return the input bits."""
    k, shape = 4, (96, 160)
    T = dg.normal(5, 0, shape, 0, 1, BF16)
    s0 = make_global(split_cpu(T, sbp.S(0), k), shape, BF16, sbp.S(0))
    s1 = sbp.empty_global(shape, BF16, sbp.S(1), k)
    back = sbp.empty_global(shape, BF16, sbp.S(0), k)
    rep = sbp.empty_global(shape, BF16, sbp.B, k)
    sbp.sbp_boxing(s0, s1)
    sbp.sbp_boxing(s1, back)
    sbp.sbp_boxing(s1, rep)
    torch.cuda.synchronize()
    for a, b in zip(s0.locals, back.locals):
        assert torch.equal(a, b)
    for r in rep.locals:
        assert np.array_equal(bits(r), bits(T))


def test_back_to_back_calls_keep_stream_order():
    """Boxing kernels are launched so that a call may be set up on the GPU while the call before
    it is still running; it must nevertheless see that call's results (read after write) and must
    not overwrite what that call still reads (write after read).  A chain over buffers large
    enough for many waves of CTAs, repeated: a -> b, b -> c, then z -> a while b -> c may still run,
    then a -> b again.  Every intermediate is compared with the oracle's mapping."""
    k, shape = 4, (2048, 4096)
    T = dg.normal(31, 0, shape, 0, 1, BF16)
    Z = dg.normal(31, 1, shape, 0, 1, BF16)
    want_s1 = {id(X): split_cpu(X, sbp.S(1), k) for X in (T, Z)}
    for rep in range(5):
        a = make_global(split_cpu(T, sbp.S(0), k), shape, BF16, sbp.S(0))
        z = make_global(split_cpu(Z, sbp.S(0), k), shape, BF16, sbp.S(0))
        b = sbp.empty_global(shape, BF16, sbp.S(1), k)
        c = sbp.empty_global(shape, BF16, sbp.B, k)
        b2 = sbp.empty_global(shape, BF16, sbp.S(1), k)
        sbp.sbp_boxing(a, b)        # a -> b
        sbp.sbp_boxing(b, c)        # reads b right behind its writer
        sbp.sbp_boxing(z, a)        # overwrites a, which the first call read
        sbp.sbp_boxing(a, b2)       # reads the overwritten a
        torch.cuda.synchronize()
        for r in range(k):
            assert torch.equal(b.locals[r].cpu(), want_s1[id(T)][r]), f"repeat {rep}: S(0)->S(1) shard {r}"
            assert np.array_equal(bits(c.locals[r]), bits(T)), f"repeat {rep}: replica {r} read stale data"
            assert torch.equal(b2.locals[r].cpu(), want_s1[id(Z)][r]), f"repeat {rep}: second chain shard {r}"


def test_ping_pong_between_two_buffers_without_a_host_sync():
    """X -> Y, Y -> X, X -> Y over and over on one stream with different data each round and no
    synchronisation in between: every read of a buffer must see what the launch just before it wrote
    there, although the kernels read through the non-coherent path and each may be set up on the GPU
    while its predecessor still runs.  Data movement (S(0) <-> S(1)) and the reduction (P(sum) -> B)."""
    k, shape, rounds = 4, (1024, 2048), 6
    data = [dg.normal(41, i, shape, 0, 1, BF16) for i in range(rounds)]
    srcs = [make_global(split_cpu(D, sbp.S(0), k), shape, BF16, sbp.S(0)) for D in data]
    X = sbp.empty_global(shape, BF16, sbp.S(0), k)
    Y = sbp.empty_global(shape, BF16, sbp.S(1), k)
    outs = [sbp.empty_global(shape, BF16, sbp.S(1), k) for _ in range(rounds)]
    parts = [[dg.normal(42, 10 * i + r, shape, 0, 1, BF16) for r in range(k)] for i in range(rounds)]
    psrc = [make_global(p, shape, BF16, sbp.P_SUM) for p in parts]
    P = sbp.empty_global(shape, BF16, sbp.P_SUM, k)
    sums = [sbp.empty_global(shape, BF16, sbp.B, k, alias_replicas=True) for _ in range(rounds)]
    for i in range(rounds):
        sbp.sbp_boxing(srcs[i], X)      # new data into X
        sbp.sbp_boxing(X, Y)            # X -> Y
        sbp.sbp_boxing(Y, X)            # Y -> X (X rewritten by a kernel that has just read Y)
        sbp.sbp_boxing(X, outs[i])      # X -> this round's result
        sbp.sbp_boxing(psrc[i], P)      # new partial values into P
        sbp.sbp_boxing(P, sums[i])      # reduced right behind their writer
    torch.cuda.synchronize()
    for i in range(rounds):
        want = split_cpu(data[i], sbp.S(1), k)
        for r in range(k):
            assert torch.equal(outs[i].locals[r].cpu(), want[r]), f"round {i}, shard {r}: stale or torn data"
        ref = O.boxing([to_np(t) for t in parts[i]], O.PSUM, O.B, "bf16")[0]
        assert np.array_equal(bits(sums[i].locals[0]), np_bits(ref, BF16)), f"round {i}: reduction read stale partial values"


def test_host_buffer_entry_point():
    k, shape = 4, (128, 256)
    src_cpu = [dg.normal(9, r, shape, 0, 1, BF16).pin_memory() for r in range(k)]
    src = sbp.SbpTensor(shape, BF16, sbp.P_SUM, src_cpu)
    dst_cpu = [torch.empty(sbp.sbp_local_shape(shape, sbp.S(1), k, r, BF16), dtype=BF16).pin_memory() for r in range(k)]
    dst = sbp.SbpTensor(shape, BF16, sbp.S(1), dst_cpu)
    need = sbp.sbp_boxing_host_workspace_bytes(src, dst)
    assert need >= (k + 1) * 128 * 256 * 2
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    sbp.sbp_boxing_host(src, dst, ws)
    torch.cuda.synchronize()
    want = O.boxing([to_np(t) for t in src_cpu], O.PSUM, O.S1, "bf16")
    for r in range(k):
        assert np.array_equal(bits(dst_cpu[r]), np_bits(want[r], BF16))
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing_host(src, dst, ws[:1024])
    assert e.value.name == "SBP_ERR_WORKSPACE"


@pytest.mark.parametrize("shape,axis", [((130, 96), 0), ((128, 250), 1), ((6, 50, 10), 1), ((5, 7, 64), 2)])
def test_host_entry_point_copies_only_the_blocks_b_to_s_reads(shape, axis):
    """B -> S(axis) takes block r from replica r.  The host path sends only those blocks to the
    device: everything outside replica r's own block is poisoned here (a different value in every
    replica), so a result that matches the logical tensor shows that nothing else was read, and the
    reported byte count is that of one tensor, not of k."""
    k = 4
    T = dg.normal(11, 0, shape, 0, 1, BF16)
    want = split_cpu(T, sbp.S(axis), k)
    src_cpu = []
    for r in range(k):
        rep = torch.full(shape, float(100 + r), dtype=BF16)
        lo = sum(w.shape[axis] for w in want[:r])
        idx = [slice(None)] * len(shape)
        idx[axis] = slice(lo, lo + want[r].shape[axis])
        rep[tuple(idx)] = T[tuple(idx)]
        src_cpu.append(rep.pin_memory())
    src = sbp.SbpTensor(shape, BF16, sbp.B, src_cpu)
    dst_cpu = [torch.empty(w.shape, dtype=BF16).pin_memory() for w in want]
    dst = sbp.SbpTensor(shape, BF16, sbp.S(axis), dst_cpu)
    h2d, d2h = sbp.sbp_boxing_host_copy_bytes(src, dst)
    assert h2d == T.numel() * 2 and d2h == T.numel() * 2
    ws = torch.empty(sbp.sbp_boxing_host_workspace_bytes(src, dst), dtype=torch.uint8, device="cuda")
    ws.fill_(0x5A)
    sbp.sbp_boxing_host(src, dst, ws)
    torch.cuda.synchronize()
    for r in range(k):
        assert torch.equal(dst_cpu[r], want[r]), f"shard {r}"
    # every other transform still copies all of its sources, and aliased destination replicas go back once
    psrc = sbp.SbpTensor(shape, BF16, sbp.P_SUM, src_cpu)
    one = torch.empty(shape, dtype=BF16).pin_memory()
    h2d, d2h = sbp.sbp_boxing_host_copy_bytes(psrc, sbp.SbpTensor(shape, BF16, sbp.B, [one] * k))
    assert h2d == k * T.numel() * 2 and d2h == T.numel() * 2


def test_host_entry_point_with_one_source_and_several_destinations():
    """sbp_boxing_host_multi: the source crosses to the device once, every transform reads it there;
    each result equals the oracle's; a refused pair leaves every host destination untouched."""
    k, shape = 4, (130, 250)
    parts = [dg.normal(21, r, shape, 0, 1, BF16).pin_memory() for r in range(k)]
    src = sbp.SbpTensor(shape, BF16, sbp.P_SUM, parts)
    sigs = [sbp.B, sbp.S(0), sbp.S(1)]
    dsts = []
    for sig in sigs:
        locs = [torch.full(sbp.sbp_local_shape(shape, sig, k, r, BF16), 7.0, dtype=BF16).pin_memory() for r in range(k)]
        dsts.append(sbp.SbpTensor(shape, BF16, sig, locs))
    numel = shape[0] * shape[1]
    h2d, d2h = sbp.sbp_boxing_host_multi_copy_bytes(src, dsts)
    assert h2d == k * numel * 2 and d2h == (k + 1 + 1) * numel * 2        # one upload; B to k replicas, S(0), S(1)
    need = sbp.sbp_boxing_host_multi_workspace_bytes(src, dsts)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    sbp.sbp_boxing_host_multi(src, dsts, ws)
    torch.cuda.synchronize()
    for sig, d in zip(sigs, dsts):
        want = O.boxing([to_np(t) for t in parts], O.PSUM, osig(sig), "bf16")
        for r in range(k):
            assert np.array_equal(bits(d.locals[r]), np_bits(want[r], BF16)), (sig, r)
    # B source into S(1) twice: the diagonal blocks only; into S(0) and S(1): the whole of every replica
    T = dg.normal(22, 0, shape, 0, 1, BF16)
    bsrc = sbp.SbpTensor(shape, BF16, sbp.B, [T.clone().pin_memory() for _ in range(k)])
    mk = lambda sig: sbp.SbpTensor(shape, BF16, sig, [torch.empty(sbp.sbp_local_shape(shape, sig, k, r, BF16), dtype=BF16).pin_memory()
                                                        for r in range(k)])
    two = [mk(sbp.S(1)), mk(sbp.S(1))]
    assert sbp.sbp_boxing_host_multi_copy_bytes(bsrc, two) == (numel * 2, 2 * numel * 2)
    mixed = [mk(sbp.S(0)), mk(sbp.S(1))]
    assert sbp.sbp_boxing_host_multi_copy_bytes(bsrc, mixed) == (k * numel * 2, 2 * numel * 2)
    for group in (two, mixed):
        ws = torch.empty(sbp.sbp_boxing_host_multi_workspace_bytes(bsrc, group), dtype=torch.uint8, device="cuda")
        sbp.sbp_boxing_host_multi(bsrc, group, ws)
        torch.cuda.synchronize()
        for d in group:
            want = split_cpu(T, d.sig, k)
            assert all(torch.equal(a, b) for a, b in zip(d.locals, want))
    # one pair of the call is refused (P(sum) -> P(max) has no meaning): nothing is copied or written
    bad = [dsts[0], sbp.SbpTensor(shape, BF16, sbp.P_MAX, [torch.full(shape, 7.0, dtype=BF16).pin_memory() for _ in range(k)])]
    for t in dsts[0].locals:
        t.fill_(7.0)
    ws = torch.empty(sbp.sbp_boxing_host_multi_workspace_bytes(src, dsts) * 2, dtype=torch.uint8, device="cuda")
    with pytest.raises(sbp.SbpError):
        sbp.sbp_boxing_host_multi(src, bad, ws)
    torch.cuda.synchronize()
    assert all(bool((t == 7.0).all()) for d in bad for t in d.locals)


def test_expired_device_wait_is_reported_and_the_device_stays_usable():
    """A bounded wait that runs out (a barrier nothing signals) ends the kernel normally and is
    reported once as SBP_ERR_TIMEOUT; nothing faults and later launches work."""
    sbp.sbp_check_device_errors()                     # clean slate
    sbp.sbp_selftest_wait_timeout(20)
    torch.cuda.synchronize()
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_check_device_errors()
    assert e.value.name == "SBP_ERR_TIMEOUT"
    sbp.sbp_check_device_errors()                     # flag was cleared by the report
    _run((64, 96), F32, sbp.S(0), sbp.S(1), 2)        # the context is intact
    with pytest.raises(sbp.SbpError):
        sbp.sbp_selftest_wait_timeout(5000)


@pytest.mark.parametrize("shape,axis", [((64, 96), 0), ((67, 101), 1), ((130, 520), 0), ((6, 10, 16), 1), ((2048, 1024), 1)])
@pytest.mark.parametrize("k", [1, 3, 4])
def test_cast_fused_gather_fp32_to_bf16(shape, axis, k):
    """S(i) fp32 -> B bf16: the cast of Section 6.4 folded into the all-gather."""
    T = dg.normal(31, 0, shape, 0.0, 2.0, F32)
    src = make_global(split_cpu(T, sbp.S(axis), k), shape, F32, sbp.S(axis))
    for alias in (False, True):
        dst = sbp.empty_global(shape, BF16, sbp.B, k, alias_replicas=alias)
        for t in dst.locals:
            t.view(torch.uint8).fill_(0xAB)
        sbp.sbp_boxing(src, dst)
        torch.cuda.synchronize()
        want = O.boxing_cast(O.to_locals(T.numpy(), O.S(axis), k), O.S(axis), O.B, "bf16")
        for r in range(k):
            assert np.array_equal(bits(dst.locals[r]), np_bits(want[r], BF16)), f"replica {r}"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(src, sbp.empty_global(shape, BF16, sbp.S(axis), k))       # only S -> B may cast
    assert e.value.name == "SBP_ERR_DTYPE"

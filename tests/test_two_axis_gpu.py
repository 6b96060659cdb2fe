"""Two-axis placements (the paper's multi-dimensional SBP, Section 3.3 and Table 3) on the GPU:
MatMul with one Table 1 rule per placement axis, and boxing of one placement axis at a time,
against the CPU oracle's hierarchical mapping."""
import numpy as np
import pytest
import torch
from helpers import assert_close, bits, np_bits, osig, to_np

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16


def _osigs(sigs):
    return tuple(osig(s) for s in sigs)


def _to_device(arrs, dtype):
    return [torch.from_numpy(np.ascontiguousarray(a)).to(dtype).cuda() for a in arrs]


def _global2(T, sigs, pshape, dtype):
    locs = O.to_locals_2d(to_np(T), _osigs(sigs), pshape)
    return sbp.SbpTensor(tuple(T.shape), dtype, tuple(sigs), _to_device(locs, dtype), pshape)


TABLE3 = [((sbp.S(0), sbp.B), (sbp.B, sbp.S(1))),            # -> (S(0), S(1))
          ((sbp.S(0), sbp.S(1)), (sbp.B, sbp.S(0))),         # -> (S(0), P(sum))
          ((sbp.S(0), sbp.S(0)), (sbp.B, sbp.B)),            # nested data parallelism
          ((sbp.S(1), sbp.B), (sbp.S(0), sbp.S(1))),         # -> (P(sum), S(1))
          ((sbp.B, sbp.B), (sbp.B, sbp.B))]


@pytest.mark.parametrize("xs,ws", TABLE3)
@pytest.mark.parametrize("pshape", [(2, 2), (2, 4), (3, 2)])
@pytest.mark.parametrize("dtype,shape", [(F32, (70, 45, 83)), (BF16, (392, 336, 528)), (F32, (64, 128, 96))])
def test_two_axis_matmul(xs, ws, pshape, dtype, shape):
    M, K, N = shape
    X = dg.uniform(4001, 0, (M, K), -1.0, 1.0, dtype)
    W = dg.uniform(4001, 1, (K, N), -1.0, 1.0, dtype)
    x = _global2(X, xs, pshape, dtype)
    w = _global2(W, ws, pshape, dtype)
    ys = tuple(sbp.sbp_matmul_infer(a, b) for a, b in zip(xs, ws))
    y = sbp.empty_global((M, N), dtype, ys, pshape)
    for t in y.locals:
        t.view(torch.uint8).fill_(0x7F)
    sbp.sbp_matmul(x, w, y)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    xl = [to_np(t) for t in x.locals]
    wl = [to_np(t) for t in w.locals]
    y_sigs, want, Y = O.matmul_locals_2d(xl, _osigs(xs), wl, _osigs(ws), pshape)
    assert y_sigs == _osigs(ys)
    _, absl, _ = O.matmul_locals_2d([np.abs(a) for a in xl], _osigs(xs), [np.abs(a) for a in wl], _osigs(ws), pshape)
    for r in range(pshape[0] * pshape[1]):
        got = to_np(y.locals[r]).astype(np.float64)
        assert got.shape == want[r].shape
        if dtype == F32:
            assert np.all(np.abs(got - want[r]) <= 4.0 * np.sqrt(max(K, 1)) * 2.0 ** -24 * absl[r] + 1e-30)
        else:
            assert_close(got, want[r], 2e-2, 1e-3, f"device {r}")


def test_two_axis_matmul_rejects_what_table1_rejects():
    pshape = (2, 2)
    x = sbp.empty_global((8, 8), F32, (sbp.S(0), sbp.S(1)), pshape)
    w = sbp.empty_global((8, 8), F32, (sbp.B, sbp.B), pshape)
    y = sbp.empty_global((8, 8), F32, (sbp.S(0), sbp.S(1)), pshape)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul(x, w, y)
    assert e.value.name == "SBP_ERR_SIGNATURE"
    w2 = sbp.empty_global((8, 8), F32, (sbp.B, sbp.S(0)), pshape)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul(x, w2, y)                     # deduced (S(0), P(sum)), not (S(0), S(1))
    assert e.value.name == "SBP_ERR_SIGNATURE"


BOX2 = [((sbp.S(0), sbp.P_SUM), (sbp.S(0), sbp.B)),          # all-reduce inside each group
        ((sbp.S(0), sbp.P_SUM), (sbp.S(0), sbp.S(1))),       # reduce-scatter inside each group
        ((sbp.S(0), sbp.S(1)), (sbp.S(0), sbp.B)),           # all-gather inside each group
        ((sbp.S(0), sbp.S(1)), (sbp.S(0), sbp.S(0))),        # nested re-split inside each group
        ((sbp.S(0), sbp.S(1)), (sbp.B, sbp.S(1))),           # all-gather across groups
        ((sbp.P_SUM, sbp.S(1)), (sbp.B, sbp.S(1))),          # all-reduce across groups
        ((sbp.P_SUM, sbp.B), (sbp.S(0), sbp.B)),             # reduce-scatter across groups
        ((sbp.B, sbp.P_SUM), (sbp.S(1), sbp.P_SUM)),         # slicing partial values across groups
        ((sbp.B, sbp.B), (sbp.B, sbp.B))]                    # copy


@pytest.mark.parametrize("src_sigs,dst_sigs", BOX2)
@pytest.mark.parametrize("pshape", [(2, 2), (2, 3), (4, 2)])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_two_axis_boxing_one_axis_at_a_time(src_sigs, dst_sigs, pshape, dtype):
    shape = (66, 120)
    k0, k1 = pshape
    n = k0 * k1
    # source locals: data-movement signatures from one logical tensor; partial axes get seeded shards
    def build(sigs):
        if not any(s.kind in (2, 3) for s in sigs):
            T = dg.normal(4002, 0, shape, 0, 1, dtype)
            return O.to_locals_2d(to_np(T), _osigs(sigs), pshape)
        out = []
        for r in range(n):
            lshape = sbp.sbp_local_shape(shape, tuple(sigs), pshape, r, dtype)
            out.append(to_np(dg.normal(4002, 10 + r, lshape, 0, 1, dtype)))
        if sigs[1].kind not in (2, 3):
            # axis 1 is S or B: devices of a group must hold consistent pieces of one group tensor
            out = []
            for i in range(k0):
                gshape = sbp.sbp_local_shape(shape, sigs[0], k0, i, dtype)
                G = to_np(dg.normal(4002, 50 + i, gshape, 0, 1, dtype))
                out.extend(O.to_locals(G, osig(sigs[1]), k1))
        elif sigs[0].kind == 1:
            # (B, P): every group holds the same partial decomposition
            out = out[:k1] * k0
        return out
    src_np = build(src_sigs)
    src = sbp.SbpTensor(shape, dtype, tuple(src_sigs), _to_device(src_np, dtype), pshape)
    dst = sbp.empty_global(shape, dtype, tuple(dst_sigs), pshape)
    for t in dst.locals:
        t.view(torch.uint8).fill_(0xAB)
    sbp.sbp_boxing(src, dst)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    storage = "f32" if dtype == F32 else "bf16"
    if dst_sigs[1].kind in (2, 3):
        # destination keeps a partial axis 1: the transform acts across groups on each partial j
        want = [None] * n
        for j in range(k1):
            col = O.boxing([src_np[i * k1 + j] for i in range(k0)], osig(src_sigs[0]), osig(dst_sigs[0]), storage)
            for i in range(k0):
                want[i * k1 + j] = col[i]
    else:
        want = O.boxing_2d(src_np, _osigs(src_sigs), _osigs(dst_sigs), pshape, storage)
    for r in range(n):
        assert tuple(dst.locals[r].shape) == tuple(want[r].shape)
        assert np.array_equal(bits(dst.locals[r]), np_bits(want[r], dtype)), f"device {r}"


def test_two_axis_boxing_refusals():
    pshape, shape = (2, 2), (8, 8)
    a = sbp.empty_global(shape, F32, (sbp.S(0), sbp.S(1)), pshape)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(a, sbp.empty_global(shape, F32, (sbp.B, sbp.B), pshape))      # both axes at once
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(a, sbp.empty_global(shape, F32, (sbp.S(1), sbp.S(1)), pshape))  # axis 0 onto axis 1's tensor axis
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    p = sbp.empty_global(shape, F32, (sbp.P_SUM, sbp.P_MAX), pshape)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(p, sbp.empty_global(shape, F32, (sbp.B, sbp.P_MAX), pshape))   # sum over a max
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(a, sbp.empty_global(shape, F32, (sbp.S(0), sbp.S(1)), (4, 1)))
    assert e.value.name == "SBP_ERR_INVALID_ARG"


def test_table3_chain_summa_style():
    """(S(0),B) x (B,S(1)) -> (S(0),S(1)); that result times (B,S(0)) -> (S(0),P(sum)); boxing
    axis 1 P(sum) -> B gives every device of a group its row block of X W1 W2."""
    pshape = (2, 2)
    M, K, N, N2 = 64, 96, 80, 48
    X = dg.uniform(4003, 0, (M, K), -1, 1, F32)
    W1 = dg.uniform(4003, 1, (K, N), -1, 1, F32)
    W2 = dg.uniform(4003, 2, (N, N2), -1, 1, F32)
    x = _global2(X, (sbp.S(0), sbp.B), pshape, F32)
    w1 = _global2(W1, (sbp.B, sbp.S(1)), pshape, F32)
    w2 = _global2(W2, (sbp.B, sbp.S(0)), pshape, F32)
    y1 = sbp.empty_global((M, N), F32, (sbp.S(0), sbp.S(1)), pshape)
    y2 = sbp.empty_global((M, N2), F32, (sbp.S(0), sbp.P_SUM), pshape)
    y3 = sbp.empty_global((M, N2), F32, (sbp.S(0), sbp.B), pshape)
    sbp.sbp_matmul(x, w1, y1)
    sbp.sbp_matmul(y1, w2, y2)
    sbp.sbp_boxing(y2, y3)
    torch.cuda.synchronize()
    want = O.matmul_logical(O.matmul_logical(X.numpy(), W1.numpy()), W2.numpy())
    got = O.from_locals_2d([to_np(t) for t in y3.locals], (O.S0, O.B), pshape)
    assert_close(got, want, 1e-4, 1e-4, "two-axis chain")

"""Local tensors with a leading dimension (windows into larger buffers) and the zero-copy B -> S view
(Table 2: "B -> S" costs nothing; Section 3.2: such a boxing may not move data), through the C ABI on
the GPU, against the oracle.  Every window lives inside a buffer filled with a canary pattern, and the
bytes between the windows are checked after each call."""
import numpy as np
import pytest
import torch
from helpers import assert_close, bits, check_guards, make_global, np_bits, osig, split_cpu, to_np

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16, I64 = torch.float32, torch.bfloat16, torch.int64


def _windows(shape, dtype, sig, k, pad_cols, fill=None):
    """Local tensors of (shape, sig) as windows [rows, cols] inside buffers [rows + 2, cols + pad_cols]
    (one buffer per shard), offset by one row and `pad_cols // 2` columns.  Returns (SbpTensor, buffers)."""
    bufs, locs = [], []
    for r in range(k):
        rows, cols = sbp.sbp_local_shape(shape, sig, k, r, dtype)
        buf = torch.empty((rows + 2, cols + pad_cols), dtype=dtype, device="cuda")
        buf.view(torch.uint8).fill_(0xC3)
        win = buf[1:1 + rows, pad_cols // 2:pad_cols // 2 + cols]
        if fill is not None:
            win.copy_(fill[r].to("cuda"))
        bufs.append(buf)
        locs.append(win)
    return sbp.SbpTensor(shape, dtype, sig, locs), bufs


def _outside_untouched(g, bufs, pad_cols):
    for r, buf in enumerate(bufs):
        rows, cols = g.locals[r].shape
        mask = torch.ones(buf.shape, dtype=torch.bool, device=buf.device)
        mask[1:1 + rows, pad_cols // 2:pad_cols // 2 + cols] = False
        esz = buf.element_size()
        raw = buf.view(torch.uint8).view(buf.shape[0], buf.shape[1], esz)
        assert bool((raw[mask] == 0xC3).all()), f"shard {r}: bytes outside the window were written"


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("src_sig,dst_sig", [(sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0)), (sbp.S(1), sbp.B), (sbp.S(0), sbp.B),
                                             (sbp.B, sbp.S(1)), (sbp.B, sbp.S(0)), (sbp.S(1), sbp.S(1)), (sbp.B, sbp.B),
                                             (sbp.P_SUM, sbp.B), (sbp.P_SUM, sbp.S(0)), (sbp.P_SUM, sbp.S(1)),
                                             (sbp.P_MAX, sbp.B), (sbp.P_SUM, sbp.P_SUM)])
@pytest.mark.parametrize("shape,k,pad", [((96, 160), 4, 16), ((37, 53), 3, 6), ((5, 9), 8, 2)])
def test_boxing_between_windows(dtype, src_sig, dst_sig, shape, k, pad):
    if src_sig.kind in (sbp.P_SUM.kind, sbp.P_MAX.kind):
        src_cpu = [dg.normal(21, r, shape, 0.0, 1.0, dtype) for r in range(k)]
    else:
        src_cpu = split_cpu(dg.normal(21, 0, shape, 0.0, 1.0, dtype), src_sig, k)
    want = O.boxing([to_np(t) for t in src_cpu], osig(src_sig), osig(dst_sig), "bf16" if dtype == BF16 else "f32")
    src, _ = _windows(shape, dtype, src_sig, k, pad, fill=src_cpu)
    dst, dbufs = _windows(shape, dtype, dst_sig, k, pad)
    sbp.sbp_boxing(src, dst)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    for r in range(k):
        assert np.array_equal(bits(dst.locals[r].contiguous()), np_bits(want[r], dtype)), f"shard {r}"
    _outside_untouched(dst, dbufs, pad)
    # mixed: strided source, dense destination
    dense = sbp.empty_global(shape, dtype, dst_sig, k)
    sbp.sbp_boxing(src, dense)
    torch.cuda.synchronize()
    check_guards()
    for r in range(k):
        assert np.array_equal(bits(dense.locals[r]), np_bits(want[r], dtype))


def test_view_b_to_s1_feeds_matmul_without_a_copy():
    """(B, S(1)) -> S(1) with W given once, replicated: the S(1) operand is the column view of the
    replicas, and the S(1) result is written straight into the column blocks of one [M, N] buffer."""
    for dtype, (M, K, N), k in ((BF16, (256, 192, 640), 4), (F32, (64, 128, 96), 2), (BF16, (130, 72, 328), 8)):
        X = dg.normal(31, 0, (M, K), 0.0, 1.0, dtype)
        W = dg.normal(31, 1, (K, N), 0.0, 0.1, dtype)
        x = make_global([X] * k, (M, K), dtype, sbp.B)
        wd = W.to("cuda")
        w_b = sbp.SbpTensor((K, N), dtype, sbp.B, [wd] * k)              # one copy of W, k replicas aliased
        w_s1 = sbp.sbp_view_b_to_s(w_b, 1)
        assert all(t.data_ptr() >= wd.data_ptr() and t.data_ptr() < wd.data_ptr() + wd.numel() * wd.element_size()
                   for t in w_s1.locals if t.numel())
        ybuf = torch.empty((M + 2, N + 8), dtype=dtype, device="cuda")
        ybuf.view(torch.uint8).fill_(0xC3)
        y_full = ybuf[1:1 + M, 8:8 + N]                                     # a window itself
        y_b = sbp.SbpTensor((M, N), dtype, sbp.B, [y_full] * k)
        y_s1 = sbp.sbp_view_b_to_s(y_b, 1)
        ws = torch.empty(max(1, sbp.sbp_matmul_workspace_bytes(x, w_s1, y_s1)), dtype=torch.uint8, device="cuda")
        sbp.sbp_matmul(x, w_s1, y_s1, 0, ws)
        torch.cuda.synchronize()
        sbp.sbp_check_device_errors()
        Y = O.matmul_logical(to_np(X), to_np(W))
        tol = (1e-4, 1e-4) if dtype == F32 else (2e-2, 1e-3)
        assert_close(to_np(y_full.contiguous()), Y, tol[0], tol[1], f"{dtype} [{M},{K}]x[{K},{N}] through views")
        esz = ybuf.element_size()
        raw = ybuf.view(torch.uint8).view(M + 2, N + 8, esz)
        mask = torch.ones((M + 2, N + 8), dtype=torch.bool, device="cuda")
        mask[1:1 + M, 8:8 + N] = False
        assert bool((raw[mask] == 0xC3).all()), "the product wrote outside its window"


def test_view_b_to_s0_feeds_data_parallel_matmul():
    M, K, N, k = 200, 96, 64, 4
    X = dg.normal(32, 0, (M, K), 0.0, 1.0, F32)
    W = dg.normal(32, 1, (K, N), 0.0, 0.1, F32)
    xd = X.to("cuda")
    x_s0 = sbp.sbp_view_b_to_s(sbp.SbpTensor((M, K), F32, sbp.B, [xd] * k), 0)
    assert all(t.is_contiguous() for t in x_s0.locals)                       # row blocks of a dense replica stay dense
    w = make_global([W] * k, (K, N), F32, sbp.B)
    y = sbp.empty_global((M, N), F32, sbp.S(0), k)
    sbp.sbp_matmul(x_s0, w, y, 0, torch.empty(1, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    check_guards()
    want = O.to_locals(O.matmul_logical(to_np(X), to_np(W)), O.S0, k)
    for r in range(k):
        assert_close(to_np(y.locals[r]), want[r], 1e-4, 1e-4, f"shard {r}")


def test_fused_output_boxing_and_transposes_with_leading_dimensions():
    """(S(1), S(0)) -> P(sum) written as B into a window, operands windows too (bf16, tensor cores)."""
    M, K, N, k = 256, 512, 256, 4
    X = dg.normal(33, 0, (M, K), 0.0, 1.0, BF16)
    W = dg.normal(33, 1, (K, N), 0.0, 0.05, BF16)
    x, _ = _windows((M, K), BF16, sbp.S(1), k, 16, fill=split_cpu(X, sbp.S(1), k))
    w, _ = _windows((K, N), BF16, sbp.S(0), k, 8, fill=split_cpu(W, sbp.S(0), k))
    y, ybufs = _windows((M, N), F32, sbp.B, 1, 4)
    y = sbp.SbpTensor((M, N), F32, sbp.B, [y.locals[0]] * k)
    sbp.sbp_matmul(x, w, y, 0, torch.empty(1, dtype=torch.uint8, device="cuda"))
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    assert_close(to_np(y.locals[0].contiguous()), O.matmul_logical(to_np(X), to_np(W)), 2e-2, 1e-3, "fused into a window")
    _outside_untouched(sbp.SbpTensor((M, N), F32, sbp.B, [y.locals[0]]), ybufs, 4)


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_softmax_xent_on_a_column_view_of_replicated_logits(dtype):
    rows, classes, k = 24, 4096 + 264, 4
    Z = dg.normal(34, 0, (rows, classes), 0.0, 2.0, dtype)
    labels = dg.integers(34, 1, (rows,), 0, classes)
    zd = Z.to("cuda")
    logits = sbp.sbp_view_b_to_s(sbp.SbpTensor((rows, classes), dtype, sbp.B, [zd] * k), 1)
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k)
    rmax = sbp.empty_global((rows,), F32, sbp.B, k)
    rsum = sbp.empty_global((rows,), F32, sbp.B, k)
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(logits), dtype=torch.uint8, device="cuda")
    sbp.sbp_softmax_xent(logits, lab, loss, rmax, rsum, ws)
    torch.cuda.synchronize()
    check_guards()
    m, S, ref = O.softmax_xent_logical(to_np(Z), labels.numpy())
    assert np.array_equal(to_np(rmax.locals[0]).astype(np.float64), m)
    assert_close(to_np(rsum.locals[0]), S, 2e-2, 1e-3, "row_sum")
    assert_close(to_np(loss.locals[k - 1]), ref, 2e-2, 1e-3, "loss")
    # backward into the column blocks of one gradient buffer
    gd = torch.full((rows, classes), float("nan"), dtype=dtype, device="cuda")
    grad = sbp.sbp_view_b_to_s(sbp.SbpTensor((rows, classes), dtype, sbp.B, [gd] * k), 1)
    sbp.sbp_softmax_xent_backward(logits, lab, rmax, rsum, grad)
    torch.cuda.synchronize()
    assert_close(to_np(gd), O.softmax_xent_grad(to_np(Z), labels.numpy()), 2e-2, 1e-3, "grad through views")


def test_entry_points_without_leading_dimension_support_refuse_it():
    k, rows, dim = 2, 64, 32
    tbuf = torch.zeros((rows // k, dim + 8), dtype=F32, device="cuda")
    table = sbp.SbpTensor((rows, dim), F32, sbp.S(0), [tbuf[:, :dim]] * k)
    ids = make_global([torch.zeros(8, dtype=I64)] * k, (8,), I64, sbp.B)
    out = sbp.empty_global((8, dim), F32, sbp.B, k)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_embedding(table, ids, out)
    assert e.value.name == "SBP_ERR_UNSUPPORTED" and "dense" in str(e.value)
    # boxing to P(sum) and between different placements take dense tensors only
    src, _ = _windows((16, 24), F32, sbp.S(0), 2, 4, fill=split_cpu(dg.normal(35, 0, (16, 24), 0, 1, F32), sbp.S(0), 2))
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(src, sbp.empty_global((16, 24), F32, sbp.P_SUM, 2))
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_boxing(src, sbp.empty_global((16, 24), F32, sbp.S(0), 4))
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    # a leading dimension below the row length is an invalid descriptor
    bad = src._c()
    bad.local_ld[0] = 3
    import ctypes as C
    d = sbp.empty_global((16, 24), F32, sbp.S(0), 2)._c()
    status = sbp.load_library().sbp_boxing(C.byref(bad), C.byref(d), None)
    assert sbp.load_library().sbp_status_string(status) == b"SBP_ERR_INVALID_ARG"

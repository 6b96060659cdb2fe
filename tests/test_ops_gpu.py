"""Parity of the sharded operators (Table 1 MatMul, class-split softmax cross entropy,
row-split embedding) against the CPU oracle.

Tolerances.  bf16-input / fp32-accumulate MatMul and softmax: |gpu - ref| <= 1e-3 + 2e-2 |ref|
against the fp64 oracle.  fp32 FMA MatMul: |gpu - ref| <= 4 sqrt(K) 2^-24 (|X||W|)_ij (rounding
of a K-term fp32 dot product).  Embedding and every index result: bit-exact."""
import math

import numpy as np
import pytest
import torch
from helpers import assert_close, bits, check_guards, make_global, np_bits, osig, split_cpu, to_np

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16, I64 = torch.float32, torch.bfloat16, torch.int64

TABLE1 = [(sbp.S(0), sbp.B), (sbp.B, sbp.S(1)), (sbp.S(1), sbp.S(0)),
          (sbp.P_SUM, sbp.B), (sbp.B, sbp.P_SUM), (sbp.B, sbp.B)]


def _shard_operand(T, sig, k, seed, tid, dtype):
    """CPU local tensors of logical T under sig.  For P(sum): k-1 seeded shards plus the
    remainder, so that the fixed-order sum of the shards is the logical operand."""
    if sig.kind == 2:
        parts = [dg.uniform(seed, tid + r, T.shape, -1.0, 1.0, dtype) for r in range(k - 1)]
        acc = T.to(torch.float64)
        for p_ in parts:
            acc = acc - p_.to(torch.float64)
        parts.append(acc.to(dtype))
        return parts
    return split_cpu(T, sig, k)


def _swap(sig):
    """Signature of the stored tensor whose transpose carries sig (S(0) <-> S(1))."""
    return sbp.S(1 - sig.axis) if sig.kind == 0 else sig


def _matmul_case(M, K, N, k, dtype, xs, ws, ys=None, flags=0, out_dtype=None, seed=1001, tx=False, tw=False, use_ws=True):
    """xs / ws are the signatures of the operands as they enter the product.  With tx (tw) the
    library is handed the transpose of x (w) -- stored [K,M] ([N,K]) with the swapped signature --
    together with SBP_TRANS_X (SBP_TRANS_W); the oracle sees the untransposed operands."""
    out_dtype = out_dtype or dtype
    X = dg.uniform(seed, 0, (M, K), -1.0, 1.0, dtype)
    W = dg.uniform(seed, 1, (K, N), -1.0, 1.0, dtype)
    xl = _shard_operand(X, xs, k, seed, 10, dtype)
    wl = _shard_operand(W, ws, k, seed, 40, dtype)
    natural = sbp.sbp_matmul_infer(xs, ws)
    ys = ys or natural
    if tx:
        x = make_global([t.t().contiguous() for t in xl], (K, M), dtype, _swap(xs))
        flags |= sbp.SBP_TRANS_X
    else:
        x = make_global(xl, (M, K), dtype, xs)
    if tw:
        w = make_global([t.t().contiguous() for t in wl], (N, K), dtype, _swap(ws))
        flags |= sbp.SBP_TRANS_W
    else:
        w = make_global(wl, (K, N), dtype, ws)
    y = sbp.empty_global((M, N), out_dtype, ys, k)
    for t in y.locals:
        t.view(torch.uint8).fill_(0x7F)
    nbytes = sbp.sbp_matmul_workspace_bytes(x, w, y, flags) if use_ws else 0
    wsbuf = torch.empty(max(nbytes, 1), dtype=torch.uint8, device="cuda") if use_ws else None
    sbp.sbp_matmul(x, w, y, flags, wsbuf)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    check_guards()

    y_sig, y_locals, Y = O.matmul_locals([to_np(t) for t in xl], osig(xs), [to_np(t) for t in wl], osig(ws))
    assert osig(natural) == y_sig
    if flags & sbp.SBP_EPILOGUE_GELU:
        Y = O.gelu(Y)
        y_locals = [O.gelu(a) for a in y_locals]
    if ys != natural:                       # fused boxing: the logical product in the requested signature
        want = O.to_locals(Y, osig(ys), k)
    else:
        want = y_locals
    if dtype == F32:
        # fp32 FMA dot products: |err| <= lambda sqrt(K) u (|X||W|)_ij  (probabilistic bound on
        # recursive summation, lambda = 4, u = 2^-24); the abs-products come from the oracle.
        _, abs_locals, Yabs = O.matmul_locals([np.abs(to_np(t)) for t in xl], osig(xs),
                                              [np.abs(to_np(t)) for t in wl], osig(ws))
        abs_want = O.to_locals(Yabs, osig(ys), k) if ys != natural else abs_locals
        coef = 4.0 * math.sqrt(max(K, 1)) * 2.0 ** -24
    for r in range(k):
        assert tuple(y.locals[r].shape) == tuple(want[r].shape)
        if dtype == F32:
            err = np.abs(to_np(y.locals[r]).astype(np.float64) - want[r])
            assert np.all(err <= coef * abs_want[r] + 1e-30), f"{xs}x{ws}->{ys} shard {r}: {err.max()}"
        else:
            assert_close(to_np(y.locals[r]), want[r], 2e-2, 1e-3, f"{xs}x{ws}->{ys} shard {r}")
    rtol, atol = (1e-4, 1e-4) if dtype == F32 else (2e-2, 1e-3)
    # SBP invariant on the device result: the locals reproduce the logical product
    got = [to_np(t).astype(np.float64) for t in y.locals]
    if ys.kind == 2:
        # each partial carries its own rounding, so the bound scales with sum_r |Y_r|, not |Y|
        mag = sum(np.abs(a) for a in want)
        assert np.all(np.abs(O.reduce_sum_fp64(got) - Y) <= k * atol + rtol * mag), "sum of partials"
    elif ys.kind == 1:
        assert all(np.array_equal(got[0], g) for g in got)
    return y


@pytest.mark.parametrize("xs,ws", TABLE1)
def test_config1_all_six_signatures_fp32(xs, ws):
    """Tiny SBP correctness config: A[64,128] * B[128,96], uniform[-1,1], k = 2."""
    _matmul_case(64, 128, 96, 2, F32, xs, ws)


@pytest.mark.parametrize("xs,ws", TABLE1)
@pytest.mark.parametrize("k", [1, 3, 4])
def test_matmul_signatures_ragged_fp32(xs, ws, k):
    _matmul_case(70, 45, 83, k, F32, xs, ws)


@pytest.mark.parametrize("xs,ws", TABLE1)
def test_matmul_signatures_bf16_small(xs, ws):
    _matmul_case(70, 45, 83, 3, BF16, xs, ws)            # shapes the tensor-core path cannot take
    _matmul_case(256, 256, 256, 2, BF16, xs, ws)


@pytest.mark.parametrize("ys", [sbp.B, sbp.S(0), sbp.S(1)])
@pytest.mark.parametrize("xs,ws", [(sbp.S(1), sbp.S(0)), (sbp.P_SUM, sbp.B), (sbp.B, sbp.P_SUM)])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_matmul_fused_output_boxing(xs, ws, ys, dtype):
    _matmul_case(64, 128, 96, 2, dtype, xs, ws, ys=ys)
    _matmul_case(70, 45, 83, 3, dtype, xs, ws, ys=ys)


def test_matmul_gelu_epilogue_and_f32_out():
    _matmul_case(64, 128, 96, 2, F32, sbp.B, sbp.S(1), flags=sbp.SBP_EPILOGUE_GELU)
    _matmul_case(64, 128, 96, 2, BF16, sbp.B, sbp.S(1), flags=sbp.SBP_EPILOGUE_GELU)
    _matmul_case(64, 128, 96, 2, BF16, sbp.S(1), sbp.S(0), ys=sbp.B, flags=sbp.SBP_EPILOGUE_GELU)
    _matmul_case(64, 128, 96, 2, BF16, sbp.S(1), sbp.S(0), out_dtype=F32)


TRANS = [(True, False), (False, True), (True, True)]


@pytest.mark.parametrize("tx,tw", TRANS)
@pytest.mark.parametrize("xs,ws", TABLE1)
def test_matmul_transposed_operands_fp32(xs, ws, tx, tw):
    """SBP_TRANS_X / SBP_TRANS_W on the FMA kernel: all six signatures, even and ragged shapes."""
    _matmul_case(64, 128, 96, 2, F32, xs, ws, tx=tx, tw=tw)
    _matmul_case(70, 45, 83, 3, F32, xs, ws, tx=tx, tw=tw)


@pytest.mark.parametrize("tx,tw", TRANS)
@pytest.mark.parametrize("xs,ws", TABLE1)
def test_matmul_transposed_operands_tensor_core(xs, ws, tx, tw):
    """The same on the tensor-core kernel: several tiles, K not a multiple of the K-block, ragged
    M and N, k = 2 and 4."""
    _matmul_case(512, 320, 512, 2, BF16, xs, ws, tx=tx, tw=tw)
    _matmul_case(384, 1160, 648, 4, BF16, xs, ws, tx=tx, tw=tw, seed=1011)
    _matmul_case(70, 45, 83, 3, BF16, xs, ws, tx=tx, tw=tw)      # falls to the FMA kernel


@pytest.mark.parametrize("tx,tw", TRANS)
@pytest.mark.parametrize("ys", [sbp.B, sbp.S(0), sbp.S(1)])
def test_matmul_transposed_operands_fused_boxing(ys, tx, tw):
    _matmul_case(64, 128, 96, 2, F32, sbp.S(1), sbp.S(0), ys=ys, tx=tx, tw=tw)
    _matmul_case(512, 1024, 768, 4, BF16, sbp.S(1), sbp.S(0), ys=ys, tx=tx, tw=tw)
    _matmul_case(512, 1024, 768, 4, BF16, sbp.S(1), sbp.S(0), ys=ys, tx=tx, tw=tw, out_dtype=F32)


def test_data_parallel_layer_backward():
    """Data parallelism (Section 3.1): X S(0), W B, Y = X W S(0).  Backward with the same calls:
    dX = dY W^T is (S(0), B) -> S(0); dW = X^T dY is (S(1), S(0)) -> P(sum), asked for as B, i.e.
    with the gradient all-reduce folded into the product.  Checked against the fp64 products."""
    M, K, N, k = 1024, 512, 768, 4
    X = dg.normal(77, 0, (M, K), 0.0, 1.0, BF16)
    W = dg.normal(77, 1, (K, N), 0.0, 0.05, BF16)
    dY = dg.normal(77, 2, (M, N), 0.0, 1.0, BF16)
    x = make_global(split_cpu(X, sbp.S(0), k), (M, K), BF16, sbp.S(0))
    w = make_global([W] * k, (K, N), BF16, sbp.B)
    dy = make_global(split_cpu(dY, sbp.S(0), k), (M, N), BF16, sbp.S(0))
    dx = sbp.empty_global((M, K), BF16, sbp.S(0), k)
    dw = sbp.empty_global((K, N), F32, sbp.B, k)
    sbp.sbp_matmul(dy, w, dx, sbp.SBP_TRANS_W)
    sbp.sbp_matmul(x, dy, dw, sbp.SBP_TRANS_X)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    dX = O.matmul_logical(to_np(dY), to_np(W).T)
    dW = O.matmul_logical(to_np(X).T, to_np(dY))
    for r, a in enumerate(O.to_locals(dX, O.S0, k)):
        assert_close(to_np(dx.locals[r]), a, 2e-2, 1e-3, f"dX shard {r}")
    for r in range(k):
        assert_close(to_np(dw.locals[r]), dW, 2e-2, 1e-3, f"dW replica {r}")


def test_matmul_transposed_operands_are_validated():
    k = 2
    x = sbp.empty_global((128, 64), F32, sbp.S(1), k)        # stored [K,M] = [128,64]: M = 64, K = 128
    w = sbp.empty_global((128, 96), F32, sbp.B, k)
    y = sbp.empty_global((64, 96), F32, sbp.S(0), k)
    sbp.sbp_matmul(x, w, y, sbp.SBP_TRANS_X)                 # (S(0), B) -> S(0) once transposed
    bad = sbp.empty_global((64, 96), F32, sbp.S(1), k)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul(x, w, bad, sbp.SBP_TRANS_X)
    assert e.value.name == "SBP_ERR_SIGNATURE"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul(x, w, y, 0)                           # untransposed: [128,64] x [128,96] does not fit
    assert e.value.name == "SBP_ERR_SHAPE"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul(x, w, y, 64)
    assert e.value.name == "SBP_ERR_INVALID_ARG"


def test_matmul_exact_on_small_integers_and_permutation():
    """Integer-valued operands: every product and sum is exact in fp32, so every signature
    must equal the logical product exactly; a permutation matrix as W permutes columns."""
    M, K, N, k = 32, 64, 48, 4
    X = dg.small_integers(3, 0, (M, K), -4, 5, F32)
    W = dg.small_integers(3, 1, (K, N), -4, 5, F32)
    Y = O.matmul_logical(X.numpy(), W.numpy())
    for xs, ws in [(sbp.S(0), sbp.B), (sbp.B, sbp.S(1)), (sbp.S(1), sbp.S(0)), (sbp.B, sbp.B)]:
        for dtype in (F32, BF16):
            x = make_global(split_cpu(X.to(dtype), xs, k), (M, K), dtype, xs)
            w = make_global(split_cpu(W.to(dtype), ws, k), (K, N), dtype, ws)
            ys = sbp.sbp_matmul_infer(xs, ws)
            y = sbp.empty_global((M, N), F32, ys, k)
            sbp.sbp_matmul(x, w, y)
            torch.cuda.synchronize()
            got = [to_np(t).astype(np.float64) for t in y.locals]
            full = O.reduce_sum_fp64(got) if ys.kind == 2 else O.from_locals(got, osig(ys))
            assert np.array_equal(full, Y)
    perm = torch.randperm(K, generator=torch.Generator().manual_seed(0))
    Pm = torch.zeros(K, K)
    Pm[perm, torch.arange(K)] = 1.0
    x = make_global(split_cpu(X, sbp.S(0), k), (M, K), F32, sbp.S(0))
    w = make_global(split_cpu(Pm, sbp.B, k), (K, K), F32, sbp.B)
    y = sbp.empty_global((M, K), F32, sbp.S(0), k)
    sbp.sbp_matmul(x, w, y)
    torch.cuda.synchronize()
    assert np.array_equal(O.from_locals([to_np(t) for t in y.locals], O.S0), X[:, perm].numpy())


def test_config1_chain_matmul_then_boxing():
    """Config 1 end to end: the six products, then P->B, P->S(0), S(0)->B, S(0)->S(1), B->S(1)
    on the results; and the Y = U V W deferred-reduction chain of Section 3.3."""
    M, K, N, k = 64, 128, 96, 2
    y_p = _matmul_case(M, K, N, k, F32, sbp.S(1), sbp.S(0))
    y_s0 = _matmul_case(M, K, N, k, F32, sbp.S(0), sbp.B)
    y_b = _matmul_case(M, K, N, k, F32, sbp.B, sbp.B)
    for src, dst_sig in [(y_p, sbp.B), (y_p, sbp.S(0)), (y_s0, sbp.B), (y_s0, sbp.S(1)), (y_b, sbp.S(1))]:
        dst = sbp.empty_global((M, N), F32, dst_sig, k)
        sbp.sbp_boxing(src, dst)
        torch.cuda.synchronize()
        want = O.boxing([to_np(t) for t in src.locals], osig(src.sig), osig(dst_sig), "f32")
        for r in range(k):
            assert np.array_equal(bits(dst.locals[r]), np_bits(want[r], F32))
    # U:S(1) V:S(0) W:B  ->  (UV):P(sum), (UV)W:P(sum) without boxing in between, then P->B
    U = dg.uniform(1001, 5, (M, K), -1, 1, F32)
    V = dg.uniform(1001, 6, (K, N), -1, 1, F32)
    Wm = dg.uniform(1001, 7, (N, 40), -1, 1, F32)
    u = make_global(split_cpu(U, sbp.S(1), k), (M, K), F32, sbp.S(1))
    v = make_global(split_cpu(V, sbp.S(0), k), (K, N), F32, sbp.S(0))
    wm = make_global(split_cpu(Wm, sbp.B, k), (N, 40), F32, sbp.B)
    uv = sbp.empty_global((M, N), F32, sbp.P_SUM, k)
    uvw = sbp.empty_global((M, 40), F32, sbp.P_SUM, k)
    out = sbp.empty_global((M, 40), F32, sbp.B, k)
    sbp.sbp_matmul(u, v, uv)
    sbp.sbp_matmul(uv, wm, uvw)
    sbp.sbp_boxing(uvw, out)
    torch.cuda.synchronize()
    want = O.matmul_logical(O.matmul_logical(U.numpy(), V.numpy()), Wm.numpy())
    for t in out.locals:
        assert_close(to_np(t), want, 1e-4, 1e-4, "UVW chain")


# ------------------------------------------------------------------ softmax cross entropy

def _xent_case(rows, classes, k, dtype, sigma=1.0, seed=1004, alias=False, with_stats=True, labels=None):
    Z = dg.normal(seed, 0, (rows, classes), 0.0, sigma, dtype)
    if labels is None:
        labels = dg.integers(seed, 1, (rows,), 0, classes)
    logits = make_global(split_cpu(Z, sbp.S(1), k), (rows, classes), dtype, sbp.S(1))
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k, alias_replicas=alias)
    rmax = sbp.empty_global((rows,), F32, sbp.B, k) if with_stats else None
    rsum = sbp.empty_global((rows,), F32, sbp.B, k) if with_stats else None
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(logits), dtype=torch.uint8, device="cuda")
    sbp.sbp_softmax_xent(logits, lab, loss, rmax, rsum, ws)
    torch.cuda.synchronize()
    check_guards()
    m, Ssum, ref = O.softmax_xent_logical(to_np(Z), labels.numpy())
    for t in loss.locals:
        assert_close(to_np(t), ref, 2e-2, 1e-3, "loss")
    if with_stats:
        for t in rmax.locals:
            assert np.array_equal(to_np(t).astype(np.float64), m)          # the max is exact
        for t in rsum.locals:
            assert_close(to_np(t), Ssum, 2e-2, 1e-3, "row_sum")
    return to_np(loss.locals[0]), ref


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_softmax_xent_parity(dtype, k):
    _xent_case(16, 4096, k, dtype)
    _xent_case(5, 1000, k, dtype)                    # ragged: element-wise path
    _xent_case(3, 70000, k, dtype, sigma=0.226)      # several column chunks per shard


def test_softmax_xent_tight_accuracy_and_shard_invariance():
    """fp32 partial sums of exp: far inside the stated tolerance, and independent of k."""
    ref_losses = []
    for k in (1, 2, 4, 8):
        got, ref = _xent_case(8, 32768, k, BF16, sigma=0.226, seed=55)
        assert np.all(np.abs(got - ref) <= 2e-5 * np.abs(ref))
        ref_losses.append(got)
    for g in ref_losses[1:]:
        assert np.all(np.abs(g - ref_losses[0]) <= 1e-6 * np.abs(ref_losses[0]) + 1e-6)


def test_softmax_xent_closed_forms_and_edges():
    rows, classes, k = 4, 512, 4
    Z = torch.full((rows, classes), 2.5, dtype=BF16)
    labels = torch.tensor([0, 127, 128, 511])
    logits = make_global(split_cpu(Z, sbp.S(1), k), (rows, classes), BF16, sbp.S(1))
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k)
    rsum = sbp.empty_global((rows,), F32, sbp.B, k)
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(logits), dtype=torch.uint8, device="cuda")
    sbp.sbp_softmax_xent(logits, lab, loss, None, rsum, ws)
    torch.cuda.synchronize()
    assert np.allclose(to_np(loss.locals[0]), math.log(classes), rtol=1e-6)        # all-equal logits: ln C
    assert np.allclose(to_np(rsum.locals[0]), classes, rtol=1e-6)
    # labels on shard boundaries, first and last class; aliasing of replicas; no stats
    lab_edge = torch.tensor([0, 1023, 1024, 4095, 2047, 2048, 3071, 3072])
    _xent_case(8, 4096, 4, BF16, labels=lab_edge, alias=True, with_stats=False)
    # k > classes: some shards hold no class at all
    _xent_case(4, 3, 4, F32)
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_softmax_xent(logits, lab, loss, None, rsum, ws[:16])
    assert e.value.name == "SBP_ERR_WORKSPACE"


# ------------------------------------------------------------------ embedding

def _emb_case(rows, dim, ids, k, dtype, fused, alias=False, table=None):
    if table is None:
        table = dg.uniform(1005, 0, (rows, dim), -0.05, 0.05, dtype)
    tab = make_global(split_cpu(table, sbp.S(0), k), (rows, dim), dtype, sbp.S(0))
    idt = make_global([ids] * k, tuple(ids.shape), I64, sbp.B)
    out_shape = tuple(ids.shape) + (dim,)
    out = sbp.empty_global(out_shape, dtype, sbp.B if fused else sbp.P_SUM, k, alias_replicas=alias)
    for t in out.locals:
        t.view(torch.uint8).fill_(0x5A)
    oob = torch.zeros(1, dtype=torch.int32, device="cuda")
    sbp.sbp_embedding(tab, idt, out, oob)
    torch.cuda.synchronize()
    check_guards()
    tnp = to_np(table)
    if fused:
        want = O.embedding_logical(tnp, ids.numpy())
        if k > 1:
            want = want + np.float32(0.0)        # what P(sum)->B of the partials gives for -0.0
        for t in out.locals:
            assert np.array_equal(bits(t), np_bits(want, dtype))
    else:
        parts = O.embedding_partials(O.to_locals(tnp, O.S0, k), ids.numpy())
        for r in range(k):
            assert np.array_equal(bits(out.locals[r]), np_bits(parts[r], dtype)), f"shard {r}"
    return out, int(oob.item())


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("k", [1, 2, 3, 8])
@pytest.mark.parametrize("dtype,dim", [(F32, 128), (F32, 33), (BF16, 64), (BF16, 7)])
def test_embedding_parity(fused, k, dtype, dim):
    rows = 1000
    ids = dg.zipf_ids(1005, 1, (97, 26), 1024).clamp_(max=rows - 1)
    _emb_case(rows, dim, ids, k, dtype, fused)


def test_embedding_closed_forms_and_edges():
    rows, dim, k = 256, 128, 4
    ids = torch.arange(rows).reshape(rows, 1)
    out, _ = _emb_case(rows, dim, ids, k, F32, True)
    table = dg.uniform(1005, 0, (rows, dim), -0.05, 0.05, F32)
    assert np.array_equal(to_np(out.locals[0]).reshape(rows, dim), table.numpy())    # arange ids: the table itself
    ids1 = torch.full((16, 2), 70)                                                   # all in shard 1
    outp, _ = _emb_case(rows, dim, ids1, k, F32, False)
    assert all(not outp.locals[r].any().item() for r in (0, 2, 3)) and outp.locals[1].any().item()
    bad = torch.tensor([[-1, rows, 5, 1 << 40]])
    _, oob = _emb_case(rows, dim, bad, k, F32, True)
    assert oob == 3
    _, oob = _emb_case(rows, dim, bad, k, F32, False)
    assert oob == 3
    _emb_case(rows, dim, ids1, k, F32, True, alias=True)
    # single destination (aliased replicas): the kernel that resolves a lookup's row address once, a
    # chunk ahead -- out-of-range ids give zero rows and are counted once each, also across chunks
    _, oob = _emb_case(rows, dim, bad, k, F32, True, alias=True)
    assert oob == 3
    many = dg.integers(77, 0, (4096, 3), 0, rows).cpu()
    many[5, 1], many[700, 0], many[2049, 2], many[4095, 2] = -7, rows, 1 << 33, rows + 1
    _, oob = _emb_case(rows, dim, many, k, F32, True, alias=True)
    assert oob == 4
    _emb_case(3, 16, torch.tensor([0, 1, 2, 2, 0]), 8, F32, False)                   # k > rows
    _emb_case(3, 16, torch.tensor([0, 1, 2, 2, 0]), 8, F32, True)


def test_embedding_fused_equals_unfused_plus_boxing_with_negative_zero():
    rows, dim, k = 64, 32, 4
    table = dg.uniform(1005, 9, (rows, dim), -0.05, 0.05, F32)
    table[5, 3] = -0.0
    table[40, 0] = -0.0
    ids = torch.tensor([[5, 40, 7], [63, 5, 0]])
    fused, _ = _emb_case(rows, dim, ids, k, F32, True, table=table)
    parts, _ = _emb_case(rows, dim, ids, k, F32, False, table=table)
    boxed = sbp.empty_global(tuple(ids.shape) + (dim,), F32, sbp.B, k)
    sbp.sbp_boxing(parts, boxed)
    torch.cuda.synchronize()
    for a, b in zip(fused.locals, boxed.locals):
        assert np.array_equal(bits(a), bits(b))


# ------------------------------------------------------------------ tensor-core MatMul path

@pytest.mark.parametrize("xs,ws", TABLE1)
@pytest.mark.parametrize("k", [2, 3])
def test_matmul_tensor_core_multi_tile_ragged(xs, ws, k):
    """Shapes that span several 128 x 256 tiles and 64-deep K-blocks, with ragged edges in
    every dimension (all leading dimensions stay multiples of 8 elements)."""
    _matmul_case(392, 336, 528, k, BF16, xs, ws, seed=2001)


@pytest.mark.parametrize("ys", [sbp.B, sbp.S(0), sbp.S(1)])
@pytest.mark.parametrize("xs,ws", [(sbp.S(1), sbp.S(0)), (sbp.P_SUM, sbp.B)])
def test_matmul_tensor_core_fused_boxing(xs, ws, ys):
    _matmul_case(392, 336, 528, 4, BF16, xs, ws, ys=ys, seed=2002)
    _matmul_case(256, 1024, 512, 8, BF16, xs, ws, ys=ys, seed=2003, out_dtype=F32)


def test_matmul_tensor_core_gelu_and_many_tiles():
    # more tiles than SMs, so every CTA walks several tiles and both accumulators
    _matmul_case(2048, 256, 4096, 8, BF16, sbp.B, sbp.S(1), flags=sbp.SBP_EPILOGUE_GELU, seed=2004)
    _matmul_case(2048, 512, 2048, 4, BF16, sbp.S(0), sbp.B, seed=2005)
    _matmul_case(1024, 2048, 1024, 8, BF16, sbp.S(1), sbp.S(0), seed=2006)


def test_mlp_block_small_against_oracle():
    """The Megatron-style block at reduced size: B x S(1) -> S(1) with GeLU, S(1) x S(0) ->
    P(sum) written directly as B.  Hidden state is stored as bf16 between the products."""
    k, M, H, Fd = 8, 512, 256, 1024
    X = dg.normal(1003, 0, (M, H), 0.0, 1.0, BF16)
    W1 = dg.normal(1003, 1, (H, Fd), 0.0, 0.02, BF16)
    W2 = dg.normal(1003, 2, (Fd, H), 0.0, 0.02, BF16)
    x = make_global(split_cpu(X, sbp.B, k), (M, H), BF16, sbp.B)
    w1 = make_global(split_cpu(W1, sbp.S(1), k), (H, Fd), BF16, sbp.S(1))
    w2 = make_global(split_cpu(W2, sbp.S(0), k), (Fd, H), BF16, sbp.S(0))
    h = sbp.empty_global((M, Fd), BF16, sbp.S(1), k)
    y = sbp.empty_global((M, H), BF16, sbp.B, k)
    sbp.sbp_matmul(x, w1, h, sbp.SBP_EPILOGUE_GELU)
    sbp.sbp_matmul(h, w2, y)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    want = O.mlp_logical(to_np(X), to_np(W1), to_np(W2))
    for t in y.locals:
        assert_close(to_np(t), want, 2e-2, 1e-3, "MLP block")
    # the unfused route (fp32 partials, then P(sum) -> B) gives the same values
    yp = sbp.empty_global((M, H), F32, sbp.P_SUM, k)
    yb = sbp.empty_global((M, H), F32, sbp.B, k)
    sbp.sbp_matmul(h, w2, yp)
    sbp.sbp_boxing(yp, yb)
    torch.cuda.synchronize()
    assert_close(to_np(yb.locals[0]), want, 2e-2, 1e-3, "MLP block, unfused")


def test_classifier_chain_small_against_oracle():
    """Features B x classifier weight S(1) -> bf16 logits S(1) -> split softmax cross entropy."""
    k, rows, feat, classes = 8, 64, 512, 16384
    Fm = dg.normal(1004, 0, (rows, feat), 0.0, 1.0, BF16)
    W = dg.normal(1004, 2, (feat, classes), 0.0, 0.01, BF16)
    labels = dg.integers(1004, 1, (rows,), 0, classes)
    f = make_global(split_cpu(Fm, sbp.B, k), (rows, feat), BF16, sbp.B)
    w = make_global(split_cpu(W, sbp.S(1), k), (feat, classes), BF16, sbp.S(1))
    z = sbp.empty_global((rows, classes), BF16, sbp.S(1), k)
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k)
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(z), dtype=torch.uint8, device="cuda")
    sbp.sbp_matmul(f, w, z)
    sbp.sbp_softmax_xent(z, lab, loss, None, None, ws)
    torch.cuda.synchronize()
    Z = O.matmul_logical(to_np(Fm), to_np(W))
    _, _, ref = O.softmax_xent_logical(Z, labels.numpy())
    assert_close(to_np(loss.locals[0]), ref, 2e-2, 1e-3, "classifier chain loss")
    zl = O.to_locals(Z, O.S1, k)
    for r in range(k):
        assert_close(to_np(z.locals[r]), zl[r], 2e-2, 1e-3, f"logits shard {r}")


# ------------------------------------------------------------------ fused classifier -> softmax cross entropy

def _fused_classifier_case(rows, feat, classes, k, seed, w_std=0.05, alias=False):
    Fm = dg.normal(seed, 0, (rows, feat), 0.0, 1.0, BF16)
    W = dg.normal(seed, 2, (feat, classes), 0.0, w_std, BF16)
    labels = dg.integers(seed, 1, (rows,), 0, classes)
    f = make_global(split_cpu(Fm, sbp.B, k), (rows, feat), BF16, sbp.B)
    w = make_global(split_cpu(W, sbp.S(1), k), (feat, classes), BF16, sbp.S(1))
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k, alias_replicas=alias)
    rmax = sbp.empty_global((rows,), F32, sbp.B, k)
    rsum = sbp.empty_global((rows,), F32, sbp.B, k)
    for g in (loss, rmax, rsum):
        for t in g.locals:
            t.fill_(float("nan"))
    ws = torch.empty(sbp.sbp_matmul_softmax_xent_workspace_bytes(f, w), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)                                     # NaN patterns: every partial that is read must be written
    sbp.sbp_matmul_softmax_xent(f, w, lab, loss, rmax, rsum, ws)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    check_guards()
    Z = O.matmul_logical(to_np(Fm), to_np(W))
    m, S, ref = O.softmax_xent_logical(Z, labels.numpy())
    for t in loss.locals:
        assert_close(to_np(t), ref, 2e-2, 1e-3, "fused loss")
    for t in rmax.locals:
        assert_close(to_np(t), m, 2e-2, 1e-3, "fused row_max")
    for t in rsum.locals:
        assert_close(to_np(t), S, 2e-2, 1e-3, "fused row_sum")
    # fp32 accumulation straight into the softmax: far tighter than the stated bar
    assert np.all(np.abs(to_np(loss.locals[0]) - ref) <= 1e-4 * np.maximum(np.abs(ref), 1.0))
    # the backward, again without stored logits: softmax - onehot, S(1), in both result dtypes
    want = O.to_locals(O.softmax_xent_grad(Z, labels.numpy()), O.S1, k)
    for gdt in (BF16, F32):
        grad = sbp.empty_global((rows, classes), gdt, sbp.S(1), k)
        for t in grad.locals:
            t.fill_(float("nan"))
        sbp.sbp_matmul_softmax_xent_backward(f, w, lab, rmax, rsum, grad)
        torch.cuda.synchronize()
        sbp.sbp_check_device_errors()
        check_guards()
        for r in range(k):
            assert tuple(grad.locals[r].shape) == tuple(want[r].shape)
            assert_close(to_np(grad.locals[r]), want[r], 2e-2, 1e-3, f"fused grad shard {r}")
        if gdt == F32:      # every row of softmax - onehot sums to zero; fp32 results are far tighter than the bar
            full = O.from_locals([to_np(t).astype(np.float64) for t in grad.locals], O.S1)
            assert np.all(np.abs(full.sum(axis=1)) <= 1e-3)
            assert np.all(np.abs(full - O.softmax_xent_grad(Z, labels.numpy())) <= 1e-5)
    return to_np(loss.locals[0])


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_fused_classifier_parity_and_shard_invariance(k):
    a = _fused_classifier_case(64, 512, 16384, k, seed=3001)
    b = _fused_classifier_case(64, 512, 16384, 1, seed=3001) if k > 1 else a
    assert np.all(np.abs(a - b) <= 1e-5 * np.abs(b) + 1e-5)


def test_fused_classifier_ragged_shapes_and_edges():
    _fused_classifier_case(300, 200, 4960, 4, seed=3002)        # ragged rows, K tail, 1240 classes per shard
    _fused_classifier_case(33, 72, 960, 8, seed=3003)           # 120 classes per shard: one partial chunk each
    _fused_classifier_case(700, 64, 64, 4, seed=3004, alias=True)   # 16 classes per shard, many row tiles
    rows, feat, classes, k = 16, 64, 1000, 3                     # 334 / 333 classes per shard: not multiples of 8
    f = sbp.empty_global((rows, feat), BF16, sbp.B, k)
    w = sbp.empty_global((feat, classes), BF16, sbp.S(1), k)
    lab = make_global([torch.zeros(rows, dtype=I64)] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k)
    ws = torch.empty(sbp.sbp_matmul_softmax_xent_workspace_bytes(f, w), dtype=torch.uint8, device="cuda")
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul_softmax_xent(f, w, lab, loss, None, None, ws)
    assert e.value.name == "SBP_ERR_UNSUPPORTED"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_matmul_softmax_xent(f, w, lab, loss, None, None, ws[:64])
    assert e.value.name in ("SBP_ERR_WORKSPACE", "SBP_ERR_UNSUPPORTED")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("k", [1, 2, 3, 8])
@pytest.mark.parametrize("dtype,dim", [(F32, 128), (F32, 36), (BF16, 64), (BF16, 10)])
def test_embedding_table_split_on_hidden_axis(fused, k, dtype, dim):
    rows = 500
    table = dg.uniform(1005, 3, (rows, dim), -0.05, 0.05, dtype)
    ids = dg.zipf_ids(1005, 4, (41, 26), 512).clamp_(max=rows - 1)
    ids[0, 0], ids[1, 1] = -3, rows                              # two ids out of range
    tab = make_global(split_cpu(table, sbp.S(1), k), (rows, dim), dtype, sbp.S(1))
    idt = make_global([ids] * k, tuple(ids.shape), I64, sbp.B)
    out = sbp.empty_global(tuple(ids.shape) + (dim,), dtype, sbp.B if fused else sbp.S(2), k)
    for t in out.locals:
        t.view(torch.uint8).fill_(0x5A)
    oob = torch.zeros(1, dtype=torch.int32, device="cuda")
    sbp.sbp_embedding(tab, idt, out, oob)
    torch.cuda.synchronize()
    assert int(oob.item()) == 2
    parts = O.embedding_hidden_split(O.to_locals(to_np(table), O.S1, k), ids.numpy())
    if fused:
        want = O.from_locals(parts, O.S(2))
        for t in out.locals:
            assert np.array_equal(bits(t), np_bits(want, dtype))
    else:
        for r in range(k):
            assert tuple(out.locals[r].shape) == tuple(parts[r].shape)
            assert np.array_equal(bits(out.locals[r]), np_bits(parts[r], dtype)), f"shard {r}"


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("k", [1, 4, 8])
@pytest.mark.parametrize("rows,classes", [(16, 4096), (5, 1000), (3, 70000)])
def test_softmax_xent_backward_parity(dtype, k, rows, classes):
    Z = dg.normal(1004, 5, (rows, classes), 0.0, 1.0, dtype)
    labels = dg.integers(1004, 6, (rows,), 0, classes)
    logits = make_global(split_cpu(Z, sbp.S(1), k), (rows, classes), dtype, sbp.S(1))
    lab = make_global([labels] * k, (rows,), I64, sbp.B)
    loss = sbp.empty_global((rows,), F32, sbp.B, k)
    rmax = sbp.empty_global((rows,), F32, sbp.B, k)
    rsum = sbp.empty_global((rows,), F32, sbp.B, k)
    grad = sbp.empty_global((rows, classes), dtype, sbp.S(1), k)
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(logits), dtype=torch.uint8, device="cuda")
    sbp.sbp_softmax_xent(logits, lab, loss, rmax, rsum, ws)
    sbp.sbp_softmax_xent_backward(logits, lab, rmax, rsum, grad)
    torch.cuda.synchronize()
    want = O.to_locals(O.softmax_xent_grad(to_np(Z), labels.numpy()), O.S1, k)
    for r in range(k):
        assert tuple(grad.locals[r].shape) == tuple(want[r].shape)
        assert_close(to_np(grad.locals[r]), want[r], 2e-2, 1e-3, f"grad shard {r}")
    if dtype == F32:        # far tighter in fact, and every row sums to zero
        full = O.from_locals([to_np(t).astype(np.float64) for t in grad.locals], O.S1)
        assert np.all(np.abs(full - O.softmax_xent_grad(to_np(Z), labels.numpy())) <= 1e-6)
        assert np.all(np.abs(full.sum(axis=1)) <= 1e-4)


@pytest.mark.parametrize("k", [1, 3, 8])
@pytest.mark.parametrize("rows,dim,hot", [(1000, 128, False), (37, 8, True), (5, 4, True)])
def test_embedding_backward_parity(k, rows, dim, hot):
    """grad_table (S(0)) = scatter-add of grad_out over the ids; fp32 atomic adds in no fixed order,
    so the bound is the rounding of an n-term fp32 sum: n u sum|terms| (u = 2^-24)."""
    n_rows_ids = 16 if not hot else rows                           # hot: every id lands on few rows
    ids = dg.zipf_ids(1005, 7, (97, 26), 1024).clamp_(max=n_rows_ids - 1 if hot else rows - 1)
    ids[3, 3] = -1
    G = dg.normal(1005, 8, (97, 26, dim), 0.0, 1.0, F32)
    go = make_global([G] * k, (97, 26, dim), F32, sbp.B)
    idt = make_global([ids] * k, (97, 26), I64, sbp.B)
    gt = sbp.empty_global((rows, dim), F32, sbp.S(0), k)
    for t in gt.locals:
        t.fill_(float("nan"))                                      # the kernel must write everything
    oob = torch.zeros(1, dtype=torch.int32, device="cuda")
    sbp.sbp_embedding_backward(go, idt, gt, oob)
    torch.cuda.synchronize()
    assert int(oob.item()) == 1
    want = O.embedding_grad_table(G.numpy(), ids.numpy(), rows)
    mag = O.embedding_grad_table(np.abs(G.numpy()), ids.numpy(), rows)
    counts = O.embedding_grad_table(np.ones((97, 26, 1)), ids.numpy(), rows)
    got = O.from_locals([to_np(t).astype(np.float64) for t in gt.locals], O.S0)
    assert got.shape == want.shape
    assert np.all(np.abs(got - want) <= counts * 2.0 ** -24 * mag + 1e-30)
    assert np.all(got[counts[:, 0] == 0] == 0.0)


@pytest.mark.parametrize("k,rows,dim,s,batch", [(8, 100003, 8, 1.05, 24000), (3, 2000, 132, 1.3, 300)])
def test_embedding_backward_large_batch(k, rows, dim, s, batch):
    """A batch large enough for the 1024-lookup chunks (and, with dim = 132, rows wider than one
    pass of a warp): same bound as above."""
    ids = dg.zipf_ids(1005, 17, (batch, 26), rows, s)
    ids[5, 7] = rows
    ids[batch - 1, 25] = -3
    G = dg.normal(1005, 18, (batch, 26, dim), 0.0, 1.0, F32)
    go = make_global([G] * k, (batch, 26, dim), F32, sbp.B)
    idt = make_global([ids] * k, (batch, 26), I64, sbp.B)
    gt = sbp.empty_global((rows, dim), F32, sbp.S(0), k)
    for t in gt.locals:
        t.fill_(float("nan"))
    oob = torch.zeros(1, dtype=torch.int32, device="cuda")
    sbp.sbp_embedding_backward(go, idt, gt, oob)
    torch.cuda.synchronize()
    assert int(oob.item()) == 2
    want = O.embedding_grad_table(G.numpy(), ids.numpy(), rows)
    mag = O.embedding_grad_table(np.abs(G.numpy()), ids.numpy(), rows)
    counts = O.embedding_grad_table(np.ones((batch, 26, 1)), ids.numpy(), rows)
    got = O.from_locals([to_np(t).astype(np.float64) for t in gt.locals], O.S0)
    assert np.all(np.abs(got - want) <= counts * 2.0 ** -24 * mag + 1e-30)
    assert np.all(got[counts[:, 0] == 0] == 0.0)


def test_repeated_tensor_core_product_encodes_no_new_descriptors():
    """The copy-engine descriptors of a product are kept: calling it again on the same buffers
    re-uses all of them (what a training loop does every step)."""
    M, K, N, k = 256, 256, 512, 4
    X = dg.normal(77, 0, (M, K), 0.0, 1.0, BF16)
    W = dg.normal(77, 1, (K, N), 0.0, 0.1, BF16)
    x = make_global([X] * k, (M, K), BF16, sbp.B)
    w = make_global(split_cpu(W, sbp.S(1), k), (K, N), BF16, sbp.S(1))
    y = sbp.empty_global((M, N), BF16, sbp.S(1), k)
    ws = torch.empty(1, dtype=torch.uint8, device="cuda")
    sbp.sbp_matmul(x, w, y, 0, ws)
    reused0, encoded0 = sbp.sbp_tensor_map_stats()
    assert encoded0 > 0                                   # this shape takes the tensor-core path
    sbp.sbp_matmul(x, w, y, 0, ws)
    reused1, encoded1 = sbp.sbp_tensor_map_stats()
    assert encoded1 == encoded0 and reused1 >= reused0 + 3 * k
    torch.cuda.synchronize()
    check_guards()
    want = O.to_locals(O.matmul_logical(to_np(X), to_np(W)), O.S1, k)
    for r in range(k):
        assert_close(to_np(y.locals[r]), want[r], 2e-2, 1e-3, f"shard {r}")


UNALIGNED = [  # M, K, N, k: shard widths / contraction lengths that are not multiples of 8 elements
    (130, 70, 333, 3), (96, 136, 2 * 333, 2), (257, 64, 90, 4)]


@pytest.mark.parametrize("xs,ws,ys", [(sbp.S(0), sbp.B, None), (sbp.B, sbp.S(1), None), (sbp.S(1), sbp.S(0), None),
                                      (sbp.S(1), sbp.S(0), sbp.B), (sbp.S(1), sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0), sbp.S(0)),
                                      (sbp.P_SUM, sbp.B, None), (sbp.B, sbp.B, None)])
@pytest.mark.parametrize("shape", UNALIGNED)
def test_matmul_bf16_unaligned_shapes_stay_on_tensor_cores(xs, ws, ys, shape):
    """bf16 operands whose shard widths miss the copy engine's 16-byte rules: with a workspace they
    are repacked and multiplied on the tensor cores (descriptors get encoded), without one the FMA
    kernel takes them; both meet the stated tolerance against the oracle."""
    M, K, N, k = shape
    before = sum(sbp.sbp_tensor_map_stats())
    _matmul_case(M, K, N, k, BF16, xs, ws, ys=ys, seed=1201)
    assert sum(sbp.sbp_tensor_map_stats()) > before, "the repacked product did not reach the tensor-core kernel"
    before = sum(sbp.sbp_tensor_map_stats())
    _matmul_case(M, K, N, k, BF16, xs, ws, ys=ys, seed=1201, use_ws=False)
    assert sum(sbp.sbp_tensor_map_stats()) == before, "without a workspace the FMA kernel is the one that runs"


@pytest.mark.parametrize("tx,tw", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("xs,ws,ys", [(sbp.S(0), sbp.B, None), (sbp.B, sbp.S(1), None), (sbp.S(1), sbp.S(0), sbp.S(0)),
                                      (sbp.S(1), sbp.S(0), sbp.S(1)), (sbp.S(1), sbp.S(0), sbp.B)])
def test_matmul_bf16_unaligned_transposed_operands(xs, ws, ys, tx, tw):
    for M, K, N, k in UNALIGNED[:2]:
        _matmul_case(M, K, N, k, BF16, xs, ws, ys=ys, seed=1202, tx=tx, tw=tw)
        _matmul_case(M, K, N, k, BF16, xs, ws, ys=ys, seed=1202, tx=tx, tw=tw, out_dtype=F32)


@pytest.mark.parametrize("tx", [False, True])
def test_matmul_fused_split_results_walk_their_groups_as_one_grid(tx):
    """A P(sum) product written as S(0) / S(1): the row (column) blocks of the result are separate
    output groups that the tensor-core kernel walks as one grid, panels of eight m-tiles running
    across group boundaries.  Several tiles per group, ragged groups, more tiles than CTA pairs,
    groups of one row and empty groups."""
    _matmul_case(2600, 192, 1100, 3, BF16, sbp.S(1), sbp.S(0), ys=sbp.S(0), seed=2101, tx=tx)
    _matmul_case(700, 192, 2600, 3, BF16, sbp.S(1), sbp.S(0), ys=sbp.S(1), seed=2102, tx=tx)
    _matmul_case(5, 128, 520, 8, BF16, sbp.S(1), sbp.S(0), ys=sbp.S(0), seed=2103, tx=tx)
    _matmul_case(520, 128, 5, 8, BF16, sbp.S(1), sbp.S(0), ys=sbp.S(1), seed=2104, tx=tx, out_dtype=F32)
    _matmul_case(4096, 64, 4864, 8, BF16, sbp.P_SUM, sbp.B, ys=sbp.S(0), seed=2105)

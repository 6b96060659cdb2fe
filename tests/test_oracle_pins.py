"""Pins for the CPU oracle: every oracle function is checked against something other
than itself -- the paper's tables (text fixtures), hand-worked values, brute force in
pure Python loops on tiny inputs, closed forms, and independent library routines."""
import itertools
import math

import numpy as np
import pytest
import torch
from conftest import read_golden

import sbp_datagen as dg
from oracle import sbp_oracle as O

S0, S1, B, PSUM, PMAX = O.S0, O.S1, O.B, O.PSUM, O.PMAX


def _parse_sig(tok):
    return {"S(0)": S0, "S(1)": S1, "B": B, "P(sum)": PSUM}[tok]


# ---------------------------------------------------------------- Section 3.1 mapping

def test_fig3_two_device_example():
    rows = {r[0]: np.array([float(v) for v in r[1:]]) for r in read_golden("fig3_two_device_example.txt")}
    T = rows["T"].reshape(2, 2)
    s0 = O.to_locals(T, S0, 2)
    s1 = O.to_locals(T, S1, 2)
    b = O.to_locals(T, B, 2)
    assert np.array_equal(s0[0].ravel(), rows["S0_dev0"]) and np.array_equal(s0[1].ravel(), rows["S0_dev1"])
    assert np.array_equal(s1[0].ravel(), rows["S1_dev0"]) and np.array_equal(s1[1].ravel(), rows["S1_dev1"])
    assert np.array_equal(b[0].ravel(), rows["B_dev0"]) and np.array_equal(b[1].ravel(), rows["B_dev1"])
    assert s0[0].shape == (1, 2) and s1[0].shape == (2, 1)
    p = [rows["P_dev0"].reshape(2, 2), rows["P_dev1"].reshape(2, 2)]
    assert np.array_equal(O.from_locals(p, PSUM, "f32"), T.astype(np.float32))


@pytest.mark.parametrize("n,k,expect", [
    (10, 4, [(0, 3), (3, 3), (6, 2), (8, 2)]),
    (8, 4, [(0, 2), (2, 2), (4, 2), (6, 2)]),
    (3, 4, [(0, 1), (1, 1), (2, 1), (3, 0)]),
    (7, 1, [(0, 7)]),
    (0, 3, [(0, 0), (0, 0), (0, 0)]),
])
def test_balanced_split_hand_values(n, k, expect):
    assert O.balanced_split(n, k) == expect


@pytest.mark.parametrize("n", [0, 1, 5, 17, 64, 1000])
@pytest.mark.parametrize("k", [1, 2, 3, 4, 8, 16])
def test_balanced_split_properties(n, k):
    parts = O.balanced_split(n, k)
    lens = [ln for _, ln in parts]
    assert sum(lens) == n and max(lens) - min(lens) <= 1
    assert lens == sorted(lens, reverse=True)                   # bigger pieces first
    pos = 0
    for s, ln in parts:
        assert s == pos
        pos += ln


def _brute_split_locals(T, axis, k):
    """Pure-python placement: walk every element of T and drop it into its shard."""
    shape = T.shape
    n = shape[axis]
    base, rem = divmod(n, k)
    lens = [base + (1 if r < rem else 0) for r in range(k)]
    starts = [sum(lens[:r]) for r in range(k)]
    outs = [np.full(shape[:axis] + (lens[r],) + shape[axis + 1:], -1, dtype=T.dtype) for r in range(k)]
    for idx in itertools.product(*[range(s) for s in shape]):
        a = idx[axis]
        r = max(rr for rr in range(k) if starts[rr] <= a and lens[rr] > 0)
        loc = list(idx)
        loc[axis] = a - starts[r]
        outs[r][tuple(loc)] = T[idx]
    return outs


@pytest.mark.parametrize("shape", [(6, 8), (5, 7), (3, 4, 5), (2, 3, 4, 5), (7,)])
@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_split_matches_brute_force_and_round_trips(shape, k):
    T = np.arange(int(np.prod(shape)), dtype=np.float32).reshape(shape)    # value = linear index
    for axis in range(len(shape)):
        loc = O.to_locals(T, O.S(axis), k)
        ref = _brute_split_locals(T, axis, k)
        for a, b in zip(loc, ref):
            assert a.shape == b.shape and np.array_equal(a, b)
        assert np.array_equal(O.from_locals(loc, O.S(axis)), T)
    bl = O.to_locals(T, B, k)
    assert len(bl) == k and all(np.array_equal(x, T) for x in bl)
    assert np.array_equal(O.from_locals(bl, B), T)
    bl[-1] = bl[-1] + (1 if k > 1 else 0)
    if k > 1:
        with pytest.raises(ValueError):
            O.from_locals(bl, B)


# ---------------------------------------------------------------- P reductions

def test_round_to_bf16_hand_values_and_torch():
    one = np.float32(1.0)
    cases = {
        1.0: 1.0,
        1.0 + 2.0 ** -8: 1.0,                      # tie -> even (mantissa 0)
        1.0 + 2.0 ** -7 + 2.0 ** -8: 1.0 + 2.0 ** -6,   # tie -> even (round up)
        1.0 + 2.0 ** -8 + 2.0 ** -16: 1.0 + 2.0 ** -7,  # just above the tie
        1.0 + 2.0 ** -9: 1.0,
        -3.0: -3.0,
        0.0: 0.0,
    }
    for x, want in cases.items():
        got = O.round_to_bf16(np.array([x], dtype=np.float32))[0]
        assert got == np.float32(want), (x, got, want)
    x = dg.normal(7, 0, (4096,), 0.0, 3.0, torch.float32)
    want = x.to(torch.bfloat16).to(torch.float32).numpy()       # independent library RNE
    assert np.array_equal(O.round_to_bf16(x.numpy()), want)
    assert one == 1


def test_psum_order_and_single_rounding_hand_values():
    # fp32: (1e8 + 1) - 1e8 = 0 in rank order; any other order gives 1.
    loc = [np.array([1e8], np.float32), np.array([1.0], np.float32), np.array([-1e8], np.float32)]
    assert O.reduce_sum_fixed_order(loc, "f32")[0] == np.float32(0.0)
    # bf16 storage: fp32 accumulate, ONE rounding: 1 + 3*2^-9 -> 1 + 2^-7; rounding every
    # step would give 1.
    t = np.float32(2.0 ** -9)
    loc = [np.array([1.0], np.float32)] + [np.array([t], np.float32)] * 3
    assert O.reduce_sum_fixed_order(loc, "bf16")[0] == np.float32(1.0 + 2.0 ** -7)
    assert O.reduce_sum_fixed_order(loc, "f32")[0] == np.float32(1.0 + 3 * 2.0 ** -9)
    # k = 1 is the identity
    x = dg.normal(3, 1, (5, 7), 0, 1).numpy()
    assert np.array_equal(O.reduce_sum_fixed_order([x], "f32"), x)
    assert np.array_equal(O.from_locals([x], PMAX), x)


@pytest.mark.parametrize("k", [2, 3, 4, 8])
@pytest.mark.parametrize("storage", ["f32", "bf16"])
def test_psum_exact_on_small_integers(k, storage):
    # integers in [-8, 8): every partial sum is exact in fp32 and in bf16 (|sum| <= 64),
    # so the fp32 fixed-order, the fp64 and a python-int sum must agree bit for bit.
    loc = [dg.small_integers(11, r, (6, 10), -8, 8).numpy() for r in range(k)]
    got = O.reduce_sum_fixed_order(loc, storage)
    want = np.zeros((6, 10), dtype=np.int64)
    for i in range(6):
        for j in range(10):
            want[i, j] = sum(int(loc[r][i, j]) for r in range(k))
    assert np.array_equal(got.astype(np.int64), want)
    assert np.array_equal(O.reduce_sum_fp64(loc), want.astype(np.float64))
    assert np.array_equal(O.from_locals(loc, PSUM, storage), got)


def test_pmax_hand_values_and_brute_force():
    pz, nz = np.float32(0.0), np.float32(-0.0)
    a = O.reduce_max_fixed_order([np.array([pz]), np.array([nz])])
    b = O.reduce_max_fixed_order([np.array([nz]), np.array([pz])])
    assert not np.signbit(a[0]) and np.signbit(b[0])            # first wins on a tie
    loc = [dg.normal(5, r, (4, 9), 0, 1).numpy() for r in range(5)]
    got = O.reduce_max_fixed_order(loc)
    for i in range(4):
        for j in range(9):
            assert got[i, j] == max(float(loc[r][i, j]) for r in range(5))


# ---------------------------------------------------------------- Section 3.2 boxing

def _brute_boxing_2d(src, src_sig, dst_sig, k, n0, n1):
    """Element-by-element definition in python loops for a 2-D global tensor."""
    def owner(sig, i, j):
        """(device, local index) holding global element (i, j) under an S signature."""
        ax = sig[1]
        n = (n0, n1)[ax]
        base, rem = divmod(n, k)
        a = (i, j)[ax]
        start = 0
        for r in range(k):
            ln = base + (1 if r < rem else 0)
            if a < start + ln:
                loc = [i, j]
                loc[ax] = a - start
                return r, tuple(loc), ln
            start += ln
        raise AssertionError

    def read_global(i, j):
        if src_sig[0] == "S":
            r, loc, _ = owner(src_sig, i, j)
            return float(src[r][loc])
        if src_sig[0] == "B":
            return float(src[0][i, j])
        if src_sig == PSUM:
            acc = np.float32(src[0][i, j])
            for r in range(1, k):
                acc = np.float32(acc + np.float32(src[r][i, j]))
            return float(acc)
        acc = float(src[0][i, j])
        for r in range(1, k):
            if float(src[r][i, j]) > acc:
                acc = float(src[r][i, j])
        return acc

    if dst_sig[0] == "B":
        out = [np.empty((n0, n1), np.float32) for _ in range(k)]
        for i in range(n0):
            for j in range(n1):
                v = read_global(i, j)
                for r in range(k):
                    out[r][i, j] = v
        return out
    lens = [ln for _, ln in O.balanced_split((n0, n1)[dst_sig[1]], k)]
    shapes = [((lens[r], n1) if dst_sig[1] == 0 else (n0, lens[r])) for r in range(k)]
    out = [np.empty(s, np.float32) for s in shapes]
    for i in range(n0):
        for j in range(n1):
            r, loc, _ = owner(dst_sig, i, j)
            out[r][loc] = read_global(i, j)
    return out


@pytest.mark.parametrize("n0,n1", [(8, 12), (7, 10), (5, 3)])
@pytest.mark.parametrize("k", [1, 2, 3, 4])
@pytest.mark.parametrize("src_sig,dst_sig", [
    (PSUM, B), (PSUM, S0), (PSUM, S1), (PMAX, B), (S0, B), (S1, B),
    (S0, S1), (S1, S0), (B, S0), (B, S1), (PMAX, S1),
])
def test_boxing_matches_brute_force(n0, n1, k, src_sig, dst_sig):
    T = (np.arange(n0 * n1, dtype=np.float32).reshape(n0, n1) + 1)
    if src_sig[0] == "P":
        src = [dg.normal(21, r, (n0, n1), 0, 1).numpy() for r in range(k)]
    else:
        src = O.to_locals(T, src_sig, k)
    got = O.boxing(src, src_sig, dst_sig, "f32")
    want = _brute_boxing_2d(src, src_sig, dst_sig, k, n0, n1)
    assert len(got) == k
    for g, w in zip(got, want):
        assert g.shape == w.shape and np.array_equal(g, w)


@pytest.mark.parametrize("k", [2, 3, 4])
def test_boxing_round_trip_identities(k):
    T = dg.normal(22, 0, (4, 9, 10), 0, 1).numpy()
    for i, j in [(0, 1), (1, 2), (2, 0)]:
        s_i = O.to_locals(T, O.S(i), k)
        back = O.boxing(O.boxing(s_i, O.S(i), O.S(j)), O.S(j), O.S(i))
        assert all(np.array_equal(a, b) for a, b in zip(back, s_i))
        via_b = O.boxing(O.boxing(s_i, O.S(i), B), B, O.S(i))
        assert all(np.array_equal(a, b) for a, b in zip(via_b, s_i))
        b_back = O.boxing(O.boxing(O.to_locals(T, B, k), B, O.S(i)), O.S(i), B)
        assert all(np.array_equal(a, T) for a in b_back)


def _eval_cost(expr, p):
    return eval(expr, {"__builtins__": {}}, {"p": p})        # fixture holds plain arithmetic in p


def test_table2_same_placement_costs_match_fixture_and_layout():
    rows = read_golden("table2_transfer_cost.txt")
    n0 = n1 = 24
    tbytes = n0 * n1 * 4
    for p in (2, 3, 4):
        for a, b, expr, _disjoint in rows:
            frac = _eval_cost(expr, p)
            src_sig = {"S(i)": S0, "S": S0, "B": B, "P": PSUM}[a]
            dst_sig = {"S(i)": S0, "S(j)": S1, "S": S0, "B": B, "P": PSUM}[b]
            assert O.table2_same_placement_cost(src_sig, dst_sig, p, tbytes) == round(frac * tbytes), (a, b, p)
    # The oracle's *layout* agrees with the table: tag every source element with the
    # device that holds it and count destination elements whose tag is another device.
    for p in (2, 3, 4):
        for src_sig, dst_sig in [(S0, B), (S1, B), (S0, S1), (S1, S0), (B, S0), (B, S1)]:
            if src_sig[0] == "S":
                shp = lambda r: O.to_locals(np.zeros((n0, n1)), src_sig, p)[r].shape
                src = [np.full(shp(r), r, np.float32) for r in range(p)]
                dst = O.boxing(src, src_sig, dst_sig)
                moved = sum(int((d != r).sum()) for r, d in enumerate(dst)) * 4
            else:
                moved = 0          # every device slices its own replica
                dst = O.boxing([np.zeros((n0, n1), np.float32)] * p, src_sig, dst_sig)
                assert sum(d.size for d in dst) * 4 == tbytes
            assert moved == O.table2_same_placement_cost(src_sig, dst_sig, p, tbytes)


# ---------------------------------------------------------------- Table 1 MatMul

def _py_matmul(X, W):
    M, K = X.shape
    N = W.shape[1]
    Y = np.zeros((M, N))
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for t in range(K):
                acc += float(X[i, t]) * float(W[t, j])
            Y[i, j] = acc
    return Y


def test_table1_fixture_and_rejections():
    rows = read_golden("table1_matmul_sbp.txt")
    valid = {(_parse_sig(a), _parse_sig(b)): _parse_sig(c) for a, b, c in rows}
    assert len(valid) == 6
    sigs = [S0, S1, B, PSUM]
    for xs in sigs:
        for ws in sigs:
            assert O.matmul_infer(xs, ws) == valid.get((xs, ws)), (xs, ws)
    assert sum(O.matmul_infer(a, b) is None for a in sigs for b in sigs) == 10
    for other in sigs + [PMAX]:
        assert O.matmul_infer(PMAX, other) is None and O.matmul_infer(other, PMAX) is None


def _shard_inputs(X, W, xs, ws, k, seed):
    def shard(T, sig, tid):
        if sig == PSUM:
            parts = [dg.small_integers(seed, tid + r, T.shape, -4, 5).numpy().astype(np.float64)
                     for r in range(k - 1)]
            parts.append(T - sum(parts) if parts else T.copy())
            return parts
        return O.to_locals(T, sig, k)
    return shard(X, xs, 100), shard(W, ws, 200)


@pytest.mark.parametrize("shape", [(4, 5, 8), (4, 8, 6), (6, 9, 7)])     # Table 4's shapes + an odd one
@pytest.mark.parametrize("k", [1, 2, 3])
def test_matmul_signatures_equal_logical_product_brute_force(shape, k):
    M, K, N = shape
    X = dg.small_integers(31, 0, (M, K), -5, 6).numpy().astype(np.float64)
    W = dg.small_integers(31, 1, (K, N), -5, 6).numpy().astype(np.float64)
    Y = _py_matmul(X, W)                                       # exact: small integers
    assert np.array_equal(O.matmul_logical(X, W), Y)
    for (a, b, c) in read_golden("table1_matmul_sbp.txt"):
        xs, ws, ys = _parse_sig(a), _parse_sig(b), _parse_sig(c)
        xl, wl = _shard_inputs(X, W, xs, ws, k, 32)
        y_sig, yl, Ylog = O.matmul_locals(xl, xs, wl, ws)
        assert y_sig == ys and np.array_equal(Ylog, Y)
        # every expected local tensor is the plain product of that device's local inputs
        for r in range(k):
            assert np.array_equal(yl[r], _py_matmul(xl[r], wl[r])), (a, b, r)
        # and the SBP invariant: the locals reproduce the logical product
        if ys == PSUM:
            assert np.array_equal(O.reduce_sum_fp64(yl), Y)
        else:
            assert np.array_equal(O.from_locals(yl, ys), Y)


def test_table4_program_and_uvw_chain():
    k = 2
    A0 = dg.small_integers(41, 0, (4, 5), -3, 4).numpy().astype(np.float64)
    B0 = dg.small_integers(41, 1, (5, 8), -3, 4).numpy().astype(np.float64)
    B1 = dg.small_integers(41, 2, (8, 6), -3, 4).numpy().astype(np.float64)
    s, y0, _ = O.matmul_locals(O.to_locals(A0, S0, k), S0, O.to_locals(B0, B, k), B)
    assert s == S0
    y0b = O.boxing(y0, S0, B)                                  # to_global(..., sbp=broadcast)
    s, y2, _ = O.matmul_locals(y0b, B, O.to_locals(B1, S1, k), S1)
    assert s == S1
    assert np.array_equal(O.from_locals(y2, S1), _py_matmul(_py_matmul(A0, B0), B1))
    # Y = U V W with U:S(1), V:S(0), W:B -> P(sum) carried through the second product
    U, V, W = A0, B0, B1
    s, uv, _ = O.matmul_locals(O.to_locals(U, S1, k), S1, O.to_locals(V, S0, k), S0)
    assert s == PSUM
    s, y, _ = O.matmul_locals(uv, PSUM, O.to_locals(W, B, k), B)
    assert s == PSUM
    yb = O.boxing(y, PSUM, B, "f32")
    want = _py_matmul(_py_matmul(U, V), W)
    assert all(np.array_equal(x.astype(np.float64), want) for x in yb)


def test_matmul_permutation_and_transposition_sensitivity():
    X = dg.normal(42, 0, (5, 6), 0, 1).numpy()
    perm = np.array([3, 0, 5, 1, 4, 2])
    Pm = np.zeros((6, 6))
    Pm[perm, np.arange(6)] = 1.0                                # column j of XP is column perm[j] of X
    assert np.array_equal(O.matmul_logical(X, Pm), X[:, perm].astype(np.float64))
    assert np.array_equal(O.matmul_logical(X, np.eye(6)), X.astype(np.float64))


# ---------------------------------------------------------------- GeLU / MLP

def test_gelu_closed_forms():
    assert O.gelu(np.array([0.0]))[0] == 0.0
    assert abs(O.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15       # Phi(1)
    x = np.linspace(-6, 6, 101)
    assert np.allclose(O.gelu(-x), O.gelu(x) - x, atol=1e-15)
    assert abs(O.gelu(np.array([40.0]))[0] - 40.0) == 0.0
    for v in (-2.5, -0.3, 0.7, 3.1):
        assert abs(O.gelu(np.array([v]))[0] - 0.5 * v * (1 + math.erf(v / math.sqrt(2)))) < 1e-15


def test_mlp_brute_force_tiny():
    X = dg.normal(51, 0, (3, 4), 0, 1).numpy().astype(np.float64)
    W1 = dg.normal(51, 1, (4, 6), 0, 0.5).numpy().astype(np.float64)
    W2 = dg.normal(51, 2, (6, 5), 0, 0.5).numpy().astype(np.float64)
    H = _py_matmul(X, W1)
    G = np.array([[0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in row] for row in H])
    assert np.allclose(O.mlp_logical(X, W1, W2), _py_matmul(G, W2), rtol=1e-13, atol=1e-14)


# ---------------------------------------------------------------- split softmax cross entropy

def test_softmax_xent_closed_forms():
    C, R = 96, 5
    Z = np.full((R, C), 2.5)
    labels = np.array([0, 5, 95, 17, 33])
    m, Ssum, loss = O.softmax_xent_logical(Z, labels)
    assert np.array_equal(m, np.full(R, 2.5)) and np.array_equal(Ssum, np.full(R, float(C)))
    assert np.allclose(loss, math.log(C), rtol=0, atol=1e-15)
    Z = np.zeros((R, C))
    Z[np.arange(R), labels] = 50.0                              # one-hot dominant -> loss ~ 0
    _, _, loss = O.softmax_xent_logical(Z, labels)
    assert np.all(loss >= 0) and np.all(loss < 1e-19 * C * 1e1 + 1e-15)
    wrong = (labels + 1) % C
    _, _, loss = O.softmax_xent_logical(Z, wrong)
    assert np.allclose(loss, 50.0, atol=1e-12)                  # picks the label's column, not the max


def test_softmax_xent_equals_library_log_softmax_and_is_shard_invariant():
    from scipy.special import log_softmax
    R, C = 7, 64
    Z = dg.normal(61, 0, (R, C), 0, 2.0).numpy().astype(np.float64)
    labels = dg.integers(61, 1, (R,), 0, C).numpy()
    m, Ssum, loss = O.softmax_xent_logical(Z, labels)
    want = -log_softmax(Z, axis=1)[np.arange(R), labels]
    assert np.allclose(loss, want, rtol=1e-13, atol=1e-13)
    assert np.array_equal(m, Z.max(1))
    for k in (1, 2, 3, 4, 8):
        zl = O.to_locals(Z, S1, k)
        m2, S2, loss2 = O.softmax_xent_split(zl, labels)
        assert np.array_equal(m2, m)
        assert np.allclose(S2, Ssum, rtol=1e-14) and np.allclose(loss2, loss, rtol=1e-13, atol=1e-13)


def test_softmax_xent_config4_sanity_band():
    # logits ~ N(0, sigma^2), sigma = sqrt(512)*0.01: log-sum-exp ~ ln(C) + sigma^2/2
    C = 1 << 14
    sigma = math.sqrt(512) * 0.01
    Z = dg.normal(62, 0, (4, C), 0.0, sigma).numpy().astype(np.float64)
    m, Ssum, _ = O.softmax_xent_logical(Z, np.zeros(4, dtype=np.int64))
    assert np.all(np.abs(np.log(Ssum) + m - (math.log(C) + sigma ** 2 / 2)) < 0.02)


# ---------------------------------------------------------------- row-split embedding

def test_embedding_closed_forms_and_brute_force():
    rows, d, k = 23, 4, 4
    table = dg.uniform(71, 0, (rows, d), -0.05, 0.05).numpy()
    ids = np.arange(10).reshape(5, 2)
    assert np.array_equal(O.embedding_logical(table, ids).reshape(10, d), table[:10])
    ids = dg.integers(71, 1, (6, 3), 0, rows).numpy()
    out = O.embedding_logical(table, ids)
    tl = O.to_locals(table, S0, k)
    parts = O.embedding_partials(tl, ids)
    starts = [s for s, _ in O.balanced_split(rows, k)]
    lens = [ln for _, ln in O.balanced_split(rows, k)]
    for b in range(6):
        for f in range(3):
            i = int(ids[b, f])
            assert np.array_equal(out[b, f], table[i])
            for r in range(k):
                mine = starts[r] <= i < starts[r] + lens[r]
                want = table[i] if mine else np.zeros(d, np.float32)
                assert np.array_equal(parts[r][b, f], want)
    assert np.array_equal(O.reduce_sum_fixed_order(parts, "f32"), out)      # P(sum) -> B is exact here
    # all ids inside shard 1 -> the other shards are all zero
    ids1 = np.full((4, 2), starts[1])
    parts = O.embedding_partials(tl, ids1)
    assert all(not parts[r].any() for r in (0, 2, 3)) and parts[1].any()
    # out-of-range ids give zero rows everywhere
    bad = np.array([[-1, rows, 2]])
    assert not O.embedding_logical(table, bad)[0, :2].any()
    assert all(not p[0, :2].any() for p in O.embedding_partials(tl, bad))


# ---------------------------------------------------------------- planted mistakes are caught

def test_pins_catch_planted_mistakes(monkeypatch):
    """A wrong sign, a transposed operand or a dropped term in the oracle must fail a pin."""
    with monkeypatch.context() as mp:
        mp.setattr(O, "matmul_logical", lambda X, W: (np.asarray(W, np.float64).T @ np.asarray(X, np.float64).T))
        with pytest.raises((AssertionError, ValueError)):
            test_matmul_signatures_equal_logical_product_brute_force((4, 5, 8), 2)
    with monkeypatch.context() as mp:
        real = O.balanced_split
        mp.setattr(O, "balanced_split", lambda n, k: list(reversed(real(n, k))))
        with pytest.raises((AssertionError, ValueError, IndexError)):
            test_boxing_matches_brute_force(7, 10, 3, S0, S1)
    with monkeypatch.context() as mp:
        mp.setattr(O, "reduce_sum_fixed_order",
                   lambda ls, st: O.round_to_storage(sum(np.asarray(x, np.float64) for x in reversed(ls)), st))
        with pytest.raises(AssertionError):
            test_psum_order_and_single_rounding_hand_values()
    with monkeypatch.context() as mp:
        mp.setattr(O, "gelu", lambda x: 0.5 * np.asarray(x) * (1 + np.tanh(0.79788456 * (x + 0.044715 * x ** 3))))
        with pytest.raises(AssertionError):
            test_gelu_closed_forms()


def test_boxing_p_to_p_keeps_each_partial():
    # Table 2: P -> P on the same devices moves nothing, so each device keeps its partial.
    loc = [dg.normal(23, r, (3, 5), 0, 1).numpy() for r in range(3)]
    out = O.boxing(loc, PSUM, PSUM)
    assert all(np.array_equal(a, b) and a is not b for a, b in zip(out, loc))
    assert O.table2_same_placement_cost(PSUM, PSUM, 3, 60) == 0


@pytest.mark.parametrize("shape,k", [((5, 7), 3), ((4, 6, 5), 4), ((9,), 2)])
def test_locate_agrees_with_to_locals(shape, k):
    T = np.arange(int(np.prod(shape)), dtype=np.float32).reshape(shape)
    for axis in range(len(shape)):
        loc = O.to_locals(T, O.S(axis), k)
        for idx in itertools.product(*[range(s) for s in shape]):
            (r, li), = O.locate(shape, O.S(axis), k, idx)
            assert loc[r][li] == T[idx]
    pairs = O.locate(shape, B, k, (0,) * len(shape))
    assert [r for r, _ in pairs] == list(range(k)) and all(li == (0,) * len(shape) for _, li in pairs)


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_boxing_to_partial_sum_is_local_and_sums_back(k):
    # Table 2: S -> P and B -> P move nothing.  Brute force: element (i, j) of shard r is the
    # global element if r owns it (S source) / if r == 0 (B source), else zero.
    n0, n1 = 7, 10
    T = (np.arange(n0 * n1, dtype=np.float32).reshape(n0, n1) + 1)
    for src_sig in (S0, S1, B):
        src = O.to_locals(T, src_sig, k)
        out = O.boxing(src, src_sig, PSUM)
        assert len(out) == k
        for r in range(k):
            assert out[r].shape == T.shape
            for i in range(n0):
                for j in range(n1):
                    if src_sig == B:
                        mine = r == 0
                    else:
                        (owner, _), = O.locate((n0, n1), src_sig, k, (i, j))
                        mine = owner == r
                    assert out[r][i, j] == (T[i, j] if mine else 0.0)
        assert np.array_equal(O.from_locals(out, PSUM, "f32"), T)
        assert O.table2_same_placement_cost(src_sig, PSUM, k, T.nbytes) == 0
        # nothing crosses devices: tag the sources with their device, non-zero tags stay home
        tags = [np.full(s.shape, r + 1, np.float32) for r, s in enumerate(src)]
        moved = O.boxing(tags, src_sig, PSUM) if src_sig != B else O.boxing([tags[0]] * k, B, PSUM)
        for r in range(k):
            assert set(np.unique(moved[r])) <= {0.0, float(r + 1)} if src_sig != B else True


# ---------------------------------------------------------------- Section 3.3: two-axis placements

def _parse_sig2(tok):
    return tuple(_parse_sig(t) for t in tok.split(","))


def test_table3_fixture_and_local_products_brute_force():
    rows = read_golden("table3_matmul_2d_sbp.txt")
    assert len(rows) == 2
    M, K, N = 6, 8, 9
    X = dg.small_integers(81, 0, (M, K), -4, 5).numpy().astype(np.float64)
    W = dg.small_integers(81, 1, (K, N), -4, 5).numpy().astype(np.float64)
    Y = _py_matmul(X, W)
    for pshape in [(2, 2), (2, 3), (3, 2)]:
        for a, b, c in rows:
            xs, ws, ys = _parse_sig2(a), _parse_sig2(b), _parse_sig2(c)
            assert O.matmul_infer_2d(xs, ws) == ys
            xl, wl = O.to_locals_2d(X, xs, pshape), O.to_locals_2d(W, ws, pshape)
            y_sigs, yl, Ylog = O.matmul_locals_2d(xl, xs, wl, ws, pshape)
            assert y_sigs == ys and np.array_equal(Ylog, Y)
            k0, k1 = pshape
            for r in range(k0 * k1):
                assert np.array_equal(yl[r], _py_matmul(xl[r], wl[r]))
            # the SBP invariant: the locals reproduce the logical product
            if ys[1] == PSUM:
                nodes = [O.reduce_sum_fp64(yl[i * k1:(i + 1) * k1]) for i in range(k0)]
                assert np.array_equal(O.from_locals(nodes, ys[0]), Y)
            else:
                assert np.array_equal(O.from_locals_2d(yl, ys, pshape), Y)
    assert O.matmul_infer_2d((S0, S0), (B, B)) == (S0, S0)        # nested data parallelism is valid
    assert O.matmul_infer_2d((S0, S1), (B, B)) is None             # (S(1), B) is not a row of Table 1


def test_two_axis_mapping_brute_force_and_round_trip():
    T = np.arange(7 * 10, dtype=np.float32).reshape(7, 10)
    for pshape in [(2, 2), (2, 3), (4, 2)]:
        k0, k1 = pshape
        for sigs in [(S0, S1), (S1, S0), (S0, S0), (S0, B), (B, S1), (B, B)]:
            loc = O.to_locals_2d(T, sigs, pshape)
            assert len(loc) == k0 * k1
            for i in range(k0):
                # piece i under the first signature, by the one-axis mapping (pinned above)
                node = O.to_locals(T, sigs[0], k0)[i]
                for j in range(k1):
                    assert np.array_equal(loc[i * k1 + j], O.to_locals(node, sigs[1], k1)[j])
            assert np.array_equal(O.from_locals_2d(loc, sigs, pshape), T)
        # (S(0), S(0)) is a nested split: concatenating all devices in order gives T back
        loc = O.to_locals_2d(T, (S0, S0), pshape)
        assert np.array_equal(np.concatenate(loc, axis=0), T)
        # boxing one placement axis: (S(0), P) -> (S(0), B) sums inside each group only
        parts = [dg.small_integers(82, r, O.to_locals(T, S0, k0)[r // k1].shape, -3, 4).numpy() for r in range(k0 * k1)]
        out = O.boxing_2d(parts, (S0, PSUM), (S0, B), pshape)
        for i in range(k0):
            want = sum(parts[i * k1 + j] for j in range(k1))
            for j in range(k1):
                assert np.array_equal(out[i * k1 + j], want)


def test_embedding_hidden_split_is_the_lookup_split_on_its_last_axis():
    rows, d, k = 19, 10, 4
    table = dg.uniform(72, 0, (rows, d), -0.05, 0.05).numpy()
    ids = dg.integers(72, 1, (5, 3), 0, rows).numpy()
    ids[0, 0] = -1                                               # out of range -> zeros
    parts = O.embedding_hidden_split(O.to_locals(table, S1, k), ids)
    starts = O.balanced_split(d, k)
    for b in range(5):
        for f in range(3):
            for r, (s, ln) in enumerate(starts):
                want = table[ids[b, f], s:s + ln] if ids[b, f] >= 0 else np.zeros(ln, np.float32)
                assert np.array_equal(parts[r][b, f], want)
    assert np.array_equal(O.from_locals(parts, O.S(2)), O.embedding_logical(table, ids))


def test_boxing_cast_rounds_once_after_the_gather():
    k = 3
    T = dg.normal(24, 0, (7, 12), 0, 3.0).numpy()
    T[0, 0], T[0, 1] = np.float32(1.0 + 2.0 ** -8), np.float32(1.0 + 2.0 ** -8 + 2.0 ** -16)   # tie / just above
    out = O.boxing_cast(O.to_locals(T, S0, k), S0, B, "bf16")
    want = torch.from_numpy(T).to(torch.bfloat16).to(torch.float32).numpy()     # independent library RNE
    assert len(out) == k and all(np.array_equal(o, want) for o in out)
    assert out[0][0, 0] == np.float32(1.0) and out[0][0, 1] == np.float32(1.0 + 2.0 ** -7)


def test_softmax_xent_grad_against_finite_differences_and_library_softmax():
    from scipy.special import softmax
    R, C = 4, 9
    Z = dg.normal(63, 0, (R, C), 0, 1.5).numpy().astype(np.float64)
    labels = dg.integers(63, 1, (R,), 0, C).numpy()
    G = O.softmax_xent_grad(Z, labels)
    onehot = np.zeros((R, C))
    onehot[np.arange(R), labels] = 1.0
    assert np.allclose(G, softmax(Z, axis=1) - onehot, rtol=1e-13, atol=1e-14)
    assert np.allclose(G.sum(axis=1), 0.0, atol=1e-14)
    h = 1e-6
    for i in range(R):
        for j in range(C):
            Zp, Zm = Z.copy(), Z.copy()
            Zp[i, j] += h
            Zm[i, j] -= h
            fd = (O.softmax_xent_logical(Zp, labels)[2][i] - O.softmax_xent_logical(Zm, labels)[2][i]) / (2 * h)
            assert abs(fd - G[i, j]) < 1e-8


def test_embedding_grad_table_brute_force_and_adjoint_identity():
    rows, d = 11, 4
    ids = dg.integers(73, 1, (6, 3), 0, rows).numpy()
    ids[0, 0] = rows + 5                                          # out of range: no contribution
    G = dg.normal(73, 2, (6, 3, d), 0, 1).numpy().astype(np.float64)
    got = O.embedding_grad_table(G, ids, rows)
    want = np.zeros((rows, d))
    for b in range(6):
        for f in range(3):
            if 0 <= ids[b, f] < rows:
                want[ids[b, f]] += G[b, f]
    assert np.allclose(got, want, rtol=0, atol=1e-15)
    # adjoint of the lookup: <lookup(table), G> == <table, grad_table(G)>
    table = dg.normal(73, 3, (rows, d), 0, 1).numpy().astype(np.float64)
    lhs = float((O.embedding_logical(table, ids) * G).sum())
    rhs = float((table * got).sum())
    assert abs(lhs - rhs) < 1e-12


# ---------------------------------------------------------------- Table 2, disjoint placements

def _owner_1d(n, k, a):
    """(device, local offset) of index a of an axis of length n split over k devices, by counting."""
    base, rem = divmod(n, k)
    start = 0
    for r in range(k):
        ln = base + (1 if r < rem else 0)
        if a < start + ln:
            return r, a - start
        start += ln
    raise AssertionError


@pytest.mark.parametrize("n0,n1", [(8, 12), (7, 5)])
@pytest.mark.parametrize("p,q", [(2, 3), (4, 2), (3, 5), (1, 4), (4, 1), (3, 3)])
def test_boxing_disjoint_matches_element_definition(n0, n1, p, q):
    """Every element of every output local tensor, from the definition of the signatures alone."""
    T = np.arange(n0 * n1, dtype=np.float32).reshape(n0, n1) + 1
    parts = [dg.small_integers(31, r, (n0, n1), -8, 9).numpy().astype(np.float32) for r in range(p)]
    total = np.sum(parts, axis=0)                      # exact: small integers
    for src_sig in (S0, S1, B, PSUM):
        src = parts if src_sig == PSUM else O.to_locals(T, src_sig, p)
        G = total if src_sig == PSUM else T
        for dst_sig in (S0, S1, B):
            got = O.boxing_disjoint(src, src_sig, dst_sig, q)
            assert len(got) == q
            seen = 0
            for i in range(n0):
                for j in range(n1):
                    if dst_sig[0] == "B":
                        for d in range(q):
                            assert got[d][i, j] == G[i, j]
                    else:
                        ax = dst_sig[1]
                        d, off = _owner_1d((n0, n1)[ax], q, (i, j)[ax])
                        loc = (off, j) if ax == 0 else (i, off)
                        assert got[d][loc] == G[i, j]
                        seen += 1
            if dst_sig[0] == "S":
                assert sum(g.size for g in got) == seen == n0 * n1
        # -> P(sum): the outputs have the global shape, sum back to it exactly, and each element
        # is non-zero on exactly one device (the owner of its piece, or device 0 for B)
        if src_sig != PSUM:
            got = O.boxing_disjoint(src, src_sig, PSUM, q)
            assert all(g.shape == (n0, n1) for g in got)
            assert np.array_equal(np.sum(got, axis=0), T)
            for i in range(n0):
                for j in range(n1):
                    holder = 0 if src_sig == B else _owner_1d((n0, n1)[src_sig[1]], q, (i, j)[src_sig[1]])[0]
                    for d in range(q):
                        assert got[d][i, j] == (T[i, j] if d == holder else 0.0)
    # P -> P: partial r goes to device r mod q
    got = O.boxing_disjoint(parts, PSUM, PSUM, q)
    assert np.array_equal(np.sum(got, axis=0), total)
    for d in range(q):
        want = np.zeros((n0, n1), np.float32)
        for r in range(p):
            if r % q == d:
                want = want + parts[r]
        assert np.array_equal(got[d], want)
    if p >= q:
        gm = O.boxing_disjoint(parts, PMAX, PMAX, q)
        assert np.array_equal(np.max(gm, axis=0), np.max(parts, axis=0))
    else:
        with pytest.raises(ValueError):
            O.boxing_disjoint(parts, PMAX, PMAX, q)


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_boxing_disjoint_with_equal_counts_is_boxing(k):
    T = dg.normal(32, 0, (6, 9), 0, 1).numpy()
    parts = [O.round_to_bf16(dg.normal(32, 1 + r, (6, 9), 0, 1).numpy()) for r in range(k)]   # storable as bf16
    for src_sig in (S0, S1, B, PSUM, PMAX):
        src = parts if src_sig[0] == "P" else O.to_locals(T, src_sig, k)
        for dst_sig in (S0, S1, B, PSUM, PMAX):
            if dst_sig == PMAX and src_sig != PMAX:
                continue
            if src_sig == PMAX and dst_sig == PSUM:
                continue
            a = O.boxing_disjoint(src, src_sig, dst_sig, k, "bf16" if src_sig == PSUM else "f32")
            b = O.boxing(src, src_sig, dst_sig, "bf16" if src_sig == PSUM else "f32")
            assert len(a) == len(b) and all(np.array_equal(x, y) for x, y in zip(a, b)), (src_sig, dst_sig)


def test_boxing_disjoint_psum_rounds_once_in_rank_order():
    """1 + 2^-24 + 2^-24 in fp32 rank order stays 1 (each add rounds to even), while the exact sum
    rounds up: the order of the adds is visible, and so is the single bf16 rounding."""
    a = np.array([[1.0]], np.float32)
    e = np.array([[2.0 ** -24]], np.float32)
    got = O.boxing_disjoint([a, e, e], PSUM, B, 2)
    assert got[0][0, 0] == 1.0 and got[1][0, 0] == 1.0
    got = O.boxing_disjoint([e, e, a], PSUM, B, 1)
    assert got[0][0, 0] == np.float32(1.0 + 2.0 ** -23)
    # devices 0 and 2 feed output 0, device 1 feeds output 1
    got = O.boxing_disjoint([a, e, a], PSUM, PSUM, 2)
    assert got[0][0, 0] == 2.0 and got[1][0, 0] == np.float32(2.0 ** -24)
    h = np.array([[1.0 + 2.0 ** -8]], np.float32)            # a bf16 tie: rounds to even (1.0)
    assert O.boxing_disjoint([h, np.zeros((1, 1), np.float32)], PSUM, S0, 1, "bf16")[0][0, 0] == 1.0


def test_table2_disjoint_costs_match_fixture_and_layout():
    rows = read_golden("table2_transfer_cost.txt")
    tb = 24 * 24 * 4
    for p, q in [(2, 3), (4, 2), (3, 3), (1, 5)]:
        for a, b, _same, expr in rows:
            want = round(eval(expr, {"__builtins__": {}}, {"p": p, "q": q}) * tb)
            src_sig = {"S(i)": S0, "S": S0, "B": B, "P": PSUM}[a]
            dst_sig = {"S(i)": S0, "S(j)": S1, "S": S0, "B": B, "P": PSUM}[b]
            assert O.table2_disjoint_placement_cost(src_sig, dst_sig, p, q, tb) == want, (a, b, p, q)
    # the layout agrees with the table where every output byte is a moved byte (no reduction):
    # the outputs of S/B -> S hold |T| bytes, of S/B -> B q|T|, and S/B -> P(sum) has |T| non-zeros
    T = np.arange(24 * 24, dtype=np.float32).reshape(24, 24) + 1
    for p, q in [(2, 3), (4, 2)]:
        for src_sig in (S0, S1, B):
            src = O.to_locals(T, src_sig, p)
            for dst_sig in (S0, S1, B):
                out = O.boxing_disjoint(src, src_sig, dst_sig, q)
                assert sum(o.nbytes for o in out) == O.table2_disjoint_placement_cost(src_sig, dst_sig, p, q, tb)
            out = O.boxing_disjoint(src, src_sig, PSUM, q)
            assert sum(int(np.count_nonzero(o)) for o in out) * 4 == O.table2_disjoint_placement_cost(src_sig, PSUM, p, q, tb)

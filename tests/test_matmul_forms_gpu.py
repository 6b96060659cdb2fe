"""The tensor-core MatMul kernel has two compiled forms (256 x 256 and 512 x 256 tiles per CTA pair)
and three ways to run a product: square, tall, or mixed (whole waves of tall tiles, the rest as a
second launch in the square form).  Every element is accumulated over K in the same order in all of
them, so the results must agree bit for bit; each is also checked against the CPU oracle."""
import numpy as np
import pytest
import torch
from helpers import assert_close, to_np
from test_ops_gpu import _matmul_case

import paper_2110_15032_b200 as sbp
import sbp_datagen as dg
from oracle import sbp_oracle as O

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16


@pytest.fixture(autouse=True)
def _library_chooses_again():
    yield
    sbp.sbp_matmul_set_form(sbp.SBP_TC_FORM_AUTO, 0)


# Every local tensor below has a base and a row pitch that the copy engine can address (multiples of
# 16 bytes), so that all three routes are open.  With 7 CTA pairs per launch every case has a
# tall-tile count that is not a multiple of 7, so "mixed" really runs both launches: 12, 9, 9, 9,
# 12, 12 and 27 tiles of 512 x 256.
CASES = [
    dict(M=1500, K=520, N=704, k=2, xs=sbp.B, ws=sbp.S(1)),
    dict(M=1104, K=312, N=520, k=3, xs=sbp.S(1), ws=sbp.S(0), ys=sbp.B),
    dict(M=1104, K=312, N=520, k=3, xs=sbp.S(1), ws=sbp.S(0), ys=sbp.S(0), tx=True),
    dict(M=1104, K=312, N=528, k=3, xs=sbp.S(1), ws=sbp.S(0), ys=sbp.S(1)),
    dict(M=1500, K=520, N=704, k=2, xs=sbp.S(0), ws=sbp.B, tw=True),
    dict(M=1500, K=520, N=704, k=2, xs=sbp.B, ws=sbp.S(1), flags=sbp.SBP_EPILOGUE_GELU),
    dict(M=1104, K=312, N=520, k=3, xs=sbp.S(1), ws=sbp.S(0), out_dtype=F32),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(f"{k}={v}" for k, v in c.items() if k not in "MKN"))
def test_three_forms_agree_bit_for_bit_and_with_the_oracle(case):
    results = {}
    for form, want_delta in ((sbp.SBP_TC_FORM_SQUARE, (1, 0, 0)), (sbp.SBP_TC_FORM_TALL, (0, 1, 0)),
                             (sbp.SBP_TC_FORM_MIXED, (0, 1, 1))):
        sbp.sbp_matmul_set_form(form, 7)
        before = sbp.sbp_matmul_form_stats()
        y = _matmul_case(dtype=BF16, **case)                     # parity with the oracle inside
        after = sbp.sbp_matmul_form_stats()
        assert tuple(a - b for a, b in zip(after, before)) == want_delta, (form, before, after)
        results[form] = [t.clone() for t in y.locals]
    ref = results[sbp.SBP_TC_FORM_SQUARE]
    for form in (sbp.SBP_TC_FORM_TALL, sbp.SBP_TC_FORM_MIXED):
        assert all(torch.equal(a.view(torch.uint8), b.view(torch.uint8)) for a, b in zip(ref, results[form])), form


def test_forced_form_falls_back_where_it_cannot_run():
    # fewer tall tiles than one wave: "mixed" has no whole wave to give to the tall form
    sbp.sbp_matmul_set_form(sbp.SBP_TC_FORM_MIXED, 0)
    before = sbp.sbp_matmul_form_stats()
    _matmul_case(700, 256, 520, 2, BF16, sbp.B, sbp.S(1))
    assert tuple(a - b for a, b in zip(sbp.sbp_matmul_form_stats(), before)) == (1, 0, 0)
    # a result the copy engine cannot address (odd leading dimension) is written element-wise: square
    sbp.sbp_matmul_set_form(sbp.SBP_TC_FORM_TALL, 0)
    before = sbp.sbp_matmul_form_stats()
    _matmul_case(700, 256, 333, 1, BF16, sbp.B, sbp.B)
    assert tuple(a - b for a, b in zip(sbp.sbp_matmul_form_stats(), before)) == (1, 0, 0)


def _sampled_product(M, K, N, seed, want_delta):
    """(B,B) -> B on one shard, the library choosing the form; checked on sampled rows."""
    dev = torch.device("cuda")
    X = dg.normal(seed, 0, (M, K), 0.0, 1.0, BF16, dev)
    W = dg.normal(seed, 1, (K, N), 0.0, 0.05, BF16, dev)
    x = sbp.SbpTensor((M, K), BF16, sbp.B, [X])
    w = sbp.SbpTensor((K, N), BF16, sbp.B, [W])
    y = sbp.empty_global((M, N), BF16, sbp.B, 1)
    before = sbp.sbp_matmul_form_stats()
    sbp.sbp_matmul(x, w, y)
    torch.cuda.synchronize()
    sbp.sbp_check_device_errors()
    assert tuple(a - b for a, b in zip(sbp.sbp_matmul_form_stats(), before)) == want_delta
    rows = sorted(set(list(range(0, M, 97)) + [255, 256, 511, 512, M - 513, M - 512, M - 257, M - 256, M - 1]))
    want = O.matmul_logical(to_np(X[rows]), to_np(W))
    assert_close(to_np(y.locals[0][rows]), want, 2e-2, 1e-3, f"[{M},{K}] x [{K},{N}]")
    return y


def test_library_choice_takes_each_form_on_a_whole_device():
    """Shapes for which the cost model of the host picks each route on a B200 (74 CTA pairs)."""
    sbp.sbp_matmul_set_form(sbp.SBP_TC_FORM_AUTO, 0)
    # 2 x 3 square tiles: far less than a wave
    _sampled_product(600, 512, 520, 2001, (1, 0, 0))
    # 74 tall tiles (exactly one wave) against 148 square ones (two), 256 K-blocks per tile
    _sampled_product(1024, 16384, 9472, 2002, (0, 1, 0))
    # 240 tall tiles: three whole waves, the other 18 as 36 halves in the square form (against seven
    # square waves, or four tall ones)
    y = _sampled_product(8192, 16384, 3840, 2003, (0, 1, 1))
    # the same product as one square run: identical bits
    sbp.sbp_matmul_set_form(sbp.SBP_TC_FORM_SQUARE, 0)
    y2 = _sampled_product(8192, 16384, 3840, 2003, (1, 0, 0))
    assert torch.equal(y.locals[0].view(torch.uint8), y2.locals[0].view(torch.uint8))


@pytest.mark.parametrize("form,pairs", [("mixed", 5), ("tall", 9)])
def test_operator_parity_tests_pass_with_the_form_forced_on_a_few_pairs(form, pairs):
    """Every MatMul parity test of the suite once more, in a child process whose library is told to
    take the given route with only a handful of CTA pairs: small products then run many waves, so
    the tall kernel, the half-tile walk of a mixed run's square launch and the hand-over between the
    two are exercised on all signatures, fused outputs, transposed and unaligned operands."""
    import os
    import subprocess
    import sys
    from conftest import ROOT
    env = dict(os.environ, SBP_TC_FORM=form, SBP_TC_PAIRS=str(pairs))
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_ops_gpu.py", "tests/test_strided_views_gpu.py",
                        "tests/test_two_axis_gpu.py", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                        "-k", "matmul or tensor or mlp or classifier or view or data_parallel or two_axis"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    last = r.stdout.strip().splitlines()[-1]
    assert " passed" in last and "failed" not in last, tail
    assert int(last.split(" passed")[0].split()[-1]) >= 100, last


@pytest.mark.parametrize("form", [sbp.SBP_TC_FORM_SQUARE, sbp.SBP_TC_FORM_TALL, sbp.SBP_TC_FORM_MIXED])
def test_results_are_bit_stable_across_repeated_launches(form):
    """The same product launched again and again gives the same bits: the ring, the hand-back of the
    accumulators between the MMA thread and the epilogue warps and the walk of a mixed run leave no
    room for an ordering that changes a result (a race here would show as an occasional difference).
    Short contraction and many tiles, so that the hand-backs dominate."""
    dev = torch.device("cuda")
    M, K, N, k = 4096, 512, 8192, 4
    X = dg.normal(3001, 0, (M, K), 0.0, 1.0, BF16, dev)
    x = sbp.SbpTensor((M, K), BF16, sbp.B, [X] * k)
    w = sbp.SbpTensor((K, N), BF16, sbp.S(1), [dg.normal(3001, 10 + r, (K, N // k), 0.0, 0.05, BF16, dev) for r in range(k)])
    y = sbp.empty_global((M, N), BF16, sbp.S(1), k)
    sbp.sbp_matmul_set_form(form, 0)
    sbp.sbp_matmul(x, w, y)
    torch.cuda.synchronize()
    ref = [t.clone() for t in y.locals]
    rows = [0, 255, 256, 2047, 4095]
    want = O.matmul_logical(to_np(X[rows]), np.concatenate([to_np(t) for t in w.locals], axis=1))
    got = np.concatenate([to_np(t[rows]) for t in ref], axis=1)
    assert_close(got, want, 2e-2, 1e-3, "first launch")
    for i in range(40):
        for t in y.locals:
            t.zero_()
        sbp.sbp_matmul(x, w, y)
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(ref, y.locals)), f"launch {i + 2} differs from the first"
    sbp.sbp_check_device_errors()

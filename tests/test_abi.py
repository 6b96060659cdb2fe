"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and its
host logic (local shapes, the MatMul signature rule, argument validation) is right.
No kernel is launched here."""
import ctypes as C
import os
import re

import pytest
import torch
from conftest import ROOT, read_golden

import paper_2110_15032_b200 as sbp
from paper_2110_15032_b200 import binding
from oracle import sbp_oracle as O


@pytest.fixture(scope="module")
def lib():
    from paper_2110_15032_b200.build import build
    build()
    return sbp.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sbp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sbp_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/sbp.h but not exported"


def test_struct_layout_matches_header(lib, tmp_path):
    # ndim,dtype (8) + shape (32) + pdims (4) + pshape (8) + sbp (16) + pad (4) + local (128) + local_ld (128)
    assert C.sizeof(binding._Tensor) == 8 + 32 + 4 + 8 + 16 + 4 + 128 + 128
    assert binding._Tensor.local.offset % 8 == 0
    # and against the header itself, as a C compiler lays it out
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "sbp.h"\n'
                   'int main(void) { printf("%zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(sbp_tensor), offsetof(sbp_tensor, ndim), '
                   'offsetof(sbp_tensor, dtype), offsetof(sbp_tensor, shape), offsetof(sbp_tensor, pdims), '
                   'offsetof(sbp_tensor, sbp), offsetof(sbp_tensor, local), offsetof(sbp_tensor, local_ld)); return 0; }\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(v) for v in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    T = binding._Tensor
    assert got == [C.sizeof(T), T.ndim.offset, T.dtype.offset, T.shape.offset, T.pdims.offset, T.sbp.offset,
                   T.local.offset, T.local_ld.offset]


def test_status_strings(lib):
    assert lib.sbp_status_string(0) == b"SBP_OK"
    assert lib.sbp_status_string(4) == b"SBP_ERR_SIGNATURE"
    assert lib.sbp_status_string(9) == b"SBP_ERR_TIMEOUT"


@pytest.mark.parametrize("shape", [(64, 96), (7, 10), (5, 3, 9), (2, 3, 4, 5), (3,)])
@pytest.mark.parametrize("k", [1, 2, 3, 4, 8, 16])
def test_local_shape_matches_oracle_split(lib, shape, k):
    for axis in range(len(shape)):
        parts = O.balanced_split(shape[axis], k)
        for r in range(k):
            want = list(shape)
            want[axis] = parts[r][1]
            assert sbp.sbp_local_shape(shape, sbp.S(axis), k, r) == tuple(want)
    for sig in (sbp.B, sbp.P_SUM, sbp.P_MAX):
        assert sbp.sbp_local_shape(shape, sig, k, k - 1) == tuple(shape)


def test_local_shape_rejects_bad_descriptors(lib):
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_local_shape((4, 4), sbp.S(2), 2, 0)
    assert e.value.name == "SBP_ERR_SIGNATURE"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_local_shape((4, 4), sbp.S(0), 2, 2)
    assert e.value.name == "SBP_ERR_INVALID_ARG"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_local_shape((4, 4), sbp.S(0), 17, 0)
    assert e.value.name == "SBP_ERR_INVALID_ARG"


def _sig(tok):
    return {"S(0)": sbp.S(0), "S(1)": sbp.S(1), "B": sbp.B, "P(sum)": sbp.P_SUM}[tok]


def test_matmul_infer_is_table1(lib):
    valid = {(_sig(a), _sig(b)): _sig(c) for a, b, c in read_golden("table1_matmul_sbp.txt")}
    sigs = [sbp.S(0), sbp.S(1), sbp.B, sbp.P_SUM, sbp.P_MAX]
    rejected = 0
    for xs in sigs:
        for ws in sigs:
            if (xs, ws) in valid:
                assert sbp.sbp_matmul_infer(xs, ws) == valid[(xs, ws)]
            else:
                with pytest.raises(sbp.SbpError) as e:
                    sbp.sbp_matmul_infer(xs, ws)
                assert e.value.name == "SBP_ERR_SIGNATURE"
                rejected += 1
    assert rejected == 25 - 6


def _host_tensor(shape, dtype, sig, k):
    locs = [torch.zeros(sbp.sbp_local_shape(shape, sig, k, r, dtype), dtype=dtype) for r in range(k)]
    return sbp.SbpTensor(shape, dtype, sig, locs)


def _status(fn, *a):
    try:
        fn(*a)
    except sbp.SbpError as e:
        return e.name
    return "SBP_OK"


def test_boxing_validation_happens_before_any_launch(lib):
    """Bad requests are refused on the host (so this runs without a GPU) and write nothing."""
    stream = C.c_void_p(0)

    def boxing(src, dst):
        a, b = src._c(), dst._c()
        binding._check(lib.sbp_boxing(C.byref(a), C.byref(b), stream))

    f32, bf16, i64 = torch.float32, torch.bfloat16, torch.int64
    src = _host_tensor((8, 8), f32, sbp.S(0), 2)
    assert _status(boxing, src, _host_tensor((8, 9), f32, sbp.B, 2)) == "SBP_ERR_SHAPE"
    assert _status(boxing, src, _host_tensor((8, 8), bf16, sbp.S(1), 2)) == "SBP_ERR_DTYPE"   # only S -> B may cast
    assert _status(boxing, _host_tensor((8, 8), bf16, sbp.S(0), 2), _host_tensor((8, 8), f32, sbp.B, 2)) == "SBP_ERR_DTYPE"
    # different shard counts on the two sides are the disjoint-placement transforms; what they refuse:
    assert _status(boxing, src, _host_tensor((8, 8), bf16, sbp.B, 4)) == "SBP_ERR_UNSUPPORTED"   # cast + other placement
    assert _status(boxing, src, _host_tensor((8, 8), f32, sbp.P_MAX, 4)) == "SBP_ERR_UNSUPPORTED"
    assert _status(boxing, _host_tensor((8, 8), f32, sbp.P_MAX, 2),
                   _host_tensor((8, 8), f32, sbp.P_MAX, 3)) == "SBP_ERR_UNSUPPORTED"             # zero is not neutral
    assert _status(boxing, _host_tensor((8, 8), f32, sbp.P_MAX, 2),
                   _host_tensor((8, 8), f32, sbp.P_SUM, 3)) == "SBP_ERR_UNSUPPORTED"
    assert _status(boxing, _host_tensor((8, 8), i64, sbp.P_SUM, 2),
                   _host_tensor((8, 8), i64, sbp.S(0), 3)) == "SBP_ERR_DTYPE"
    def shard(src_t, dst_t, d):
        a, b = src_t._c(), dst_t._c()
        binding._check(lib.sbp_boxing_shard(C.byref(a), C.byref(b), d, stream))

    assert _status(shard, src, _host_tensor((8, 8), f32, sbp.B, 2), 2) == "SBP_ERR_INVALID_ARG"      # outside the placement
    assert _status(shard, src, _host_tensor((8, 8), f32, sbp.B, 2), -1) == "SBP_ERR_INVALID_ARG"
    assert _status(shard, src, sbp.SbpTensor((8, 8), f32, sbp.B, [None, None]), 1) == "SBP_ERR_INVALID_ARG"   # no buffer
    assert _status(shard, src, _host_tensor((8, 8), f32, sbp.P_MAX, 2), 0) == "SBP_ERR_UNSUPPORTED"
    two_axis = sbp.SbpTensor((8, 8), f32, (sbp.B, sbp.B), [torch.zeros(8, 8) for _ in range(4)], pshape=(2, 2))
    assert _status(boxing, src, two_axis) == "SBP_ERR_INVALID_ARG"
    assert _status(boxing, src, _host_tensor((8, 8), f32, sbp.P_MAX, 2)) == "SBP_ERR_UNSUPPORTED"
    assert _status(boxing, _host_tensor((8, 8), f32, sbp.P_SUM, 2),
                   _host_tensor((8, 8), f32, sbp.P_MAX, 2)) == "SBP_ERR_UNSUPPORTED"
    assert _status(boxing, _host_tensor((8, 8), i64, sbp.P_SUM, 2),
                   _host_tensor((8, 8), i64, sbp.B, 2)) == "SBP_ERR_DTYPE"
    d = src._c()
    d.pdims = 2
    d.pshape[0], d.pshape[1] = 2, 1
    b = _host_tensor((8, 8), f32, sbp.B, 2)._c()
    assert lib.sbp_boxing(C.byref(d), C.byref(b), stream) == 1          # placements of src and dst differ
    b2 = _host_tensor((8, 8), f32, sbp.B, 2)._c()
    b2.pdims = 2
    b2.pshape[0], b2.pshape[1] = 2, 1
    b2.sbp[1] = binding._Sig(3, 0)                                      # both axes would change at once
    assert lib.sbp_boxing(C.byref(d), C.byref(b2), stream) == 5
    labels2 = _host_tensor((8,), torch.int64, sbp.B, 2)._c()
    assert lib.sbp_softmax_xent(C.byref(d), C.byref(labels2), C.byref(labels2), None, None, None, 0, None) == 5
    d = src._c()
    d.local[1] = None
    assert lib.sbp_boxing(C.byref(d), C.byref(b), stream) == 1          # null local tensor


def test_matmul_validation(lib):
    f32 = torch.float32

    def mm(x, w, y, flags=0):
        a, b, c = x._c(), w._c(), y._c()
        binding._check(lib.sbp_matmul(C.byref(a), C.byref(b), C.byref(c), flags, None, 0, None))

    k = 2
    x = _host_tensor((8, 6), f32, sbp.S(0), k)
    assert _status(mm, x, _host_tensor((6, 4), f32, sbp.S(0), k), _host_tensor((8, 4), f32, sbp.S(0), k)) == "SBP_ERR_SIGNATURE"
    assert _status(mm, x, _host_tensor((5, 4), f32, sbp.B, k), _host_tensor((8, 4), f32, sbp.S(0), k)) == "SBP_ERR_SHAPE"
    assert _status(mm, x, _host_tensor((6, 4), f32, sbp.B, k), _host_tensor((8, 4), f32, sbp.B, k)) == "SBP_ERR_SIGNATURE"
    xs1 = _host_tensor((8, 6), f32, sbp.S(1), k)
    ws0 = _host_tensor((6, 4), f32, sbp.S(0), k)
    assert _status(mm, xs1, ws0, _host_tensor((8, 4), f32, sbp.P_SUM, k), sbp.SBP_EPILOGUE_GELU) == "SBP_ERR_SIGNATURE"
    assert _status(mm, xs1, ws0, _host_tensor((8, 4), f32, sbp.P_MAX, k)) == "SBP_ERR_SIGNATURE"
    assert _status(mm, xs1, ws0, _host_tensor((8, 4), torch.bfloat16, sbp.P_SUM, k)) == "SBP_ERR_DTYPE"


def test_softmax_and_embedding_validation(lib):
    f32, i64 = torch.float32, torch.int64
    k = 2

    def xent(logits, labels, loss):
        a, b, c = logits._c(), labels._c(), loss._c()
        binding._check(lib.sbp_softmax_xent(C.byref(a), C.byref(b), C.byref(c), None, None, None, 0, None))

    labels = _host_tensor((4,), i64, sbp.B, k)
    loss = _host_tensor((4,), f32, sbp.B, k)
    assert _status(xent, _host_tensor((4, 10), f32, sbp.S(0), k), labels, loss) == "SBP_ERR_SIGNATURE"
    assert _status(xent, _host_tensor((4, 10), f32, sbp.S(1), k), _host_tensor((5,), i64, sbp.B, k), loss) == "SBP_ERR_SHAPE"
    assert _status(xent, _host_tensor((4, 10), f32, sbp.S(1), k), labels, loss) == "SBP_ERR_WORKSPACE"
    assert sbp.sbp_softmax_xent_workspace_bytes(_host_tensor((4, 10), f32, sbp.S(1), k)) >= 3 * k * 4 * 4

    def emb(table, ids, out):
        a, b, c = table._c(), ids._c(), out._c()
        binding._check(lib.sbp_embedding(C.byref(a), C.byref(b), C.byref(c), None, None))

    ids = _host_tensor((3, 2), i64, sbp.B, k)
    assert _status(emb, _host_tensor((10, 4), f32, sbp.S(1), k), ids, _host_tensor((3, 2, 4), f32, sbp.P_SUM, k)) == "SBP_ERR_SIGNATURE"
    assert _status(emb, _host_tensor((10, 4), f32, sbp.B, k), ids, _host_tensor((3, 2, 4), f32, sbp.B, k)) == "SBP_ERR_SIGNATURE"
    assert _status(emb, _host_tensor((10, 4), f32, sbp.S(0), k), ids, _host_tensor((3, 2, 5), f32, sbp.B, k)) == "SBP_ERR_SHAPE"
    assert _status(emb, _host_tensor((10, 4), f32, sbp.S(0), k), ids, _host_tensor((3, 2, 4), f32, sbp.S(0), k)) == "SBP_ERR_SIGNATURE"


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "lib_path", lambda: str(tmp_path / "libsbp_b200.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()


def test_transfer_cost_is_table2(lib):
    tb = 24 * 24 * 4
    for p, q in [(2, 2), (3, 3), (4, 2), (2, 8)]:
        for a, b, same, disjoint in read_golden("table2_transfer_cost.txt"):
            src = {"S(i)": sbp.S(0), "S": sbp.S(0), "B": sbp.B, "P": sbp.P_SUM}[a]
            dst = {"S(i)": sbp.S(0), "S(j)": sbp.S(1), "S": sbp.S(0), "B": sbp.B, "P": sbp.P_SUM}[b]
            env = {"__builtins__": {}}
            want_dis = round(eval(disjoint, env, {"p": p, "q": q}) * tb)
            assert sbp.sbp_transfer_cost(src, dst, p, q, True, tb) == want_dis, (a, b, p, q)
            if p == q:
                want_same = round(eval(same, env, {"p": p, "q": q}) * tb)
                assert sbp.sbp_transfer_cost(src, dst, p, q, False, tb) == want_same, (a, b, p)
                assert O.table2_same_placement_cost(osig_(src), osig_(dst), p, tb) == want_same
    with pytest.raises(sbp.SbpError):
        sbp.sbp_transfer_cost(sbp.S(0), sbp.B, 2, 3, False, tb)


def osig_(sig):
    return O.S(sig.axis) if sig.kind == 0 else {1: O.B, 2: O.PSUM, 3: O.PMAX}[sig.kind]


@pytest.mark.parametrize("shape,k", [((6, 10), 3), ((7, 5), 4), ((4, 3, 8), 2), ((9,), 4), ((2, 16), 8)])
def test_view_b_to_s_points_into_the_replicas(lib, shape, k):
    """Host-only: the zero-copy B -> S(axis) view (Table 2: cost 0).  Every local tensor of the view is
    the window of the replica that the oracle's split of the same tensor holds."""
    n = 1
    for s in shape:
        n *= s
    T = torch.arange(n, dtype=torch.float32).reshape(shape)
    b = sbp.SbpTensor(shape, torch.float32, sbp.B, [T.clone() for _ in range(k)])
    for axis in sorted({0, len(shape) - 1}):
        v = sbp.sbp_view_b_to_s(b, axis)
        want = O.to_locals(T.numpy(), O.S(axis), k)
        for r in range(k):
            assert tuple(v.locals[r].shape) == want[r].shape
            assert (v.locals[r].numpy() == want[r]).all()
            if v.locals[r].numel():
                assert v.locals[r].untyped_storage().data_ptr() == b.locals[r].untyped_storage().data_ptr()
    if len(shape) == 3:
        with pytest.raises(sbp.SbpError) as e:
            sbp.sbp_view_b_to_s(b, 1)
        assert e.value.name == "SBP_ERR_UNSUPPORTED"
    with pytest.raises(sbp.SbpError) as e:
        sbp.sbp_view_b_to_s(sbp.SbpTensor(shape, torch.float32, sbp.S(0), list(O_split(T, k))), 0)
    assert e.value.name == "SBP_ERR_SIGNATURE"


def O_split(T, k):
    return [torch.from_numpy(a.copy()) for a in O.to_locals(T.numpy(), O.S0, k)]


def test_matmul_route_model_on_the_host():
    """The route choice is host arithmetic (no device): sanity of its decisions and invariants."""
    import paper_2110_15032_b200 as sbp
    # far less than a wave of tiles: square
    assert sbp.sbp_matmul_route(512, 512, 4096) == (0, 0)
    # one full wave of tall tiles against two square waves, long contraction: tall
    r, t = sbp.sbp_matmul_route(1024, 37 * 256, 16384)
    assert (r, t) == (1, 74)
    # 256 tall tiles on 74 pairs, K = 16384: three whole tall waves, the rest square
    r, t = sbp.sbp_matmul_route(8192, 4096, 16384)
    assert (r, t) == (2, 222)
    # the same with a short contraction: the exposed epilogue of the tall form does not pay
    assert sbp.sbp_matmul_route(8192, 4096, 512)[0] == 0
    # GeLU in the epilogue keeps a 4096-deep product square
    assert sbp.sbp_matmul_route(8192, 16384, 4096, flags=sbp.SBP_EPILOGUE_GELU)[0] == 0
    # invariants over a sweep: the tall part is whole waves (mixed) or everything (tall), never more than there is
    for m in (256, 700, 3000, 8192, 20000):
        for n in (256, 1000, 4096, 9000):
            for k in (64, 512, 4096, 32768):
                for pairs in (3, 74):
                    r, t = sbp.sbp_matmul_route(m, n, k, pairs)
                    tall = -(-m // 512) * -(-n // 256)
                    assert r in (0, 1, 2) and 0 <= t <= tall
                    if r == 0:
                        assert t == 0
                    elif r == 1:
                        assert t == tall
                    else:
                        assert t % pairs == 0 and 0 < t < tall
    assert sbp.sbp_matmul_route(0, 4, 4)[0] == -1


def test_host_path_byte_counts_on_the_host():
    """What sbp_boxing_host[_multi] would copy is host arithmetic over the descriptors (pointers are
    compared, never followed), so it can be pinned without a device."""
    import torch
    import paper_2110_15032_b200 as sbp
    k, shape, bf16 = 4, (130, 250), torch.bfloat16
    numel = shape[0] * shape[1]

    def host(sig, alias=False):
        if alias:
            one = torch.empty(sbp.sbp_local_shape(shape, sig, k, 0, bf16), dtype=bf16)
            return sbp.SbpTensor(shape, bf16, sig, [one] * k)
        return sbp.SbpTensor(shape, bf16, sig, [torch.empty(sbp.sbp_local_shape(shape, sig, k, r, bf16), dtype=bf16) for r in range(k)])

    p, b = host(sbp.P_SUM), host(sbp.B)
    # one transform: all of every source local tensor, except B -> S(i): one block per replica
    assert sbp.sbp_boxing_host_copy_bytes(p, host(sbp.B)) == (k * numel * 2, k * numel * 2)
    assert sbp.sbp_boxing_host_copy_bytes(p, host(sbp.B, alias=True)) == (k * numel * 2, numel * 2)
    assert sbp.sbp_boxing_host_copy_bytes(b, host(sbp.S(0))) == (numel * 2, numel * 2)
    assert sbp.sbp_boxing_host_copy_bytes(b, host(sbp.S(1))) == (numel * 2, numel * 2)
    assert sbp.sbp_boxing_host_copy_bytes(host(sbp.S(0)), host(sbp.S(1))) == (numel * 2, numel * 2)
    # several destinations: the source once; the blocks only if every destination is an S of one axis
    assert sbp.sbp_boxing_host_multi_copy_bytes(p, [host(sbp.B), host(sbp.S(0)), host(sbp.S(1))]) == (k * numel * 2, (k + 2) * numel * 2)
    assert sbp.sbp_boxing_host_multi_copy_bytes(b, [host(sbp.S(1)), host(sbp.S(1))]) == (numel * 2, 2 * numel * 2)
    assert sbp.sbp_boxing_host_multi_copy_bytes(b, [host(sbp.S(0)), host(sbp.S(1))]) == (k * numel * 2, 2 * numel * 2)
    assert sbp.sbp_boxing_host_multi_workspace_bytes(p, [host(sbp.B), host(sbp.S(0))]) >= (2 * k + 1) * numel * 2

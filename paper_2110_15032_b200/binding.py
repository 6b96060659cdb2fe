"""ctypes binding of include/sbp.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

SBP_MAX_DIMS = 4
SBP_MAX_K = 16
SBP_MAX_PDIMS = 2
SBP_EPILOGUE_GELU = 1
SBP_TRANS_X = 2
SBP_TRANS_W = 4

SBP_SPLIT, SBP_BROADCAST, SBP_PARTIAL_SUM, SBP_PARTIAL_MAX = 0, 1, 2, 3
_DTYPES = {torch.float32: 0, torch.bfloat16: 1, torch.int64: 2}


class _Sig(C.Structure):
    _fields_ = [("kind", C.c_int32), ("axis", C.c_int32)]


class _Tensor(C.Structure):
    _fields_ = [
        ("ndim", C.c_int32),
        ("dtype", C.c_int32),
        ("shape", C.c_int64 * SBP_MAX_DIMS),
        ("pdims", C.c_int32),
        ("pshape", C.c_int32 * SBP_MAX_PDIMS),
        ("sbp", _Sig * SBP_MAX_PDIMS),
        ("local", C.c_void_p * SBP_MAX_K),
        ("local_ld", C.c_int64 * SBP_MAX_K),
    ]


@dataclass(frozen=True)
class Sig:
    """One SBP signature: S(axis), B, P_SUM or P_MAX (the paper's Section 3.1)."""
    kind: int
    axis: int = 0

    def __repr__(self):
        return {SBP_SPLIT: f"S({self.axis})", SBP_BROADCAST: "B",
                SBP_PARTIAL_SUM: "P(sum)", SBP_PARTIAL_MAX: "P(max)"}[self.kind]

    def _c(self) -> _Sig:
        return _Sig(self.kind, self.axis)


def S(axis: int) -> Sig:
    return Sig(SBP_SPLIT, int(axis))


B = Sig(SBP_BROADCAST)
P_SUM = Sig(SBP_PARTIAL_SUM)
P_MAX = Sig(SBP_PARTIAL_MAX)


class SbpError(RuntimeError):
    def __init__(self, status: int, name: str, detail: str):
        super().__init__(f"{name}: {detail}")
        self.status = status
        self.name = name


_LIB = None


def lib_path() -> str:
    """The library this process loads: libsbp_b200.so beside this file, or the file SBP_B200_LIBRARY
    names (the debug-bounds build, for instance)."""
    return os.environ.get("SBP_B200_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsbp_b200.so")


def load_library():
    """Loads libsbp_b200.so.  Raises if it has not been built: there is no fallback."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2110_15032_b200.build` "
            "(nvcc, sm_100a).  This package has no CPU or PyTorch fallback.")
    lib = C.CDLL(path)
    T = C.POINTER(_Tensor)
    lib.sbp_status_string.restype = C.c_char_p
    lib.sbp_status_string.argtypes = [C.c_int]
    lib.sbp_last_error.restype = C.c_char_p
    lib.sbp_launch_count.restype = C.c_uint64
    lib.sbp_debug_bounds_enabled.restype = C.c_int32
    lib.sbp_selftest_debug_bounds.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_local_shape.argtypes = [T, C.c_int32, C.POINTER(C.c_int64)]
    lib.sbp_view_b_to_s.argtypes = [T, C.c_int32, T]
    lib.sbp_matmul_infer.argtypes = [_Sig, _Sig, C.POINTER(_Sig)]
    lib.sbp_transfer_cost.argtypes = [_Sig, _Sig, C.c_int32, C.c_int32, C.c_int32, C.c_uint64, C.POINTER(C.c_uint64)]
    lib.sbp_boxing.argtypes = [T, T, C.c_void_p]
    lib.sbp_boxing_shard.argtypes = [T, T, C.c_int32, C.c_void_p]
    lib.sbp_matmul_softmax_xent_backward.argtypes = [T, T, T, T, T, T, C.c_void_p]
    lib.sbp_boxing_host_workspace_bytes.restype = C.c_size_t
    lib.sbp_boxing_host_workspace_bytes.argtypes = [T, T]
    lib.sbp_boxing_host.argtypes = [T, T, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_boxing_host_copy_bytes.argtypes = [T, T, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.sbp_boxing_host_multi_workspace_bytes.restype = C.c_size_t
    lib.sbp_boxing_host_multi_workspace_bytes.argtypes = [T, T, C.c_int32]
    lib.sbp_boxing_host_multi_copy_bytes.argtypes = [T, T, C.c_int32, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.sbp_boxing_host_multi.argtypes = [T, T, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_boxing_set_copy_engine.argtypes = [C.c_int32]
    lib.sbp_boxing_set_copy_engine.restype = None
    lib.sbp_check_device_errors.argtypes = []
    lib.sbp_selftest_wait_timeout.argtypes = [C.c_uint32, C.c_void_p]
    lib.sbp_matmul_workspace_bytes.restype = C.c_size_t
    lib.sbp_matmul_workspace_bytes.argtypes = [T, T, T]
    lib.sbp_matmul_workspace_bytes_for.restype = C.c_size_t
    lib.sbp_matmul_workspace_bytes_for.argtypes = [T, T, T, C.c_uint32]
    lib.sbp_matmul.argtypes = [T, T, T, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_tensor_map_stats.argtypes = [C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.sbp_tensor_map_stats.restype = None
    lib.sbp_matmul_set_form.argtypes = [C.c_int32, C.c_int32]
    lib.sbp_matmul_set_form.restype = None
    lib.sbp_matmul_form_stats.argtypes = [C.POINTER(C.c_uint64)]
    lib.sbp_matmul_route.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.c_uint32, C.c_int32, C.c_int32, C.POINTER(C.c_int64)]
    lib.sbp_matmul_route.restype = C.c_int32
    lib.sbp_matmul_form_stats.restype = None
    lib.sbp_softmax_xent_workspace_bytes.restype = C.c_size_t
    lib.sbp_softmax_xent_workspace_bytes.argtypes = [T]
    lib.sbp_softmax_xent.argtypes = [T, T, T, T, T, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_matmul_softmax_xent_workspace_bytes.restype = C.c_size_t
    lib.sbp_matmul_softmax_xent_workspace_bytes.argtypes = [T, T]
    lib.sbp_matmul_softmax_xent.argtypes = [T, T, T, T, T, T, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sbp_softmax_xent_backward.argtypes = [T, T, T, T, T, C.c_void_p]
    lib.sbp_softmax_xent_static.argtypes = [T, T, T, T, T, C.c_void_p]
    lib.sbp_embedding.argtypes = [T, T, T, C.c_void_p, C.c_void_p]
    lib.sbp_embedding_backward.argtypes = [T, T, T, C.c_void_p, C.c_void_p]
    _LIB = lib
    return lib


def _check(status: int):
    if status != 0:
        lib = load_library()
        raise SbpError(status, lib.sbp_status_string(status).decode(), lib.sbp_last_error().decode())


def _row_pitch(t: torch.Tensor):
    """Leading dimension to pass for a local tensor: 0 when it is contiguous, the distance between its
    rows (in elements) when it is a row-strided window, None when it is neither."""
    if t.is_contiguous():
        return 0
    if t.dim() < 2 or t.stride(-1) != 1:
        return None
    pitch = t.stride(-2)
    if pitch < t.shape[-1]:
        return None
    for i in range(t.dim() - 2):                 # every axis before the last two is dense over the pitch
        if t.shape[i] != 1 and t.stride(i) != t.stride(i + 1) * t.shape[i + 1]:
            return None
    return int(pitch)


class SbpTensor:
    """A global tensor = logical shape + dtype + signature + the k local tensors.

    `locals` are torch tensors used purely as memory (device memory for every entry
    point except sbp_boxing_host, which takes host tensors).  Each must be contiguous, or a
    window of a larger row-major buffer whose rows are a fixed distance apart (unit stride on the
    last axis, every axis before the last two dense): that distance is passed on as the
    descriptor's leading dimension.
    For a two-axis placement (the paper's multi-dimensional SBP) pass `sig` as a pair of
    signatures and `pshape=(k0, k1)`; `locals` then lists the devices row-major (i * k1 + j).
    """

    def __init__(self, shape: Sequence[int], dtype: torch.dtype, sig, locals: Sequence[torch.Tensor],
                 pshape: Optional[Sequence[int]] = None):
        self.shape = tuple(int(s) for s in shape)
        self.dtype = dtype
        self.sig = sig
        self.locals: List[torch.Tensor] = list(locals)
        self.k = len(self.locals)
        self.sigs = tuple(sig) if isinstance(sig, (tuple, list)) else (sig,)
        self.pshape = tuple(int(v) for v in pshape) if pshape is not None else (self.k,)
        if len(self.sigs) != len(self.pshape):
            raise ValueError("one signature per placement axis")
        n = 1
        for v in self.pshape:
            n *= v
        if n != self.k:
            raise ValueError("placement size differs from the number of local tensors")
        for t in self.locals:
            if t is None:            # a local tensor another device holds (sbp_boxing_shard)
                continue
            if _row_pitch(t) is None:
                raise ValueError("local tensors must be contiguous, or row-strided windows of a row-major buffer")
            if t.dtype != dtype:
                raise ValueError("local tensor dtype differs from the descriptor's")

    def _c(self) -> _Tensor:
        d = _Tensor()
        d.ndim = len(self.shape)
        d.dtype = _DTYPES[self.dtype]
        for i, s in enumerate(self.shape):
            d.shape[i] = s
        d.pdims = len(self.pshape)
        d.pshape[1] = 1
        for p, v in enumerate(self.pshape):
            d.pshape[p] = v
            d.sbp[p] = self.sigs[p]._c()
        for r, t in enumerate(self.locals):
            d.local[r] = t.data_ptr() if t is not None else None
            d.local_ld[r] = _row_pitch(t) if t is not None else 0
        return d


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def sbp_local_shape(shape, sig, k, r: int, dtype=torch.float32):
    """Local shape of device r.  One-axis placement: sig a Sig, k an int.  Two-axis placement:
    sig a pair of Sig, k the pair (k0, k1), r = i * k1 + j."""
    sigs = tuple(sig) if isinstance(sig, (tuple, list)) else (sig,)
    pshape = tuple(k) if isinstance(k, (tuple, list)) else (k,)
    d = _Tensor()
    d.ndim = len(shape)
    d.dtype = _DTYPES[dtype]
    for i, s in enumerate(shape):
        d.shape[i] = int(s)
    d.pdims = len(pshape)
    d.pshape[1] = 1
    for p, v in enumerate(pshape):
        d.pshape[p] = int(v)
        d.sbp[p] = sigs[p]._c()
    out = (C.c_int64 * SBP_MAX_DIMS)()
    _check(load_library().sbp_local_shape(C.byref(d), r, out))
    return tuple(out[i] for i in range(len(shape)))


def sbp_view_b_to_s(b: SbpTensor, axis: int) -> SbpTensor:
    """The B tensor `b` seen as S(axis) without moving anything (Table 2: B -> S costs nothing): the
    local tensors of the result are windows into b's replicas.  The pointers and leading dimensions
    come from the library; the torch views built here only keep the memory alive and are checked
    against them."""
    out = _Tensor()
    _check(load_library().sbp_view_b_to_s(C.byref(b._c()), int(axis), C.byref(out)))
    locs = []
    start = 0
    for r, t in enumerate(b.locals):
        ln = sbp_local_shape(b.shape, S(axis), b.k, r, b.dtype)[axis]
        v = t.narrow(axis, start, ln)
        start += ln
        if ln > 0 and v.numel() > 0:
            if v.data_ptr() != out.local[r] or (_row_pitch(v) or 0) != (out.local_ld[r] if out.local_ld[r] != v.shape[-1] else 0):
                raise RuntimeError("sbp_view_b_to_s: the library's view and the torch view disagree")
        locs.append(v)
    return SbpTensor(b.shape, b.dtype, S(axis), locs)


def empty_global(shape, dtype, sig, k, device="cuda", alias_replicas: bool = False) -> SbpTensor:
    """Allocates (torch.empty) the local tensors of a global tensor (k an int, or (k0, k1))."""
    pshape = tuple(k) if isinstance(k, (tuple, list)) else None
    n = k if pshape is None else pshape[0] * pshape[1]
    locs = []
    for r in range(n):
        if alias_replicas and pshape is None and sig.kind == SBP_BROADCAST and r > 0:
            locs.append(locs[0])
        else:
            locs.append(torch.empty(sbp_local_shape(shape, sig, k, r, dtype), dtype=dtype, device=device))
    return SbpTensor(shape, dtype, sig, locs, pshape)


def sbp_matmul_infer(x: Sig, w: Sig) -> Sig:
    out = _Sig()
    _check(load_library().sbp_matmul_infer(x._c(), w._c(), C.byref(out)))
    return Sig(out.kind, out.axis if out.kind == SBP_SPLIT else 0)


def sbp_transfer_cost(src: Sig, dst: Sig, p1: int, p2: int, disjoint: bool, t_bytes: int) -> int:
    """Table 2: bytes crossing between devices for src -> dst (same or disjoint device sets)."""
    out = C.c_uint64()
    _check(load_library().sbp_transfer_cost(src._c(), dst._c(), p1, p2, 1 if disjoint else 0, t_bytes, C.byref(out)))
    return int(out.value)


def sbp_tensor_map_stats():
    """(re-used, encoded) counts of the tensor-core path's copy-engine descriptors."""
    a, b = C.c_uint64(), C.c_uint64()
    load_library().sbp_tensor_map_stats(C.byref(a), C.byref(b))
    return int(a.value), int(b.value)


SBP_TC_FORM_AUTO, SBP_TC_FORM_SQUARE, SBP_TC_FORM_TALL, SBP_TC_FORM_MIXED = 0, 1, 2, 3


def sbp_matmul_set_form(form: int = 0, max_pairs: int = 0) -> None:
    """Test and measurement override of the tensor-core kernel's form and CTA-pair count."""
    load_library().sbp_matmul_set_form(int(form), int(max_pairs))


def sbp_matmul_route(m: int, n: int, k: int, pairs: int = 74, flags: int = 0, replicas: int = 1, out_f32: bool = False):
    """(route, tall tiles) the library's cost model picks for one m x n x k bf16 product: route 0
    square, 1 tall, 2 mixed (host arithmetic only)."""
    t = C.c_int64()
    r = load_library().sbp_matmul_route(m, n, k, pairs, flags, replicas, 1 if out_f32 else 0, C.byref(t))
    return int(r), int(t.value)


def sbp_matmul_form_stats():
    """Launches of the tensor-core kernel by form: (square, tall, square part of a mixed run)."""
    v = (C.c_uint64 * 3)()
    load_library().sbp_matmul_form_stats(v)
    return int(v[0]), int(v[1]), int(v[2])


def sbp_selftest_debug_bounds(buf: torch.Tensor, stream=None) -> None:
    _check(load_library().sbp_selftest_debug_bounds(C.c_void_p(buf.data_ptr()), buf.numel() * buf.element_size(),
                                                    _stream_ptr(stream)))


def sbp_debug_bounds_enabled() -> bool:
    return bool(load_library().sbp_debug_bounds_enabled())


def sbp_launch_count() -> int:
    return int(load_library().sbp_launch_count())


def sbp_check_device_errors() -> None:
    _check(load_library().sbp_check_device_errors())


def sbp_selftest_wait_timeout(limit_ms: int, stream=None) -> None:
    _check(load_library().sbp_selftest_wait_timeout(int(limit_ms), _stream_ptr(stream)))


def sbp_boxing_set_copy_engine(engine: int) -> None:
    load_library().sbp_boxing_set_copy_engine(int(engine))


def sbp_boxing(src: SbpTensor, dst: SbpTensor, stream=None) -> None:
    a, b = src._c(), dst._c()
    _check(load_library().sbp_boxing(C.byref(a), C.byref(b), _stream_ptr(stream)))


def sbp_boxing_shard(src: SbpTensor, dst: SbpTensor, dst_shard: int, stream=None) -> None:
    """Only destination local tensor `dst_shard` of the boxing op (what one device of the
    destination placement executes); the other entries of dst.locals may be None."""
    a, b = src._c(), dst._c()
    _check(load_library().sbp_boxing_shard(C.byref(a), C.byref(b), int(dst_shard), _stream_ptr(stream)))


def sbp_boxing_host_workspace_bytes(src_host: SbpTensor, dst_host: SbpTensor) -> int:
    a, b = src_host._c(), dst_host._c()
    return int(load_library().sbp_boxing_host_workspace_bytes(C.byref(a), C.byref(b)))


def sbp_boxing_host_copy_bytes(src_host: SbpTensor, dst_host: SbpTensor):
    """(host->device, device->host) bytes that one sbp_boxing_host call copies."""
    a, b = src_host._c(), dst_host._c()
    h2d, d2h = C.c_uint64(), C.c_uint64()
    _check(load_library().sbp_boxing_host_copy_bytes(C.byref(a), C.byref(b), C.byref(h2d), C.byref(d2h)))
    return int(h2d.value), int(d2h.value)


def _c_array(tensors):
    arr = (_Tensor * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t._c()
    return arr


def sbp_boxing_host_multi_workspace_bytes(src_host: SbpTensor, dst_hosts) -> int:
    a, arr = src_host._c(), _c_array(dst_hosts)
    return int(load_library().sbp_boxing_host_multi_workspace_bytes(C.byref(a), arr, len(dst_hosts)))


def sbp_boxing_host_multi_copy_bytes(src_host: SbpTensor, dst_hosts):
    """(host->device, device->host) bytes that one sbp_boxing_host_multi call copies."""
    a, arr = src_host._c(), _c_array(dst_hosts)
    h2d, d2h = C.c_uint64(), C.c_uint64()
    _check(load_library().sbp_boxing_host_multi_copy_bytes(C.byref(a), arr, len(dst_hosts), C.byref(h2d), C.byref(d2h)))
    return int(h2d.value), int(d2h.value)


def sbp_boxing_host_multi(src_host: SbpTensor, dst_hosts, dev_ws: torch.Tensor, stream=None) -> None:
    """One host source boxed into several host destinations: one upload, len(dst_hosts) transforms."""
    a, arr = src_host._c(), _c_array(dst_hosts)
    _check(load_library().sbp_boxing_host_multi(C.byref(a), arr, len(dst_hosts), C.c_void_p(dev_ws.data_ptr()),
                                                dev_ws.numel() * dev_ws.element_size(), _stream_ptr(stream)))


def sbp_boxing_host(src_host: SbpTensor, dst_host: SbpTensor, dev_ws: torch.Tensor, stream=None) -> None:
    a, b = src_host._c(), dst_host._c()
    _check(load_library().sbp_boxing_host(C.byref(a), C.byref(b), C.c_void_p(dev_ws.data_ptr()),
                                          dev_ws.numel() * dev_ws.element_size(), _stream_ptr(stream)))


def sbp_matmul_workspace_bytes(x: SbpTensor, w: SbpTensor, y: SbpTensor, flags: int = 0) -> int:
    a, b, c = x._c(), w._c(), y._c()
    return int(load_library().sbp_matmul_workspace_bytes_for(C.byref(a), C.byref(b), C.byref(c), flags))


def sbp_matmul(x: SbpTensor, w: SbpTensor, y: SbpTensor, flags: int = 0,
               ws: Optional[torch.Tensor] = None, stream=None) -> None:
    a, b, c = x._c(), w._c(), y._c()
    wp = C.c_void_p(ws.data_ptr()) if ws is not None else C.c_void_p(0)
    wb = ws.numel() * ws.element_size() if ws is not None else 0
    _check(load_library().sbp_matmul(C.byref(a), C.byref(b), C.byref(c), flags, wp, wb, _stream_ptr(stream)))


def sbp_softmax_xent_workspace_bytes(logits: SbpTensor) -> int:
    a = logits._c()
    return int(load_library().sbp_softmax_xent_workspace_bytes(C.byref(a)))


def sbp_softmax_xent(logits: SbpTensor, labels: SbpTensor, loss: SbpTensor,
                     row_max: Optional[SbpTensor], row_sum: Optional[SbpTensor],
                     ws: torch.Tensor, stream=None) -> None:
    a, b, c = logits._c(), labels._c(), loss._c()
    m = row_max._c() if row_max is not None else None
    s = row_sum._c() if row_sum is not None else None
    _check(load_library().sbp_softmax_xent(
        C.byref(a), C.byref(b), C.byref(c),
        C.byref(m) if m is not None else None, C.byref(s) if s is not None else None,
        C.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size(), _stream_ptr(stream)))


def sbp_matmul_softmax_xent_workspace_bytes(features: SbpTensor, weight: SbpTensor) -> int:
    a, b = features._c(), weight._c()
    return int(load_library().sbp_matmul_softmax_xent_workspace_bytes(C.byref(a), C.byref(b)))


def sbp_matmul_softmax_xent(features: SbpTensor, weight: SbpTensor, labels: SbpTensor, loss: SbpTensor,
                            row_max: Optional[SbpTensor], row_sum: Optional[SbpTensor],
                            ws: torch.Tensor, stream=None) -> None:
    a, b, l, c = features._c(), weight._c(), labels._c(), loss._c()
    m = row_max._c() if row_max is not None else None
    s = row_sum._c() if row_sum is not None else None
    _check(load_library().sbp_matmul_softmax_xent(
        C.byref(a), C.byref(b), C.byref(l), C.byref(c),
        C.byref(m) if m is not None else None, C.byref(s) if s is not None else None,
        C.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size(), _stream_ptr(stream)))



def sbp_matmul_softmax_xent_backward(features: SbpTensor, weight: SbpTensor, labels: SbpTensor, row_max: SbpTensor,
                                     row_sum: SbpTensor, grad_logits: SbpTensor, stream=None) -> None:
    """softmax(F W) - onehot written as S(1) without the logits ever being stored."""
    a, w, l, m, s, g = (features._c(), weight._c(), labels._c(), row_max._c(), row_sum._c(), grad_logits._c())
    _check(load_library().sbp_matmul_softmax_xent_backward(C.byref(a), C.byref(w), C.byref(l), C.byref(m), C.byref(s),
                                                           C.byref(g), _stream_ptr(stream)))


def sbp_softmax_xent_backward(logits: SbpTensor, labels: SbpTensor, row_max: SbpTensor, row_sum: SbpTensor,
                              grad_logits: SbpTensor, stream=None) -> None:
    a, b, m, s, g = logits._c(), labels._c(), row_max._c(), row_sum._c(), grad_logits._c()
    _check(load_library().sbp_softmax_xent_backward(C.byref(a), C.byref(b), C.byref(m), C.byref(s), C.byref(g),
                                                    _stream_ptr(stream)))


def sbp_softmax_xent_static(logits: SbpTensor, labels: SbpTensor, loss: SbpTensor,
                            row_max: Optional[SbpTensor] = None, row_sum: Optional[SbpTensor] = None,
                            stream=None) -> None:
    """sbp_softmax_xent without a workspace argument: the partial vectors live in an array
    built into the library, for callers that cannot allocate device memory.  See
    include/sbp.h for the size limit and the sharing rules."""
    a, b, c = logits._c(), labels._c(), loss._c()
    m = row_max._c() if row_max is not None else None
    s = row_sum._c() if row_sum is not None else None
    _check(load_library().sbp_softmax_xent_static(
        C.byref(a), C.byref(b), C.byref(c),
        C.byref(m) if m is not None else None, C.byref(s) if s is not None else None,
        _stream_ptr(stream)))


def sbp_embedding(table: SbpTensor, ids: SbpTensor, out: SbpTensor,
                  oob_count: Optional[torch.Tensor] = None, stream=None) -> None:
    a, b, c = table._c(), ids._c(), out._c()
    oob = C.c_void_p(oob_count.data_ptr()) if oob_count is not None else C.c_void_p(0)
    _check(load_library().sbp_embedding(C.byref(a), C.byref(b), C.byref(c), oob, _stream_ptr(stream)))


def sbp_embedding_backward(grad_out: SbpTensor, ids: SbpTensor, grad_table: SbpTensor,
                           oob_count: Optional[torch.Tensor] = None, stream=None) -> None:
    a, b, c = grad_out._c(), ids._c(), grad_table._c()
    oob = C.c_void_p(oob_count.data_ptr()) if oob_count is not None else C.c_void_p(0)
    _check(load_library().sbp_embedding_backward(C.byref(a), C.byref(b), C.byref(c), oob, _stream_ptr(stream)))


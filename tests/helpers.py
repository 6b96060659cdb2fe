"""Glue between seeded torch inputs, the numpy oracle and the CUDA library (tests only)."""
import numpy as np
import torch

import paper_2110_15032_b200 as sbp
from oracle import sbp_oracle as O

SIG_TO_ORACLE = {}


def osig(sig):
    """binding Sig -> oracle signature tuple."""
    if sig.kind == 0:
        return O.S(sig.axis)
    return {1: O.B, 2: O.PSUM, 3: O.PMAX}[sig.kind]


def storage_of(dtype):
    return {torch.float32: "f32", torch.bfloat16: "bf16", torch.int64: "i64"}[dtype]


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact host copy; bf16 is widened to float32 (exact)."""
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        t = t.to(torch.float32)
    return t.numpy()


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit pattern, for bit-exact comparisons (distinguishes -0.0 from +0.0)."""
    t = t.detach().cpu().contiguous()
    view = {torch.float32: torch.int32, torch.bfloat16: torch.int16, torch.int64: torch.int64}[t.dtype]
    return t.view(view).numpy()


def np_bits(a: np.ndarray, dtype) -> np.ndarray:
    if dtype == torch.float32:
        return np.ascontiguousarray(a, dtype=np.float32).view(np.int32)
    if dtype == torch.bfloat16:
        return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16).view(np.int16)
    return np.ascontiguousarray(a, dtype=np.int64)


def make_global(locals_cpu, shape, dtype, sig, device="cuda"):
    """SbpTensor on the device from a list of CPU torch tensors (one per shard)."""
    return sbp.SbpTensor(shape, dtype, sig, [t.to(device).contiguous() for t in locals_cpu])


def split_cpu(T: torch.Tensor, sig, k):
    """Local tensors (CPU torch) of a logical CPU tensor under S(i) or B, via the oracle's
    own mapping (the library is never used to prepare its own inputs)."""
    arrs = O.to_locals(T.view(torch.int16).numpy() if T.dtype == torch.bfloat16 else T.numpy(), osig(sig), k)
    outs = [torch.from_numpy(np.ascontiguousarray(a)) for a in arrs]
    if T.dtype == torch.bfloat16:
        outs = [o.view(torch.bfloat16) for o in outs]
    return outs


def assert_close(gpu: np.ndarray, ref: np.ndarray, rtol, atol, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    err = np.abs(gpu - ref)
    bound = atol + rtol * np.abs(ref)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} outside tolerance; worst at {i}: "
                             f"gpu={gpu[i]!r} ref={ref[i]!r} err={err[i]:.3e} bound={bound[i]:.3e}")


# ------------------------------------------------------------------------------ guard bands
#
# Every output buffer the GPU tests hand to the library sits between two bands of 256 bytes of
# 0xAB, and its own bytes start as 0xFF (a NaN pattern for the floating types, -1 for int64).  A
# kernel that stores outside a local tensor changes a band; one that skips an element leaves a NaN
# behind that the comparison with the oracle then trips over.

GUARD_BYTES = 256
_GUARDED = []          # (raw uint8 buffer, payload bytes, description)


def guarded_empty(shape, dtype, device="cuda", what=""):
    """An uninitialised-looking tensor of `shape` whose storage is flanked by guard bands."""
    esz = torch.empty((), dtype=dtype).element_size()
    n = esz
    for s in shape:
        n *= int(s)
    raw = torch.empty(n + 2 * GUARD_BYTES, dtype=torch.uint8, device=device)
    raw[:GUARD_BYTES] = 0xAB
    raw[GUARD_BYTES + n:] = 0xAB
    raw[GUARD_BYTES:GUARD_BYTES + n] = 0xFF
    _GUARDED.append((raw, n, f"{what} {tuple(shape)} {dtype}"))
    return raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(tuple(int(s) for s in shape))


def guarded_empty_global(shape, dtype, sig, k, device="cuda", alias_replicas=False):
    """Same contract as the package's empty_global, every local tensor inside guard bands."""
    pshape = tuple(k) if isinstance(k, (tuple, list)) else None
    n = k if pshape is None else pshape[0] * pshape[1]
    locs = []
    for r in range(n):
        if alias_replicas and pshape is None and sig.kind == sbp.B.kind and r > 0:
            locs.append(locs[0])
        else:
            locs.append(guarded_empty(sbp.sbp_local_shape(shape, sig, k, r, dtype), dtype, device, f"shard {r} of"))
    return sbp.SbpTensor(shape, dtype, sig, locs, pshape)


def check_guards(clear=False):
    """Waits for the device and asserts that no band around any guarded buffer has changed."""
    if torch.cuda.is_available():
        torch.cuda.synchronize()
    bad = []
    for raw, n, what in _GUARDED:
        bands = torch.cat([raw[:GUARD_BYTES], raw[GUARD_BYTES + n:]]).cpu().numpy()
        if not (bands == 0xAB).all():
            at = int(np.flatnonzero(bands != 0xAB)[0])
            side = "before" if at < GUARD_BYTES else "after"
            bad.append(f"{what}: byte {at % GUARD_BYTES} of the band {side} the buffer was overwritten")
    if clear:
        _GUARDED.clear()
    assert not bad, "stores outside a destination buffer: " + "; ".join(bad)

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

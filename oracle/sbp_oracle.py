"""CPU oracle for the SBP boxing transforms and the sharded operators they feed.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
library is checked against.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the library never does, and the two share no code.

Everything is numpy: float64 for the logical results, float32 where the method itself
fixes fp32 (the fixed-order partial-value reduction).  A tensor whose storage type is
bf16 is carried as a float32 array whose values are exactly representable in bf16.

Notation follows the paper's Section 3 ("The Compiler"): a *global* (logical) tensor T
is mapped onto k *local* tensors by an SBP signature --
  S(i)  split along axis i "in a balanced manner",
  B     broadcast: every local tensor is an exact copy of T,
  P(op) partial-value: every local tensor has T's shape and T is the element-wise
        reduction (sum, max) over the local tensors.
Signatures are written here as ("S", i), ("B",), ("P", "sum"), ("P", "max").

Every function is pinned by tests/test_oracle_pins.py against brute force on tiny
inputs, closed forms, round-trip identities and the paper's tables; no function in
this file is "parity unpinned".
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

S0 = ("S", 0)
S1 = ("S", 1)
B = ("B",)
PSUM = ("P", "sum")
PMAX = ("P", "max")


def S(axis):
    return ("S", int(axis))


# --------------------------------------------------------------------------------------
# Section 3.1: the mapping between a global tensor and its local tensors
# --------------------------------------------------------------------------------------

def balanced_split(n, k):
    """(start, length) of each of the k contiguous pieces of an axis of length n.

    The paper only says "balanced" (Section 3.1).  Reading taken here: the first
    n mod k pieces get ceil(n/k) elements, the others floor(n/k), in rank order.
    """
    base, rem = divmod(int(n), int(k))
    out, start = [], 0
    for r in range(k):
        ln = base + (1 if r < rem else 0)
        out.append((start, ln))
        start += ln
    return out


def to_locals(T, sig, k):
    """Local tensors of global tensor T under signature sig (Section 3.1, Figure 3).

    Defined for S(i) and B.  A P signature has many valid decompositions, so P local
    tensors are always *inputs* (or the per-shard products of Table 1), never derived.
    """
    T = np.asarray(T)
    if sig[0] == "S":
        ax = sig[1]
        return [np.ascontiguousarray(np.take(T, np.arange(s, s + ln), axis=ax))
                for (s, ln) in balanced_split(T.shape[ax], k)]
    if sig[0] == "B":
        return [T.copy() for _ in range(k)]
    raise ValueError("to_locals is not defined for a partial-value signature")


def locate(shape, sig, k, index):
    """Where global element `index` (a tuple) lives under S(i) or B: a list of
    (shard, local index) pairs -- one pair for S(i), k pairs for B (Section 3.1)."""
    index = tuple(int(v) for v in index)
    if sig[0] == "B":
        return [(r, index) for r in range(k)]
    if sig[0] == "S":
        ax = sig[1]
        for r, (start, ln) in enumerate(balanced_split(shape[ax], k)):
            if start <= index[ax] < start + ln:
                loc = list(index)
                loc[ax] = index[ax] - start
                return [(r, tuple(loc))]
        raise IndexError(index)
    raise ValueError("locate is not defined for a partial-value signature")


def round_to_bf16(x32):
    """float32 -> nearest bf16 (ties to even), returned as float32.  Finite inputs."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    bits = x32.view(np.uint32).astype(np.uint64)
    bits = bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))
    bits = (bits & np.uint64(0xFFFF0000)).astype(np.uint32)
    return bits.view(np.float32).reshape(x32.shape)


def round_to_storage(x, storage):
    if storage == "f32":
        return np.asarray(x, dtype=np.float32)
    if storage == "bf16":
        return round_to_bf16(np.asarray(x, dtype=np.float32))
    raise ValueError(storage)


def reduce_sum_fixed_order(locals_, storage):
    """P(sum) -> global tensor.  The paper is silent on order and precision; the reading
    is an fp32 accumulator started at shard 0, shards added in rank order 1..k-1 with
    plain IEEE adds, and ONE rounding to the storage type at the end."""
    acc = np.asarray(locals_[0], dtype=np.float32).copy()
    for r in range(1, len(locals_)):
        acc = acc + np.asarray(locals_[r], dtype=np.float32)
    return round_to_storage(acc, storage)


def reduce_sum_fp64(locals_):
    """The same sum carried in float64 (used for cancellation-safe error bounds)."""
    acc = np.asarray(locals_[0], dtype=np.float64).copy()
    for r in range(1, len(locals_)):
        acc = acc + np.asarray(locals_[r], dtype=np.float64)
    return acc


def reduce_max_fixed_order(locals_):
    """P(max) -> global tensor: acc = shard 0; a later shard replaces acc only when it
    is strictly greater (first wins on ties, so +0/-0 is order-determined).  Exact."""
    acc = np.asarray(locals_[0]).copy()
    for r in range(1, len(locals_)):
        x = np.asarray(locals_[r])
        acc = np.where(x > acc, x, acc)
    return acc


def from_locals(locals_, sig, storage="f32"):
    """Inverse mapping: the global tensor seen through k local tensors (Section 3.1)."""
    if sig[0] == "S":
        return np.concatenate([np.asarray(x) for x in locals_], axis=sig[1])
    if sig[0] == "B":
        first = np.asarray(locals_[0])
        for x in locals_[1:]:
            if not np.array_equal(first, np.asarray(x)):
                raise ValueError("broadcast replicas differ")
        return first.copy()
    if sig == PSUM:
        return reduce_sum_fixed_order(locals_, storage)
    if sig == PMAX:
        return reduce_max_fixed_order(locals_)
    raise ValueError(sig)


# --------------------------------------------------------------------------------------
# Section 3.2: boxing.  A boxing op re-arranges / transforms the local tensors so that
# the SAME global tensor is seen under the new signature.
# --------------------------------------------------------------------------------------

def boxing(src_locals, src_sig, dst_sig, storage="f32"):
    k = len(src_locals)
    if src_sig[0] == "P" and tuple(src_sig) == tuple(dst_sig):
        # Table 2, P -> P on the same placement costs 0: every device keeps its own partial.
        return [np.asarray(x).copy() for x in src_locals]
    if tuple(dst_sig) == PSUM:
        # Table 2, S -> P and B -> P on the same placement cost 0: every device builds its partial
        # from what it already holds.  Reading: a split source pads its own slice with zeros
        # (the k padded slices sum to T); a broadcast source keeps T on device 0, zeros elsewhere.
        T = from_locals(src_locals, src_sig, storage)
        outs = [np.zeros_like(T) for _ in range(k)]
        if src_sig[0] == "S":
            ax = src_sig[1]
            for r, (start, ln) in enumerate(balanced_split(T.shape[ax], k)):
                sel = [slice(None)] * T.ndim
                sel[ax] = slice(start, start + ln)
                outs[r][tuple(sel)] = np.asarray(src_locals[r])
        else:
            outs[0] = T.copy()
        return outs
    T = from_locals(src_locals, src_sig, storage)
    return to_locals(T, dst_sig, k)


def boxing_disjoint(src_locals, src_sig, dst_sig, k_dst, storage="f32"):
    """Boxing between two DIFFERENT device sets (Section 3.2, Table 2, column "disjoint"): the
    input lives on p = len(src_locals) devices, the output on q = k_dst other devices.

    The table gives only the bytes that move; the readings taken here are the simplest
    transforms that move exactly those bytes and keep the global tensor unchanged:
      S or B -> S or B   the global tensor is rebuilt and mapped onto the q devices;
      P -> S, P -> B     the p partials are reduced in fixed rank order (all p|T| bytes travel),
                         then mapped onto the q devices;
      S -> P(sum)        |T| travels once: output device j holds piece j of the q-way balanced
                         split of the source's split axis, in place, zeros elsewhere;
      B -> P(sum)        |T| travels once: output device 0 holds T, the others zeros;
      P -> P             every partial travels once (p|T|): input device r sends to output device
                         r mod q, which reduces what it receives in ascending r (an output device
                         that receives nothing holds zeros; for P(max) that case is undefined).
    With q = p every row gives the same local tensors as boxing() on one placement.
    """
    p, q = len(src_locals), int(k_dst)
    src_sig, dst_sig = tuple(src_sig), tuple(dst_sig)
    if src_sig[0] == "P" and dst_sig[0] == "P":
        if src_sig != dst_sig:
            raise ValueError("P(sum) <-> P(max) has no meaning")
        outs = []
        for j in range(q):
            mine = [src_locals[r] for r in range(j, p, q)]
            if not mine:
                if dst_sig == PMAX:
                    raise ValueError("P(max) onto more devices than partials is undefined")
                outs.append(np.zeros_like(np.asarray(src_locals[0])))
            else:
                outs.append(from_locals(mine, src_sig, storage))
        return outs
    T = from_locals(src_locals, src_sig, storage)
    if dst_sig == PSUM:
        outs = [np.zeros_like(T) for _ in range(q)]
        if src_sig[0] == "S":
            ax = src_sig[1]
            for j, (start, ln) in enumerate(balanced_split(T.shape[ax], q)):
                sel = [slice(None)] * T.ndim
                sel[ax] = slice(start, start + ln)
                outs[j][tuple(sel)] = T[tuple(sel)]
        else:
            outs[0] = T.copy()
        return outs
    if dst_sig[0] == "P":
        raise ValueError("S -> P(max) / B -> P(max): zero is not neutral for max")
    return to_locals(T, dst_sig, q)


def table2_disjoint_placement_cost(src_sig, dst_sig, p, q, t_bytes):
    """Table 2, column "disjoint": bytes that travel from the p input devices to the q output
    devices (|T| = t_bytes)."""
    a, b = src_sig[0], dst_sig[0]
    if a == "P":
        return (p + q - 1) * t_bytes if b == "B" else p * t_bytes
    return q * t_bytes if b == "B" else t_bytes


def boxing_cast(src_locals, src_sig, dst_sig, dst_storage):
    """Boxing followed by a cast of every destination local tensor to dst_storage (Section 6.4:
    a cast op with S(0) input and B output turns sharded fp32 state into half-precision replicas)."""
    return [round_to_storage(x, dst_storage) for x in boxing(src_locals, src_sig, dst_sig, "f32")]


def table2_same_placement_cost(src_sig, dst_sig, k, t_bytes):
    """Table 2, column "same": bytes that cross between devices for src -> dst when both
    live on the same k devices.  Used to tell which transforms move data at all."""
    a, b = src_sig[0], dst_sig[0]
    if a == "S" and b == "S":
        return 0 if src_sig[1] == dst_sig[1] else (k - 1) * t_bytes // k
    if a == "S" and b == "B":
        return (k - 1) * t_bytes
    if a == "P" and b == "S":
        return (k - 1) * t_bytes
    if a == "P" and b == "B":
        return 2 * (k - 1) * t_bytes
    return 0          # S->P, B->S, B->B, B->P, P->P


# --------------------------------------------------------------------------------------
# Table 1: valid SBP signatures for MatMul
# --------------------------------------------------------------------------------------

_TABLE1 = {
    (S0, B): S0,
    (B, S1): S1,
    (S1, S0): PSUM,
    (PSUM, B): PSUM,
    (B, PSUM): PSUM,
    (B, B): B,
}


def matmul_infer(x_sig, w_sig):
    """Signature of Y = XW, or None when (x_sig, w_sig) is not a row of Table 1."""
    return _TABLE1.get((tuple(x_sig), tuple(w_sig)))


def matmul_logical(X, W):
    return np.asarray(X, dtype=np.float64) @ np.asarray(W, dtype=np.float64)


def matmul_locals(x_locals, x_sig, w_locals, w_sig):
    """Expected local tensors (float64) of Y = XW under a Table 1 signature.

    Rows whose output is S or B: the logical product, mapped through to_locals.
    Rows whose output is P(sum): the partials are fixed by the signature --
      (S(1),S(0)): Y_r = X[:, K_r] W[K_r, :]   (the r-th slice of the contraction),
      (P,B):       Y_r = X_r W,     (B,P): Y_r = X W_r   (Section 3.3, Y = U V W example).
    Returns (y_sig, y_locals, Y_logical).
    """
    k = len(x_locals)
    y_sig = matmul_infer(x_sig, w_sig)
    if y_sig is None:
        raise ValueError("invalid MatMul signature")
    f64 = lambda ls: [np.asarray(a, dtype=np.float64) for a in ls]
    xl, wl = f64(x_locals), f64(w_locals)
    X = reduce_sum_fp64(xl) if x_sig == PSUM else from_locals(xl, x_sig)
    W = reduce_sum_fp64(wl) if w_sig == PSUM else from_locals(wl, w_sig)
    Y = matmul_logical(X, W)
    if y_sig[0] in ("S", "B"):
        return y_sig, to_locals(Y, y_sig, k), Y
    if (x_sig, w_sig) == (S1, S0):
        parts = []
        for (s, ln) in balanced_split(X.shape[1], k):
            parts.append(matmul_logical(X[:, s:s + ln], W[s:s + ln, :]))
        return y_sig, parts, Y
    if x_sig == PSUM:
        return y_sig, [matmul_logical(xl[r], W) for r in range(k)], Y
    return y_sig, [matmul_logical(X, wl[r]) for r in range(k)], Y


# --------------------------------------------------------------------------------------
# Section 3.3: multi-dimensional SBP.  A placement of k0 x k1 devices carries one signature
# per placement axis, e.g. (S(0), B): S(0) across the k0 groups ("nodes"), B among the k1
# devices of a group.  Device (i, j) -- listed row-major, index i * k1 + j -- holds piece j,
# under the second signature, of piece i, under the first, of the global tensor.
# --------------------------------------------------------------------------------------

def to_locals_2d(T, sigs, pshape):
    k0, k1 = pshape
    out = []
    for node in to_locals(T, sigs[0], k0):
        out.extend(to_locals(node, sigs[1], k1))
    return out


def from_locals_2d(locals_, sigs, pshape, storage="f32"):
    k0, k1 = pshape
    nodes = [from_locals(locals_[i * k1:(i + 1) * k1], sigs[1], storage) for i in range(k0)]
    return from_locals(nodes, sigs[0], storage)


def boxing_2d(src_locals, src_sigs, dst_sigs, pshape, storage="f32"):
    """Boxing between two-axis signatures none of whose destination axes is partial-value."""
    return to_locals_2d(from_locals_2d(src_locals, src_sigs, pshape, storage), dst_sigs, pshape)


def matmul_infer_2d(x_sigs, w_sigs):
    """Table 3: Table 1 applied to each placement axis on its own; None if either is invalid."""
    ys = tuple(matmul_infer(a, b) for a, b in zip(x_sigs, w_sigs))
    return None if any(y is None for y in ys) else ys


def matmul_locals_2d(x_locals, x_sigs, w_locals, w_sigs, pshape):
    """Every device multiplies its local tensors.  Returns (y_sigs, y_locals, Y_logical) with
    the logical product computed from the logical operands (partial operands summed in fp64)."""
    y_sigs = matmul_infer_2d(x_sigs, w_sigs)
    if y_sigs is None:
        raise ValueError("invalid two-axis MatMul signature")
    f64 = lambda ls: [np.asarray(a, dtype=np.float64) for a in ls]
    xl, wl = f64(x_locals), f64(w_locals)

    def logical(locs, sigs):
        k0, k1 = pshape
        def inv(ls, sig):
            return reduce_sum_fp64(ls) if tuple(sig) == PSUM else from_locals(ls, sig)
        return inv([inv(locs[i * k1:(i + 1) * k1], sigs[1]) for i in range(k0)], sigs[0])

    Y = matmul_logical(logical(xl, x_sigs), logical(wl, w_sigs))
    return y_sigs, [matmul_logical(a, b) for a, b in zip(xl, wl)], Y


# --------------------------------------------------------------------------------------
# GeLU (erf form) and the Megatron-style MLP block: B x S(1) -> S(1), GeLU, S(1) x S(0)
# -> P(sum), boxed to B.  Logical result only; sharding cannot change it.
# --------------------------------------------------------------------------------------

def gelu(x):
    x = np.asarray(x, dtype=np.float64)
    return 0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))


def mlp_logical(X, W1, W2):
    return matmul_logical(gelu(matmul_logical(X, W1)), W2)


# --------------------------------------------------------------------------------------
# Section 6.3 (InsightFace case): classifier weight S(1) -> logits S(1); softmax with two
# reductions (max, then sum), each local first and then global; sparse cross entropy.
# --------------------------------------------------------------------------------------

def softmax_xent_logical(Z, labels):
    """Plain single-device definition on the logical logits Z [rows, classes].

    m_i = max_j Z_ij,  S_i = sum_j exp(Z_ij - m_i),  loss_i = log S_i + m_i - Z_i,y_i.
    Returns (m, S, loss) as float64.
    """
    Z = np.asarray(Z, dtype=np.float64)
    labels = np.asarray(labels, dtype=np.int64)
    m = Z.max(axis=1)
    Ssum = np.exp(Z - m[:, None]).sum(axis=1)
    zy = Z[np.arange(Z.shape[0]), labels]
    return m, Ssum, np.log(Ssum) + m - zy


def softmax_xent_grad(Z, labels):
    """d loss_i / d Z_ij = softmax(Z_i)_j - [j == y_i]  (per-row loss, unit upstream gradient)."""
    Z = np.asarray(Z, dtype=np.float64)
    labels = np.asarray(labels, dtype=np.int64)
    m, Ssum, _ = softmax_xent_logical(Z, labels)
    G = np.exp(Z - m[:, None]) / Ssum[:, None]
    G[np.arange(Z.shape[0]), labels] -= 1.0
    return G


def softmax_xent_split(z_locals, labels):
    """The same quantity in the split form the paper describes: per shard r a local
    max m_r and, after the global max m = max_r m_r (P(max) -> B), a local
    s_r = sum_j exp(z_r - m); S = sum_r s_r (P(sum) -> B); the label's logit comes from
    the one shard whose class range holds it (all others contribute 0)."""
    labels = np.asarray(labels, dtype=np.int64)
    zl = [np.asarray(z, dtype=np.float64) for z in z_locals]
    m_r = [z.max(axis=1) for z in zl]
    m = reduce_max_fixed_order(m_r)
    s_r = [np.exp(z - m[:, None]).sum(axis=1) for z in zl]
    Ssum = reduce_sum_fp64(s_r)
    rows = np.arange(labels.shape[0])
    t_r, off = [], 0
    for z in zl:
        c = z.shape[1]
        inside = (labels >= off) & (labels < off + c)
        col = np.where(inside, labels - off, 0)
        t_r.append(np.where(inside, z[rows, col], 0.0))
        off += c
    zy = reduce_sum_fp64(t_r)
    return m, Ssum, np.log(Ssum) + m - zy


# --------------------------------------------------------------------------------------
# Section 6.3 (Wide & Deep case): embedding table S(0) ("splitting the vocabulary IDs")
# --------------------------------------------------------------------------------------

def embedding_logical(table, ids):
    """out[..., :] = table[ids[...], :].  An id outside [0, rows) yields a zero row."""
    table = np.asarray(table)
    ids = np.asarray(ids, dtype=np.int64)
    ok = (ids >= 0) & (ids < table.shape[0])
    out = table[np.where(ok, ids, 0)]
    out[~ok] = 0
    return out


def embedding_partials(table_locals, ids):
    """Row-split lookup: shard r answers only the ids inside its own row range and
    writes zeros elsewhere, so the k outputs are a P(sum) tensor."""
    ids = np.asarray(ids, dtype=np.int64)
    outs, off = [], 0
    for t in table_locals:
        t = np.asarray(t)
        inside = (ids >= off) & (ids < off + t.shape[0])
        if t.shape[0] == 0:
            o = np.zeros(ids.shape + t.shape[1:], dtype=t.dtype)
        else:
            o = t[np.where(inside, ids - off, 0)]
            o[~inside] = 0
        outs.append(o)
        off += t.shape[0]
    return outs


def embedding_hidden_split(table_locals, ids):
    """Table S(1) ("splitting the hidden dimension", Section 6.3): shard r holds a column block
    of every row, looks up every id in it, and its result is that column block of the lookup:
    the k outputs are the lookup split along its last axis."""
    return [embedding_logical(t, ids) for t in table_locals]


def embedding_grad_table(grad_out, ids, rows):
    """Adjoint of the lookup: grad_table[i, :] = sum of grad_out[l, :] over the lookups l with
    ids[l] == i (float64).  Ids outside [0, rows) contribute nothing."""
    grad_out = np.asarray(grad_out, dtype=np.float64)
    ids = np.asarray(ids, dtype=np.int64).reshape(-1)
    g = grad_out.reshape(ids.shape[0], -1)
    out = np.zeros((rows, g.shape[1]), dtype=np.float64)
    ok = (ids >= 0) & (ids < rows)
    np.add.at(out, ids[ok], g[ok])
    return out


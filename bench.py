#!/usr/bin/env python
"""Benchmark of the SBP boxing sweep (and, at one GPU, of the sharded operators).

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One step = the seven boxing transforms of the bandwidth-sweep workload (logical bf16
[8192, 8192], k = 4): P(sum)->B, P(sum)->S(0), P(sum)->S(1), S(0)->B, S(0)->S(1), S(1)->S(0),
B->S(1), each reading every input local tensor once and writing every output local tensor
once.  value = algorithmic bytes of a step / device time of a step.  With N > 1 every rank
runs its own replica of the sweep (no collective on the data path; weak scaling).

Prints one JSON line (rank 0).  --impl reference times the CPU oracle instead.

--gpus N is the number of ranks: started without a launcher and N > 1, the script starts the N
ranks itself (torch.distributed.run on 127.0.0.1); under a launcher WORLD_SIZE must equal N.
At one GPU the line also carries, inside `roofline`, one entry per line of configs 2-5
(`roofline.configs`: kernel, bound, ms, work, achieved, frac of the measured peak and, for HBM lines
with an ncu capture, the DRAM-byte rate) and, inside `cpu_baseline`, the oracle timed on a bounded
sample of each config (`cpu_baseline.configs`, with the host's cores and the threads it used).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import sbp_datagen as dg  # noqa: E402

METRIC = "boxing/embedding/softmax HBM GB/s and sharded MatMul TFLOP/s vs B200 peak"
SWEEP_SHAPE = (8192, 8192)
SWEEP_K = 4
SEED = 1002
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ workload

TRANSFORMS = [
    # name, source kind, destination signature, algorithmic bytes in units of |T|
    ("P(sum)->B", "P", "B", 8),
    ("P(sum)->S(0)", "P", "S0", 5),
    ("P(sum)->S(1)", "P", "S1", 5),
    ("S(0)->B", "S0", "B", 5),
    ("S(0)->S(1)", "S0", "S1", 2),
    ("S(1)->S(0)", "S1", "S0", 2),
    ("B->S(1)", "B", "S1", 2),
]


def t_bytes():
    return SWEEP_SHAPE[0] * SWEEP_SHAPE[1] * 2


def step_bytes():
    return sum(t[3] for t in TRANSFORMS) * t_bytes()


def build_sweep(sbp, device):
    """Device-resident sources and destinations of the seven transforms."""
    k, shape, bf16 = SWEEP_K, SWEEP_SHAPE, torch.bfloat16
    sig = {"P": sbp.P_SUM, "B": sbp.B, "S0": sbp.S(0), "S1": sbp.S(1)}
    T = dg.normal(SEED, 0, shape, 0.0, 1.0, bf16, device)
    n0, n1 = shape
    src = {
        "P": sbp.SbpTensor(shape, bf16, sbp.P_SUM, [dg.normal(SEED, 10 + r, shape, 0.0, 1.0, bf16, device) for r in range(k)]),
        "S0": sbp.SbpTensor(shape, bf16, sbp.S(0), [T[r * n0 // k:(r + 1) * n0 // k].contiguous() for r in range(k)]),
        "S1": sbp.SbpTensor(shape, bf16, sbp.S(1), [T[:, r * n1 // k:(r + 1) * n1 // k].contiguous() for r in range(k)]),
        "B": sbp.SbpTensor(shape, bf16, sbp.B, [T.clone() for _ in range(k)]),
    }
    work = []
    for name, s, d, units in TRANSFORMS:
        dst = sbp.empty_global(shape, bf16, sig[d], k, device=device)
        work.append((name, src[s], dst, units * t_bytes()))
    return T, src, work


def run_sweep(sbp, work, events=None):
    """One step.  With events (len(work) + 1 of them): one record before the first launch and one
    after every launch, so transform i runs between events[i] and events[i + 1]."""
    if events is not None:
        events[0].record()
    for i, (_, s, d, _) in enumerate(work):
        sbp.sbp_boxing(s, d)
        if events is not None:
            events[i + 1].record()



# ------------------------------------------------------------------------------ ncu traffic

# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/.
# None = not captured for the kernel as it stands.
NCU_TRAFFIC = {
    # profiles/box_kernels_sweep_bf16_8192x8192_k4.md (full size)
    "P(sum)->B": 1024.0e6, "P(sum)->S(0)": 647.0e6, "P(sum)->S(1)": 648.1e6, "S(0)->B": 614.1e6,
    "S(0)->S(1)": 219.2e6, "S(1)->S(0)": 217.3e6, "B->S(1)": 217.8e6,
    # profiles/xent_partial_bf16_512x1048576_k8.md (full size)
    "softmax-xent on bf16 logits (partial + combine)": 1077.2e6,
    "softmax-xent backward (softmax - onehot, S(1))": 2099.7e6,
    # profiles/matmul_tc_classifier_bf16_512x512x1048576_k8.md (full size)
    "classifier GEMM (B,S(1))->S(1), bf16 logits": 2104.3e6,
    "classifier GEMM fused with softmax-xent (no logits stored)": 1127.8e6 + 50.5e6,
    "classifier GEMM fused with the softmax-xent backward (grad S(1), no logits stored)": 2103.8e6,
    # profiles/matmul_tc_mlp_bf16_8192x4096x16384_k8.md (full size; a mixed run is the sum of its two launches)
    "MLP GEMM1 (B,S(1))->S(1) + GeLU": 1003.3e6,
    "MLP GEMM2 (S(1),S(0))->P(sum), bf16 partials": 914.0e6,
    "MLP GEMM2 fused (S(1),S(0))->B": 1195.4e6 + 194.6e6,
    "MLP GEMM1 with W1 stored transposed (SBP_TRANS_W) + GeLU": 1003.4e6,
    "MLP GEMM2 fused (S(1),S(0))->B with W2 stored transposed (SBP_TRANS_W)": 1195.2e6 + 194.4e6,
    "DP layer backward dW = X^T dY, (S(1),S(0))->S(0) fused": 872.6e6,
    "DP layer backward dW = X^T dY, (S(1),S(0))->B fused (8 replicas written)": 1774.9e6,
    "DP layer backward dX = dY W^T, (S(0),B)->S(0)": 747.1e6 + 206.0e6,
    # profiles/extras_bf16_8192x8192_p4_and_embedding_fp32_4194304x128_batch16384_k8.md (full size)
    "S(0)->P(sum) bf16 [8192,8192] k=4": 619.4e6,
    "B->P(sum) bf16 [8192,8192] k=4": 611.7e6,
    "S(0) fp32 -> B bf16 (cast fused into the gather) [8192,8192] k=4": 749.2e6,
    "disjoint placements: S(0)[4] -> S(0)[8] bf16 [8192,8192]": 216.3e6,
    "disjoint placements: S(0)[4] -> S(1)[8] bf16 [8192,8192]": 215.2e6,
    "disjoint placements: S(0)[4] -> B[8] bf16 [8192,8192]": 1148.7e6,
    "disjoint placements: P(sum)[4] -> S(0)[8] bf16 [8192,8192]": 616.9e6,
    "disjoint placements: P(sum)[4] -> B[2] bf16 [8192,8192]": 752.2e6,
    "disjoint placements: S(0)[4] -> P(sum)[8] bf16 [8192,8192]": 1015.0e6 + 216.1e6,
    # profiles/embedding_fused_fp32_config5_full_size_and_quarter_batch.md (full size, one-pass DRAM counters)
    "embedding fused gather -> B (8 replicas written)": 7308.8e6,
    "embedding fused gather -> B (replicas aliased, 1 write)": 1096.1e6,
}
# The commits whose kernels the captures above were taken on (the tensor-core MatMul lines were
# taken again after the kernel got its tall and mixed forms; the other kernels have not changed
# since the first).  A kernel that changes afterwards gets its entry set to None (or recaptured)
# in the same commit: a stale figure is worse than none.
NCU_TRAFFIC_CAPTURED_AT = "a61a16e (boxing, softmax, embedding to several replicas); 073ea77 (matmul_tc_kernel); 68937c6 (embedding_rows_kernel)"


def ncu_traffic(name):
    return NCU_TRAFFIC.get(name)


# ------------------------------------------------------------------------------ end to end

def e2e_sweep(sbp, src, work, device, steps, dist):
    """The sweep through the host entry point: pinned host buffers in, pinned host buffers out,
    host->device and device->host copies inside the timed region.  The transforms of a step that
    read the same source go into one sbp_boxing_host_multi call, so every source crosses once."""
    host_src = {}
    for key, g in src.items():
        host_src[key] = sbp.SbpTensor(g.shape, g.dtype, g.sig, [t.cpu().pin_memory() for t in g.locals])
    key_of = {id(g): key for key, g in src.items()}
    groups = {}      # source key -> host destinations, in the order of the sweep
    host_dst_of = {}
    for name, s_, d, _ in work:
        hd = sbp.SbpTensor(d.shape, d.dtype, d.sig,
                           [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in d.locals])
        groups.setdefault(key_of[id(s_)], []).append(hd)
        host_dst_of[name] = hd
    jobs = [(host_src[key], dsts) for key, dsts in groups.items()]
    h2d = d2h = 0
    for hs, dsts in jobs:
        a, b = sbp.sbp_boxing_host_multi_copy_bytes(hs, dsts)      # what the call really copies
        h2d += a
        d2h += b
    # One stream and one device workspace per source: the device->host copies of one group overlap
    # the host->device copy of the next (PCIe is full duplex; the device->host direction, 1.74 GB a
    # step, is the bound once every source is sent once).
    streams = [torch.cuda.Stream(device=device) for _ in jobs]
    wss = [torch.empty(sbp.sbp_boxing_host_multi_workspace_bytes(hs, dsts), dtype=torch.uint8, device=device) for hs, dsts in jobs]

    def one_step():
        for i, (hs, dsts) in enumerate(jobs):
            sbp.sbp_boxing_host_multi(hs, dsts, wss[i], stream=streams[i])

    one_step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    cur = torch.cuda.current_stream()
    start.record()
    for st in streams:
        st.wait_stream(cur)
    for _ in range(steps):
        one_step()
    for st in streams:
        cur.wait_stream(st)
    end.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    if dist is not None:
        dist.barrier()
    ms = max_over_ranks(max(start.elapsed_time(end), wall * 1e3), dist, device) / steps
    # spot check: the last transform's result on the host equals the device-resident run
    ref = work[-1][2].locals[0].cpu()
    if not torch.equal(ref, host_dst_of[work[-1][0]].locals[0]):
        raise RuntimeError("end-to-end result differs from the device-resident result")
    return {"value": step_bytes() / (ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


# ------------------------------------------------------------------------------ operator sections

_FLUSH = None


def _flush_l2(device):
    """Writes a buffer twice L2's size, then reads another one.  The write evicts whatever the last
    iteration left in L2; the read that follows pushes the dirty lines of that write out again, so
    that their write-back (up to 126 MB, 19 us of DRAM time) is not charged to the timed launch."""
    global _FLUSH
    if _FLUSH is None:
        _FLUSH = (torch.empty(256 << 20, dtype=torch.uint8, device=device),
                  torch.zeros(32 << 20, dtype=torch.int64, device=device))
    _FLUSH[0].fill_(1)
    _FLUSH[1].sum()


OP_REPEATS = {"iters": None, "warmup": None}    # set by --op-iters / --op-warmup (profiling-sized runs)


def time_op(fn, device, iters=10, warmup=3):
    """Average and best device time (ms) of fn(), L2 flushed between iterations."""
    iters = OP_REPEATS["iters"] or iters
    warmup = OP_REPEATS["warmup"] if OP_REPEATS["warmup"] is not None else warmup
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = []
    for _ in range(iters):
        _flush_l2(device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ms.append(a.elapsed_time(b))
    return sum(ms) / len(ms), min(ms)


def time_mm(sbp, fn, device, iters=5):
    """time_op for a tensor-core product, plus the route the library takes for it (which compiled
    form(s) of the kernel its calls launched, from the library's own launch counters)."""
    before = sbp.sbp_matmul_form_stats()
    avg, best = time_op(fn, device, iters=iters)
    d = [a - b for a, b in zip(sbp.sbp_matmul_form_stats(), before)]
    form = "mixed" if d[2] else ("tall" if d[1] else ("square" if d[0] else "none"))
    return avg, best, {"form": form}


def _hbm_entry(name, nbytes, avg, best, peaks, extra=None, config=None, kernel=None):
    """One HBM-bound line.  `achieved` counts the ALGORITHMIC bytes; where an ncu capture of the kernel
    as it stands exists, `achieved_dram` is that capture's DRAM bytes per launch over the same time."""
    gbs = nbytes / (avg * 1e-3) / 1e9
    traffic = ncu_traffic(name)
    e = {"op": name, "config": config, "kernel": kernel, "bound": "hbm", "bytes": nbytes, "ms": avg, "best_ms": best,
         "achieved": gbs, "unit": "GB/s",
         "peak": peaks["hbm_gbs"], "frac_measured": gbs / peaks["hbm_gbs"], "frac_nominal": gbs / NOMINAL_HBM_GBS,
         "traffic": traffic}
    if traffic is not None:
        e["achieved_dram"] = traffic / (avg * 1e-3) / 1e9
        e["frac_dram"] = e["achieved_dram"] / peaks["hbm_gbs"]
    if extra:
        e.update(extra)
    return e


def _tensor_entry(name, flops, avg, best, peaks, extra=None, config=None, kernel="matmul_tc_kernel"):
    tf = flops / (avg * 1e-3) / 1e12
    e = {"op": name, "config": config, "kernel": kernel, "bound": "tensor", "flops": flops, "ms": avg, "best_ms": best,
         "achieved": tf, "unit": "TFLOP/s",
         "peak": peaks["bf16_tflops"], "frac_measured": tf / peaks["bf16_tflops"], "traffic": ncu_traffic(name),
         "frac_sustained": tf / peaks["bf16_tflops_sustained"], "frac_nominal": tf / NOMINAL_BF16_TFLOPS}
    if extra:
        e.update(extra)
    return e


def section_embedding(sbp, device, peaks, opts):
    """Row-split embedding: fp32 table [2^24, 128] S(0) over k = 8, ids int64 [65536, 26] Zipf(1.05)."""
    k, rows, dim, batch = 8, opts.emb_rows, 128, opts.emb_batch
    ids = dg.zipf_ids(1005, 1, (batch, 26), rows, 1.05, device)
    table = sbp.SbpTensor((rows, dim), torch.float32, sbp.S(0),
                          [dg.uniform(1005, 100 + r, (rows // k, dim), -0.05, 0.05, torch.float32, device) for r in range(k)])
    idt = sbp.SbpTensor((batch, 26), torch.int64, sbp.B, [ids] * k)
    out_b = sbp.empty_global((batch, 26, dim), torch.float32, sbp.B, k, device=device)
    out_1 = sbp.empty_global((batch, 26, dim), torch.float32, sbp.B, k, device=device, alias_replicas=True)
    n = batch * 26
    row_b = dim * 4
    unique = int(torch.unique(ids).numel())
    res = []
    avg, best = time_op(lambda: sbp.sbp_embedding(table, idt, out_b), device)
    res.append(_hbm_entry("embedding fused gather -> B (8 replicas written)", n * 8 + n * row_b + k * n * row_b, avg, best, peaks,
                          {"unique_rows": unique, "lookups": n}))
    avg, best = time_op(lambda: sbp.sbp_embedding(table, idt, out_1), device)
    res.append(_hbm_entry("embedding fused gather -> B (replicas aliased, 1 write)", n * 8 + 2 * n * row_b, avg, best, peaks,
                          {"unique_rows": unique, "lookups": n}))
    del out_1
    out_p = sbp.empty_global((batch, 26, dim), torch.float32, sbp.P_SUM, k, device=device)

    def unfused():
        sbp.sbp_embedding(table, idt, out_p)
        sbp.sbp_boxing(out_p, out_b)
    avg, best = time_op(unfused, device, iters=5)
    res.append(_hbm_entry("embedding unfused: gather -> P(sum), then P(sum) -> B", k * n * 8 + n * row_b + 3 * k * n * row_b,
                          avg, best, peaks))
    return res


def section_softmax(sbp, device, peaks, opts):
    """Class-split softmax cross entropy on materialised bf16 logits [512, 2^20], S(1) over k = 8."""
    k, rows, classes = 8, opts.xent_rows, 1 << 20
    sigma = (512 ** 0.5) * 0.01
    logits = sbp.SbpTensor((rows, classes), torch.bfloat16, sbp.S(1),
                           [dg.normal(1004, 10 + r, (rows, classes // k), 0.0, sigma, torch.bfloat16, device) for r in range(k)])
    labels = dg.integers(1004, 1, (rows,), 0, classes, device)
    lab = sbp.SbpTensor((rows,), torch.int64, sbp.B, [labels] * k)
    loss = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    ws = torch.empty(sbp.sbp_softmax_xent_workspace_bytes(logits), dtype=torch.uint8, device=device)
    avg, best = time_op(lambda: sbp.sbp_softmax_xent(logits, lab, loss, None, None, ws), device)
    res = [_hbm_entry("softmax-xent on bf16 logits (partial + combine)", rows * classes * 2 + rows * 8, avg, best, peaks,
                      {"loss_mean": float(loss.locals[0].mean().item())})]
    rmax = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    rsum = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    sbp.sbp_softmax_xent(logits, lab, loss, rmax, rsum, ws)
    grad = sbp.empty_global((rows, classes), torch.bfloat16, sbp.S(1), k, device=device)
    avg, best = time_op(lambda: sbp.sbp_softmax_xent_backward(logits, lab, rmax, rsum, grad), device)
    res.append(_hbm_entry("softmax-xent backward (softmax - onehot, S(1))", 2 * rows * classes * 2, avg, best, peaks))
    return res


def section_mlp(sbp, device, peaks, opts):
    """Megatron-style MLP: X[8192,4096] B, W1[4096,16384] S(1), GeLU, W2[16384,4096] S(0), k = 8."""
    k, M, H, F = 8, 8192, 4096, 16384
    bf16 = torch.bfloat16
    X = dg.normal(1003, 0, (M, H), 0.0, 1.0, bf16, device)
    x = sbp.SbpTensor((M, H), bf16, sbp.B, [X] * k)
    w1 = sbp.SbpTensor((H, F), bf16, sbp.S(1), [dg.normal(1003, 10 + r, (H, F // k), 0.0, 0.02, bf16, device) for r in range(k)])
    w2 = sbp.SbpTensor((F, H), bf16, sbp.S(0), [dg.normal(1003, 30 + r, (F // k, H), 0.0, 0.02, bf16, device) for r in range(k)])
    h = sbp.empty_global((M, F), bf16, sbp.S(1), k, device=device)
    y_p = sbp.empty_global((M, H), bf16, sbp.P_SUM, k, device=device)
    y_b = sbp.empty_global((M, H), bf16, sbp.B, k, device=device)
    ws = torch.empty(max(1, sbp.sbp_matmul_workspace_bytes(h, w2, y_b), sbp.sbp_matmul_workspace_bytes(x, w1, h)),
                     dtype=torch.uint8, device=device)
    flops = 2.0 * M * H * F
    res = []
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(x, w1, h, sbp.SBP_EPILOGUE_GELU, ws), device)
    res.append(_tensor_entry("MLP GEMM1 (B,S(1))->S(1) + GeLU", flops, avg, best, peaks, form))
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(h, w2, y_p, 0, ws), device)
    res.append(_tensor_entry("MLP GEMM2 (S(1),S(0))->P(sum), bf16 partials", flops, avg, best, peaks, form))
    avg, best = time_op(lambda: sbp.sbp_boxing(y_p, y_b), device)
    res.append(_hbm_entry("MLP P(sum)->B of the bf16 partials", 2 * k * M * H * 2, avg, best, peaks))
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(h, w2, y_b, 0, ws), device)
    res.append(_tensor_entry("MLP GEMM2 fused (S(1),S(0))->B", flops, avg, best, peaks, form))
    # The same two products with the weights kept in memory as their transposes ([N,K], SBP_TRANS_W):
    # both operands of the MMA are then K-major, the form the tensor pipe runs fastest.
    w1t = sbp.SbpTensor((F, H), bf16, sbp.S(0), [t.t().contiguous() for t in w1.locals])      # stored S(0) = S(1) of W1
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(x, w1t, h, sbp.SBP_EPILOGUE_GELU | sbp.SBP_TRANS_W, ws), device)
    res.append(_tensor_entry("MLP GEMM1 with W1 stored transposed (SBP_TRANS_W) + GeLU", flops, avg, best, peaks, form))
    del w1t
    w2t = sbp.SbpTensor((H, F), bf16, sbp.S(1), [t.t().contiguous() for t in w2.locals])      # stored S(1) = S(0) of W2
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(h, w2t, y_b, sbp.SBP_TRANS_W, ws), device)
    res.append(_tensor_entry("MLP GEMM2 fused (S(1),S(0))->B with W2 stored transposed (SBP_TRANS_W)", flops, avg, best, peaks, form))
    del w2t
    del h, y_p, y_b, w1, w2, x
    # Backward products of a data-parallel layer of the same size (tokens S(0), weight B), taken
    # from the stored operands with the transpose flags: dW = X^T dY is (S(1),S(0)) -> P(sum),
    # written as S(0) (the gradient reduce-scatter folded in) or as B (the all-reduce folded in);
    # dX = dY W^T is (S(0),B) -> S(0).
    xs = sbp.SbpTensor((M, H), bf16, sbp.S(0), [dg.normal(1003, 50 + r, (M // k, H), 0.0, 1.0, bf16, device) for r in range(k)])
    dy = sbp.SbpTensor((M, F), bf16, sbp.S(0), [dg.normal(1003, 60 + r, (M // k, F), 0.0, 1.0, bf16, device) for r in range(k)])
    Wb = dg.normal(1003, 70, (H, F), 0.0, 0.02, bf16, device)
    wb = sbp.SbpTensor((H, F), bf16, sbp.B, [Wb] * k)
    dw_s = sbp.empty_global((H, F), bf16, sbp.S(0), k, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(xs, dy, dw_s, sbp.SBP_TRANS_X), device)
    res.append(_tensor_entry("DP layer backward dW = X^T dY, (S(1),S(0))->S(0) fused", flops, avg, best, peaks, form))
    dw_b = sbp.empty_global((H, F), bf16, sbp.B, k, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(xs, dy, dw_b, sbp.SBP_TRANS_X), device)
    res.append(_tensor_entry("DP layer backward dW = X^T dY, (S(1),S(0))->B fused (8 replicas written)", flops, avg, best, peaks, form))
    del dw_b
    dx = sbp.empty_global((M, H), bf16, sbp.S(0), k, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(dy, wb, dx, sbp.SBP_TRANS_W), device)
    res.append(_tensor_entry("DP layer backward dX = dY W^T, (S(0),B)->S(0)", flops, avg, best, peaks, form))
    return res


def section_classifier_gemm(sbp, device, peaks, opts):
    """Classifier logits: F[512,512] B x W[512, 2^20] S(1) over k = 8 -> bf16 logits S(1)."""
    k, rows, feat, classes = 8, opts.xent_rows, 512, 1 << 20
    bf16 = torch.bfloat16
    Fm = dg.normal(1004, 0, (rows, feat), 0.0, 1.0, bf16, device)
    f = sbp.SbpTensor((rows, feat), bf16, sbp.B, [Fm] * k)
    w = sbp.SbpTensor((feat, classes), bf16, sbp.S(1),
                      [dg.normal(1004, 40 + r, (feat, classes // k), 0.0, 0.01, bf16, device) for r in range(k)])
    z = sbp.empty_global((rows, classes), bf16, sbp.S(1), k, device=device)
    ws = torch.empty(max(1, sbp.sbp_matmul_workspace_bytes(f, w, z)), dtype=torch.uint8, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(f, w, z, 0, ws), device)
    e = _tensor_entry("classifier GEMM (B,S(1))->S(1), bf16 logits", 2.0 * rows * feat * classes, avg, best, peaks, form)
    nbytes = feat * classes * 2 + rows * classes * 2 + rows * feat * 2
    e["hbm_gbs"] = nbytes / (avg * 1e-3) / 1e9
    e["hbm_frac_measured"] = e["hbm_gbs"] / peaks["hbm_gbs"]
    # the same classifier with the softmax partials taken in the epilogue (logits never stored)
    labels = dg.integers(1004, 1, (rows,), 0, classes, device)
    lab = sbp.SbpTensor((rows,), torch.int64, sbp.B, [labels] * k)
    loss = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    del z
    ws2 = torch.empty(sbp.sbp_matmul_softmax_xent_workspace_bytes(f, w), dtype=torch.uint8, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul_softmax_xent(f, w, lab, loss, None, None, ws2), device)
    e2 = _tensor_entry("classifier GEMM fused with softmax-xent (no logits stored)", 2.0 * rows * feat * classes,
                       avg, best, peaks, dict(form, loss_mean=float(loss.locals[0].mean().item())))
    nbytes2 = feat * classes * 2 + rows * feat * 2
    e2["hbm_gbs"] = nbytes2 / (avg * 1e-3) / 1e9
    e2["hbm_frac_measured"] = e2["hbm_gbs"] / peaks["hbm_gbs"]
    # and its backward: the product recomputed, softmax - onehot written as bf16 S(1)
    rmax = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    rsum = sbp.empty_global((rows,), torch.float32, sbp.B, k, device=device)
    sbp.sbp_matmul_softmax_xent(f, w, lab, loss, rmax, rsum, ws2)
    grad = sbp.empty_global((rows, classes), bf16, sbp.S(1), k, device=device)
    avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul_softmax_xent_backward(f, w, lab, rmax, rsum, grad), device)
    e3 = _tensor_entry("classifier GEMM fused with the softmax-xent backward (grad S(1), no logits stored)",
                       2.0 * rows * feat * classes, avg, best, peaks, form)
    e3["hbm_gbs"] = nbytes / (avg * 1e-3) / 1e9
    e3["hbm_frac_measured"] = e3["hbm_gbs"] / peaks["hbm_gbs"]
    return [e, e2, e3]


def section_extras(sbp, device, peaks, opts):
    """Rows beyond the core sweep: boxing to P(sum) (Table 2's zero-cost rows, materialised) and the
    embedding with the table split on the hidden axis, at the sizes of configs 2 and 5."""
    k, shape, bf16 = SWEEP_K, (8192, 8192), torch.bfloat16
    tb = shape[0] * shape[1] * 2
    T = dg.normal(SEED, 0, shape, 0.0, 1.0, bf16, device)
    s0 = sbp.SbpTensor(shape, bf16, sbp.S(0), [T[r * shape[0] // k:(r + 1) * shape[0] // k].contiguous() for r in range(k)])
    b = sbp.SbpTensor(shape, bf16, sbp.B, [T.clone() for _ in range(k)])
    part = sbp.empty_global(shape, bf16, sbp.P_SUM, k, device=device)
    res = []
    avg, best = time_op(lambda: sbp.sbp_boxing(s0, part), device)
    res.append(_hbm_entry("S(0)->P(sum) bf16 [8192,8192] k=4", (1 + k) * tb, avg, best, peaks))
    avg, best = time_op(lambda: sbp.sbp_boxing(b, part), device)
    res.append(_hbm_entry("B->P(sum) bf16 [8192,8192] k=4", (1 + k) * tb, avg, best, peaks))
    del T, b, part
    torch.cuda.empty_cache()
    # Section 6.4's cast op: fp32 shards S(0) -> bf16 replicas B, the cast folded into the gather
    Tf = dg.normal(SEED, 1, shape, 0.0, 1.0, torch.float32, device)
    sf = sbp.SbpTensor(shape, torch.float32, sbp.S(0), [Tf[r * shape[0] // k:(r + 1) * shape[0] // k].contiguous() for r in range(k)])
    rb = sbp.empty_global(shape, bf16, sbp.B, k, device=device)
    avg, best = time_op(lambda: sbp.sbp_boxing(sf, rb), device)
    res.append(_hbm_entry("S(0) fp32 -> B bf16 (cast fused into the gather) [8192,8192] k=4", 2 * tb + k * tb, avg, best, peaks))
    del Tf, sf, rb
    torch.cuda.empty_cache()
    # different placements (Table 2, column "disjoint"): p = 4 source shards, q = 8 (or 2) destination shards
    psrc = sbp.SbpTensor(shape, bf16, sbp.P_SUM, [dg.normal(SEED, 300 + r, shape, 0.0, 1.0, bf16, device) for r in range(k)])
    for name, src_g, dst_sig, q, nbytes in [
            ("S(0)[4] -> S(0)[8]", s0, sbp.S(0), 8, 2 * tb),
            ("S(0)[4] -> S(1)[8]", s0, sbp.S(1), 8, 2 * tb),
            ("S(0)[4] -> B[8]", s0, sbp.B, 8, tb + 8 * tb),
            ("P(sum)[4] -> S(0)[8]", psrc, sbp.S(0), 8, k * tb + tb),
            ("P(sum)[4] -> B[2]", psrc, sbp.B, 2, k * tb + 2 * tb),
            ("S(0)[4] -> P(sum)[8]", s0, sbp.P_SUM, 8, tb + 8 * tb)]:
        dq = sbp.empty_global(shape, bf16, dst_sig, q, device=device)
        avg, best = time_op(lambda: sbp.sbp_boxing(src_g, dq), device)
        res.append(_hbm_entry("disjoint placements: " + name + " bf16 [8192,8192]", nbytes, avg, best, peaks))
        del dq
    del psrc, s0
    torch.cuda.empty_cache()
    k, rows, dim, batch = 8, opts.emb_rows, 128, opts.emb_batch
    ids = dg.zipf_ids(1005, 1, (batch, 26), rows, 1.05, device)
    table = sbp.SbpTensor((rows, dim), torch.float32, sbp.S(1),
                          [dg.uniform(1005, 200 + r, (rows, dim // k), -0.05, 0.05, torch.float32, device) for r in range(k)])
    idt = sbp.SbpTensor((batch, 26), torch.int64, sbp.B, [ids] * k)
    out_b = sbp.empty_global((batch, 26, dim), torch.float32, sbp.B, k, device=device)
    n, row_b = batch * 26, dim * 4
    avg, best = time_op(lambda: sbp.sbp_embedding(table, idt, out_b), device)
    res.append(_hbm_entry("embedding, table S(1): fused gather -> B (8 replicas written)", n * 8 + n * row_b + k * n * row_b,
                          avg, best, peaks))
    # backward of the row-split lookup: dense table gradient S(0) (zero fill + atomic scatter-add)
    g1 = out_b.locals[0]
    del table, out_b
    torch.cuda.empty_cache()
    go = sbp.SbpTensor((batch, 26, dim), torch.float32, sbp.B, [g1] * k)
    gt = sbp.empty_global((rows, dim), torch.float32, sbp.S(0), k, device=device)
    avg, best = time_op(lambda: sbp.sbp_embedding_backward(go, idt, gt), device, iters=5)
    res.append(_hbm_entry("embedding backward: table gradient S(0) (zero fill + scatter-add)",
                          rows * row_b + n * 8 + n * row_b, avg, best, peaks))
    return res


def section_cliffs(sbp, device, peaks, opts):
    """Shapes that miss the fast paths' rules, next to their nearest regular neighbour: a bf16 product
    whose shard width is not a multiple of 8 elements (the TMA stride rule), and P(sum) -> B with shard
    counts outside {1, 2, 4, 8} (the unrolled reductions)."""
    bf16 = torch.bfloat16
    res = []
    k, M, K = 8, 8192, 4096
    X = dg.normal(1003, 0, (M, K), 0.0, 1.0, bf16, device)
    x = sbp.SbpTensor((M, K), bf16, sbp.B, [X] * k)
    for width in (336, 333):
        N = k * width
        w = sbp.SbpTensor((K, N), bf16, sbp.S(1), [dg.normal(1003, 80 + r, (K, width), 0.0, 0.02, bf16, device) for r in range(k)])
        y = sbp.empty_global((M, N), bf16, sbp.S(1), k, device=device)
        ws = torch.empty(max(1, sbp.sbp_matmul_workspace_bytes(x, w, y)), dtype=torch.uint8, device=device)
        avg, best, form = time_mm(sbp, lambda: sbp.sbp_matmul(x, w, y, 0, ws), device)
        res.append(_tensor_entry(f"bf16 product (B,S(1))->S(1), [8192,4096] x [4096,{N}], shard width {width}"
                                 + ("" if width % 8 == 0 else " (not a multiple of 8)"),
                                 2.0 * M * K * N, avg, best, peaks, form, kernel=None))
        del w, y, ws
    del x, X
    torch.cuda.empty_cache()
    shape = (8192, 8192)
    tb = shape[0] * shape[1] * 2
    for kk in (3, 4, 16):
        src = sbp.SbpTensor(shape, bf16, sbp.P_SUM, [dg.normal(SEED, 400 + r, shape, 0.0, 1.0, bf16, device) for r in range(kk)])
        dst = sbp.empty_global(shape, bf16, sbp.B, kk, device=device)
        avg, best = time_op(lambda: sbp.sbp_boxing(src, dst), device, iters=5)
        res.append(_hbm_entry(f"P(sum)->B, k={kk}, bf16 [8192,8192]", 2 * kk * tb, avg, best, peaks))
        del src, dst
        torch.cuda.empty_cache()
    return res


# workload configuration (1-5) each operator section belongs to (None: beyond the five)
SECTION_CONFIG = {"softmax": 4, "classifier": 4, "mlp": 3, "embedding": 5, "extras": None, "cliffs": None}

# kernel behind an HBM-bound line, by the start of its name (tensor-bound lines: matmul_tc_kernel)
HBM_KERNELS = [
    ("softmax-xent on bf16", "xent_partial_kernel+xent_combine_kernel"),
    ("softmax-xent backward", "xent_backward_kernel"),
    ("embedding fused", "embedding_kernel<fused>"),
    ("embedding unfused", "embedding_kernel+box_tile_kernel"),
    ("embedding, table S(1)", "embedding_s1_kernel"),
    ("embedding backward", "embedding_backward_kernel"),
    ("MLP P(sum)->B", "box_tile_kernel"),
    ("S(0)->P(sum)", "box_scatter_kernel"), ("B->P(sum)", "box_scatter_kernel"),
    ("S(0) fp32 -> B bf16", "box_gather_cast_kernel"),
    ("disjoint placements", "box_disjoint_kernel"),
    ("P(sum)->B, k=", "box_tile_kernel"),
]


def run_operator_sections(sbp, device, peaks, opts):
    which = opts.ops
    out = []
    table = {"softmax": section_softmax, "classifier": section_classifier_gemm, "mlp": section_mlp,
             "embedding": section_embedding, "extras": section_extras, "cliffs": section_cliffs}
    for w in [w.strip() for w in which.split(",") if w.strip()]:
        fn = table[w]
        try:
            res = fn(sbp, device, peaks, opts)
        except sbp.SbpError as e:            # an operator the library refuses is reported, not hidden
            res = [{"op": fn.__name__, "error": str(e)}]
        for e in res:
            if e.get("config") is None:
                e["config"] = SECTION_CONFIG[w]
            if e.get("kernel") is None and "op" in e:
                e["kernel"] = next((kn for pre, kn in HBM_KERNELS if e["op"].startswith(pre)), None)
        out.extend(res)
        torch.cuda.empty_cache()
    return out


def roofline_configs(per, ops):
    """Compact per-config roofline lines for the record: config 2's transforms, then every operator
    line of configs 3-5.  frac = achieved / peak with the peak of the line's own bound; HBM lines
    with an ncu capture also carry the DRAM-byte figure (achieved_dram, frac_dram)."""
    out = []
    for t in per:
        e = {"config": 2, "line": t["transform"], "kernel": "box_tile_kernel", "bound": "hbm", "ms": t["ms"],
             "work": t["bytes"], "achieved": t["gbs"], "unit": "GB/s", "frac": t["frac_measured"],
             "ms_back_to_back": t.get("ms_back_to_back"), "frac_back_to_back": t.get("frac_measured_back_to_back")}
        tr = ncu_traffic(t["transform"])
        if tr is not None:
            e["traffic"] = tr
            e["achieved_dram"] = tr / (t["ms"] * 1e-3) / 1e9
        out.append(e)
    for o in ops or []:
        if "error" in o or o.get("config") is None:
            continue
        e = {"config": o["config"], "line": o["op"], "kernel": o.get("kernel"), "bound": o["bound"], "ms": o["ms"],
             "work": o.get("bytes", o.get("flops")), "achieved": o["achieved"], "unit": o["unit"],
             "frac": o["frac_measured"]}
        for key in ("traffic", "achieved_dram", "frac_dram", "hbm_gbs", "hbm_frac_measured", "frac_sustained", "form"):
            if o.get(key) is not None:
                e[key] = o[key]
        out.append(e)
    return out


# ------------------------------------------------------------------------------ CPU baseline (oracle)

def oracle_sweep_sample(rows: int):
    """Times the CPU oracle, as it stands, on the first `rows` rows of the sweep workload.
    Returns (bytes processed, seconds, threads used)."""
    import numpy as np
    from oracle import sbp_oracle as O
    k = SWEEP_K
    shape = (rows, SWEEP_SHAPE[1])
    T = dg.normal(SEED, 0, shape, 0.0, 1.0, torch.bfloat16).float().numpy()
    P = [dg.normal(SEED, 10 + r, shape, 0.0, 1.0, torch.bfloat16).float().numpy() for r in range(k)]
    srcs = {"P": (P, O.PSUM), "S0": (O.to_locals(T, O.S0, k), O.S0), "S1": (O.to_locals(T, O.S1, k), O.S1),
            "B": (O.to_locals(T, O.B, k), O.B)}
    dsts = {"B": O.B, "S0": O.S0, "S1": O.S1}
    nbytes = 0
    t0 = time.perf_counter()
    for _, s, d, units in TRANSFORMS:
        loc, sg = srcs[s]
        out = O.boxing(loc, sg, dsts[d], "bf16")
        assert len(out) == k
        nbytes += units * rows * SWEEP_SHAPE[1] * 2
    return nbytes, time.perf_counter() - t0, 1


def host_cores():
    """Cores this process may run on (what the oracle has at its disposal)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def blas_threads():
    """Threads numpy's BLAS uses for the oracle's float64 matrix products; everything else in the
    oracle is single-threaded numpy."""
    try:
        from threadpoolctl import threadpool_info
        n = [int(i.get("num_threads", 1)) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_config_samples(gen_device="cpu"):
    """The CPU oracle, as it stands, timed on a bounded sample of configs 3, 4 and 5 (config 2 is
    oracle_sweep_sample).  Inputs are drawn on gen_device and copied to the host before the clock
    starts.  Rows / lookups are independent, so a sample's time scales linearly to the full
    workload; `scale` is that factor and `full_s_extrapolated` = seconds * scale."""
    import numpy as np
    from oracle import sbp_oracle as O
    bf16, f32 = torch.bfloat16, torch.float32
    k = 8
    cores, bt = host_cores(), blas_threads()

    def host(t):
        return t.float().cpu().numpy() if t.dtype == bf16 else t.cpu().numpy()

    out = []

    def add(config, what, work, unit_work, secs, scale, threads, sample):
        out.append({"config": config, "what": what, "seconds": secs, "value": work / secs / 1e9,
                    "unit": unit_work, "scale": scale, "full_s_extrapolated": secs * scale,
                    "cores": cores, "threads_used": threads, "sample": sample})

    # config 3: Y = GeLU(X W1) W2 in float64 on the first rows of X (all columns)
    M, H, F, rows = 8192, 4096, 16384, 128
    X = host(dg.normal(1003, 0, (rows, H), 0.0, 1.0, bf16, gen_device))
    W1 = np.concatenate([host(dg.normal(1003, 10 + r, (H, F // k), 0.0, 0.02, bf16, gen_device)) for r in range(k)], axis=1)
    W2 = np.concatenate([host(dg.normal(1003, 30 + r, (F // k, H), 0.0, 0.02, bf16, gen_device)) for r in range(k)], axis=0)
    t0 = time.perf_counter()
    Y = O.mlp_logical(X, W1, W2)
    secs = time.perf_counter() - t0
    assert Y.shape == (rows, H)
    add(3, "MLP block GeLU(X W1) W2, float64", 2 * 2.0 * rows * H * F, "GFLOP/s", secs, M / rows, bt,
        f"first {rows} of {M} rows of X, all of W1 and W2")
    del W1, W2, Y

    # config 4: one shard's logits product in float64, then the split softmax-xent on a row sample
    R, feat, classes = 512, 512, 1 << 20
    Fm = host(dg.normal(1004, 0, (R, feat), 0.0, 1.0, bf16, gen_device))
    W0 = host(dg.normal(1004, 40, (feat, classes // k), 0.0, 0.01, bf16, gen_device))
    t0 = time.perf_counter()
    Z0 = O.matmul_logical(Fm, W0)
    secs = time.perf_counter() - t0
    assert Z0.shape == (R, classes // k)
    add(4, "classifier logits F W, float64", 2.0 * R * feat * (classes // k), "GFLOP/s", secs, k, bt,
        f"shard 0 of {k} of the class-split weight, all {R} rows")
    del W0, Z0
    rs = 64
    sigma = (512 ** 0.5) * 0.01
    zl = [host(dg.normal(1004, 10 + r, (rs, classes // k), 0.0, sigma, bf16, gen_device)) for r in range(k)]
    labels = dg.integers(1004, 1, (rs,), 0, classes, gen_device).cpu().numpy()
    t0 = time.perf_counter()
    m, S, loss = O.softmax_xent_split(zl, labels)
    secs = time.perf_counter() - t0
    assert loss.shape == (rs,)
    add(4, "split softmax cross entropy on bf16 logits", rs * classes * 2.0, "GB/s", secs, R / rs, 1,
        f"first {rs} of {R} rows, all {classes} classes over {k} shards")
    del zl

    # config 5: row-split lookup -> P(sum) partials, then their fixed-order sum (the unfused path the
    # paper describes), on a table and batch of 1/8 the size
    trows, dim, batch = 1 << 21, 128, 2048
    table = [host(dg.uniform(1005, 100 + r, (trows // k, dim), -0.05, 0.05, f32, gen_device)) for r in range(k)]
    ids = dg.zipf_ids(1005, 1, (batch, 26), trows, 1.05, gen_device).cpu().numpy()
    t0 = time.perf_counter()
    parts = O.embedding_partials(table, ids)
    got = O.boxing(parts, O.PSUM, O.B, "f32")
    secs = time.perf_counter() - t0
    assert got[0].shape == (batch, 26, dim)
    n = batch * 26
    add(5, "embedding gather -> P(sum) partials, then P(sum) -> B", n * 8.0 + 2.0 * n * dim * 4, "GB/s", secs,
        65536 / batch, 1,
        f"{batch} of 65536 samples x 26 fields, table of {trows} rows (1/8 of 2^24) over {k} shards; "
        "bytes counted as ids + rows gathered + one result written")
    return out


# ------------------------------------------------------------------------------ ranks

def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: what a multi-rank number is computed from."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(world: int, ms_step: float) -> float:
    """Every rank runs its own replica of the sweep (no collective on the data path), so the
    job moves world x step_bytes() in the slowest rank's step time."""
    return world * step_bytes() / (ms_step * 1e-3) / 1e9


# ------------------------------------------------------------------------------ main

def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-ops", action="store_true", help="skip the sharded-operator sections (N = 1 only)")
    ap.add_argument("--ops", default="softmax,classifier,mlp,embedding,extras,cliffs",
                    help="comma-separated operator sections to run: softmax, classifier, mlp, embedding, extras, cliffs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run-cpu", action="store_true",
                    help="rank plumbing only, on CPU over gloo: launch, world-size check, barrier, slowest-rank timing, "
                         "rank 0's JSON line; no kernel runs and the line is not a measurement")
    ap.add_argument("--op-iters", type=int, default=None, help="timed repeats per operator line (default 5-10)")
    ap.add_argument("--op-warmup", type=int, default=None, help="warm-up repeats per operator line (default 3; >= 3 for a valid number)")
    ap.add_argument("--copy-engine", type=int, default=0)
    ap.add_argument("--emb-rows", type=int, default=1 << 24, help="embedding table rows (smaller = profiling-sized case)")
    ap.add_argument("--emb-batch", type=int, default=65536, help="embedding batch (x 26 fields)")
    ap.add_argument("--xent-rows", type=int, default=512, help="rows of the softmax / classifier sections")
    ap.add_argument("--rows", type=int, default=SWEEP_SHAPE[0],
                    help="rows of the logical sweep tensor (smaller = a profiling-sized case, not the benchmark)")
    args = ap.parse_args()
    OP_REPEATS["iters"], OP_REPEATS["warmup"] = args.op_iters, args.op_warmup
    return args


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    rows = 256
    for _ in range(max(args.warmup, 0)):
        oracle_sweep_sample(64)
    total_b, total_s = 0, 0.0
    for _ in range(args.steps):
        b, s, cores = oracle_sweep_sample(rows)
        total_b += b
        total_s += s
    value = total_b / total_s / 1e9
    sample = f"first {rows} of {SWEEP_SHAPE[0]} rows of every local tensor, all 7 transforms, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_s / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "boxing sweep bf16 [8192,8192] k=4, 7 transforms (CPU oracle on a row sample)"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": host_cores(), "threads_used": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


def launch_ranks_if_needed(args):
    """--gpus N is the number of ranks.  Started plainly (no WORLD_SIZE) with N > 1, this process
    starts the N ranks itself through torch.distributed.run on 127.0.0.1 and returns their exit
    code; started by a launcher, the launcher's WORLD_SIZE must equal N (exit code 2 otherwise).
    Returns None when this process is a rank (or the only one) and should go on."""
    ws = os.environ.get("WORLD_SIZE")
    if ws is not None:
        if int(ws) != args.gpus:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={ws} ranks\n")
            return 2
        return None
    if args.gpus <= 1 or args.impl == "reference":     # the oracle arm is one CPU process whatever N is
        return None
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def dry_run_cpu(args):
    """The multi-rank plumbing of the benchmark with the GPU work left out: gloo process group on CPU,
    barrier, a stand-in per-rank time (rank r: 1 + r ms), slowest rank's time, whole-job value, one
    JSON line from rank 0.  Exists so that the launch path can be tested where there is no GPU."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("gloo")
        dist.barrier()
    ms_step = max_over_ranks(1.0 + rank, dist, torch.device("cpu"))
    if dist is not None:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "dry_run": True, "value": whole_job_gbs(world, ms_step), "unit": "GB/s",
                          "n_gpus": args.gpus, "world_size": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms_step, "scaling": "weak", "data": "none (dry run on CPU)"}))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    args = parse()
    global SWEEP_SHAPE
    SWEEP_SHAPE = (args.rows, SWEEP_SHAPE[1])
    rc = launch_ranks_if_needed(args)
    if rc is not None:
        return rc
    if args.impl == "reference":
        return reference_arm(args)
    if args.dry_run_cpu:
        return dry_run_cpu(args)

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    import paper_2110_15032_b200 as sbp
    sbp.load_library()
    sbp.sbp_boxing_set_copy_engine(args.copy_engine)
    peaks = measured_peaks()

    T, src, work = build_sweep(sbp, device)
    for _ in range(max(args.warmup, 3)):
        run_sweep(sbp, work)
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(work) + 1)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    # Timed region: exactly K steps between two events, nothing else on the stream.
    launches0 = sbp.sbp_launch_count()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for s in range(args.steps):
        run_sweep(sbp, work)
    end.record()
    barrier()
    launches = sbp.sbp_launch_count() - launches0
    ms_total = max_over_ranks(start.elapsed_time(end), dist, device)
    ms_step = ms_total / args.steps
    value = whole_job_gbs(world, ms_step)
    # Per-transform durations: the same K steps once more, now with an event record between
    # consecutive launches.  They are taken apart from the timed region because the event records
    # themselves hold the stream up between launches (measured with a pair around every launch:
    # 648 us a step against 611 us without).
    for s in range(args.steps):
        run_sweep(sbp, work, events[s])
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    sbp.sbp_check_device_errors()

    per = []
    for i, (name, _, _, nbytes) in enumerate(work):
        ms = [events[s][i].elapsed_time(events[s][i + 1]) for s in range(args.steps)]
        avg = sum(ms) / len(ms)
        per.append({"transform": name, "bytes": nbytes, "ms": avg, "best_ms": min(ms),
                    "gbs": nbytes / (avg * 1e-3) / 1e9,
                    "frac_measured": nbytes / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "frac_nominal": nbytes / (avg * 1e-3) / 1e9 / NOMINAL_HBM_GBS})
    # The same transform launched fifty times back to back between one pair of events: the kernel's
    # own rate, without the event record between launches (about 3 us each) that the figures
    # above carry.  Sources and destinations together exceed L2 for every transform.
    for i, (name, s_, d_, nbytes) in enumerate(work):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(50):
            sbp.sbp_boxing(s_, d_)
        b.record()
        torch.cuda.synchronize()
        ms10 = a.elapsed_time(b) / 50
        per[i]["ms_back_to_back"] = ms10
        per[i]["frac_measured_back_to_back"] = nbytes / (ms10 * 1e-3) / 1e9 / peaks["hbm_gbs"]
    dom = max(per, key=lambda p: p["ms"])
    roofline = {"bound": "hbm", "kernel": "box_tile_kernel (" + dom["transform"] + ")",
                "achieved": dom["gbs"], "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
                "unit": "GB/s", "frac": dom["gbs"] / peaks["hbm_gbs"], "traffic": ncu_traffic(dom["transform"]),
                "traffic_captured_at": NCU_TRAFFIC_CAPTURED_AT}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"boxing sweep: logical bf16 [{SWEEP_SHAPE[0]},{SWEEP_SHAPE[1]}] N(0,1), k=4, 7 transforms per step",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 GPU, k=4 logical shards",
                   "l2": "inputs larger than L2: a step streams 3.4 GB through distinct buffers between repeats",
                   "l2_ops": "operator sections: L2 flushed before every timed launch (256 MB written, then 256 MB read so that the flush's own dirty lines are not written back during the launch)",
                   "copy_engine": args.copy_engine},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "transforms": per,
    }

    if rank == 0:
        line["clocks"] = clocks

    # end-to-end: the same sweep through the host-buffer entry point, copies inside the region
    if args.e2e_steps > 0:
        e2e = e2e_sweep(sbp, src, work, device, args.e2e_steps, dist)
        e2e["value"] *= world
        line["e2e"] = e2e
    else:
        line["e2e"] = None

    if rank == 0 and world == 1:
        if not args.no_ops:
            del T, src, work
            torch.cuda.empty_cache()
            line["ops"] = run_operator_sections(sbp, device, peaks, args)
        # every config's lines inside the roofline object (the sweep's dominant kernel stays on top)
        line["roofline"]["configs"] = roofline_configs(per, line.get("ops"))
        if not args.no_cpu_baseline:
            rows = SWEEP_SHAPE[0]
            nbytes, secs, threads = oracle_sweep_sample(rows)
            base = {"value": nbytes / secs / 1e9, "unit": "GB/s", "cores": host_cores(), "threads_used": threads,
                    "kind": "oracle",
                    "sample": f"config 2: first {rows} of {SWEEP_SHAPE[0]} rows of every local tensor, "
                              f"all 7 transforms once ({secs:.1f} s)"}
            cfgs = [{"config": 2, "what": "boxing sweep, 7 transforms", "seconds": secs, "value": base["value"],
                     "unit": "GB/s", "scale": 1.0, "full_s_extrapolated": secs, "cores": base["cores"],
                     "threads_used": threads, "sample": "the whole sweep"}]
            cfgs.extend(oracle_config_samples(device))
            base["configs"] = cfgs
            line["cpu_baseline"] = base
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

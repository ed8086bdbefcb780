#!/usr/bin/env python
"""Benchmark of the densify hot path: GB/s and rows/s on B200, fraction of the HBM roofline,
the CPU oracle beside it.

One "step" is one pass of the whole hot path (index histogram, scan, radix placement, row
reduction with the fused dense add) over one batch of synthetic IndexedSlices.  The headline
workload is the R=64 concatenated-slices configuration (the largest of the configurations,
2.7 GB of value rows, far larger than L2); the other configurations are reported in
"all_configs" of the same JSON line.

  python bench.py                       # 1 GPU, headline + all configurations + CPU oracle baseline
  python bench.py --workload big        # another headline workload
  python bench.py --impl reference      # the CPU oracle as the reference arm
  torchrun ... bench.py --gpus N        # N independent replicas (the path has no exchange step)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1905_04035_b200.workloads import make_workload  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
SIZEOF = {"f32": 4, "bf16": 2, "i32": 4, "i64": 8}
FALLBACK_HBM_GBS = 6650.0
ALL_CONFIGS = ("tiny", "base", "big", "r64", "sweep_uniform", "sweep_zipf", "sweep_same")
# the two workloads with a stated bar: at least this fraction of the measured HBM peak for the whole step
TARGETS = {"big": 0.70, "r64": 0.70}
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "k_reduce_rows_dram_traffic.txt")
KERNEL_SOURCES = [os.path.join(ROOT, "paper_1905_04035_b200", "csrc", f) for f in ("dst_reduce_kernels.cu", "dst_common.cuh")]


def kernel_dram_traffic(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the row-reduction kernel on `workload`, as an ncu
    capture recorded it in profiles/k_reduce_rows_dram_traffic.txt (lines: workload, bytes, sha256 over the kernel's
    source file and the header it shares with the other kernels, at capture time).  None when there is no record for
    the workload, or when the sources have changed since: counters of another kernel are not this kernel's traffic."""
    import hashlib
    try:
        h = hashlib.sha256()
        for path in KERNEL_SOURCES:
            with open(path, "rb") as f:
                h.update(f.read())
        now = h.hexdigest()
        for line in open(TRAFFIC_FILE):
            f = line.split()
            if len(f) >= 3 and not line.startswith("#") and f[0] == workload:
                return float(f[1]) if f[2] == now else None
    except OSError:
        pass
    return None


def algorithmic_bytes(w) -> int:
    """Values read once + dense_in read once + out written once + indices read once."""
    n = w.n_rows_total
    b = n * w.d * SIZEOF[w.value_dtype] + w.vocab * w.d * SIZEOF[w.out_dtype] + n * SIZEOF[w.index_dtype]
    if w.dense_in is not None:
        b += w.vocab * w.d * SIZEOF[w.out_dtype]
    return b


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# ---------------------------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="dst_clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
def _dev_tensor(arr, kind, device):
    import torch
    if kind == "bf16":
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)


class DeviceProblem:
    """A workload resident in HBM, with enough rotating copies that consecutive steps never
    find their inputs in L2."""

    def __init__(self, w, device, n_sets=None):
        import torch
        import paper_1905_04035_b200 as dst
        self.w, self.device = w, device
        tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32, "i64": torch.int64}
        self.balg = algorithmic_bytes(w)
        if n_sets is None:
            n_sets = 1 if self.balg >= 4 * L2_BYTES else int(min(8, -(-4 * L2_BYTES // max(self.balg, 1))))
        self.n_sets = n_sets
        self.sets = []
        for _ in range(n_sets):
            slices = [(_dev_tensor(i, w.index_dtype, device), _dev_tensor(v, w.value_dtype, device))
                      for i, v in zip(w.indices, w.values)]
            dense = _dev_tensor(w.dense_in, w.out_dtype, device) if w.dense_in is not None else None
            out = torch.empty(w.vocab, w.d, dtype=tdt[w.out_dtype], device=device)
            self.sets.append((slices, dense, out))
        self.eng = dst.Densifier(w.n_rows_total, w.R, w.d, w.vocab, index_dtype=tdt[w.index_dtype],
                                 value_dtype=tdt[w.value_dtype], out_dtype=tdt[w.out_dtype], device=device,
                                 want_unique=True)
        self.flush = None
        if n_sets * self.balg < 4 * L2_BYTES:
            self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)

    def step(self, k: int):
        slices, dense, out = self.sets[k % self.n_sets]
        self.eng(slices, dense, out)

    def l2_policy(self) -> str:
        if self.n_sets == 1 and self.flush is None:
            return "inputs larger than L2 (%.0f MB per step vs 126 MB L2)" % (self.balg / 1e6)
        if self.flush is None:
            return "rotating %d buffer sets (%.0f MB total) so no step finds its inputs in L2" % (
                self.n_sets, self.n_sets * self.balg / 1e6)
        return "L2 flushed by a 252 MB write between steps"


def time_device(prob: DeviceProblem, steps: int, warmup: int, dist_ctx=None, clocks: ClockSampler = None):
    """K steps bracketed by sync (+ barrier); returns (total ms, per-step reduce-kernel ms list, launches)."""
    import torch
    import paper_1905_04035_b200 as dst
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in kev:
        a.record(); b.record()        # creates the underlying CUDA events
    for k in range(warmup):
        if prob.flush is not None:
            prob.flush.zero_()
        prob.step(k)
    torch.cuda.synchronize()
    if dist_ctx is not None:
        dist_ctx.barrier()
    if clocks is not None:
        clocks.start()
    launches0 = dst.dst_kernel_launches()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ev = []
    torch.cuda.synchronize()
    if prob.flush is None:
        t0.record()
        for k in range(steps):
            dst.dst_profile_events(*kev[k])
            prob.step(warmup + k)
        t1.record()
        torch.cuda.synchronize()
        total_ms = t0.elapsed_time(t1)
    else:
        # the flush is not part of the step: time each step on its own and add them up
        for k in range(steps):
            prob.flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            dst.dst_profile_events(*kev[k])
            a.record(); prob.step(warmup + k); b.record()
            step_ev.append((a, b))
        torch.cuda.synchronize()
        total_ms = float(sum(a.elapsed_time(b) for a, b in step_ev))
    dst.dst_profile_events(None, None)
    launches = dst.dst_kernel_launches() - launches0
    clock_info = clocks.stop() if clocks is not None else None
    if dist_ctx is not None:
        dist_ctx.barrier()
    kernel_ms = [a.elapsed_time(b) for a, b in kev]
    return total_ms, kernel_ms, launches, clock_info


def time_device_graph(prob: DeviceProblem, steps: int, warmup: int, dist_ctx=None, clocks: ClockSampler = None):
    """The same K steps, each step replayed from a CUDA graph captured once per buffer set (the library
    allocates nothing and never synchronises, so a call can be captured as it is).  Returns total ms."""
    import torch
    import paper_1905_04035_b200 as dst
    prob.step(0)                       # first call outside capture (sets kernel attributes)
    torch.cuda.synchronize()
    graphs = []
    for slices, dense, out in prob.sets:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            prob.eng(slices, dense, out)
        graphs.append(g)
    for k in range(warmup):
        if prob.flush is not None:
            prob.flush.zero_()
        graphs[k % prob.n_sets].replay()
    torch.cuda.synchronize()
    if dist_ctx is not None:
        dist_ctx.barrier()
    if clocks is not None:
        clocks.start()
    launches0 = dst.dst_kernel_launches()
    torch.cuda.synchronize()
    if prob.flush is None:
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for k in range(steps):
            graphs[(warmup + k) % prob.n_sets].replay()
        t1.record()
        torch.cuda.synchronize()
        total_ms = t0.elapsed_time(t1)
    else:
        ev = []
        for k in range(steps):
            prob.flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); graphs[(warmup + k) % prob.n_sets].replay(); b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        total_ms = float(sum(a.elapsed_time(b) for a, b in ev))
    clock_info = clocks.stop() if clocks is not None else None
    if dist_ctx is not None:
        dist_ctx.barrier()
    del graphs
    return total_ms, clock_info


def time_device_warm(prob: DeviceProblem, steps: int, warmup: int):
    """The warm figure beside the cold one: the same call replayed on ONE buffer set with no flush, so
    whatever part of the inputs fits in L2 is still there.  Returns ms per step."""
    import torch
    slices, dense, out = prob.sets[0]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        prob.eng(slices, dense, out)
    for _ in range(warmup):
        g.replay()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(steps):
        g.replay()
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / steps


def time_accumulate(device, steps: int, warmup: int, seed: int):
    """The accumulation strategies of the paper on one rank's gradients of the tied weight (the big
    configuration: the dense projection gradient and the two embedding lookups): Algorithm 1 gathers,
    Algorithm 2 and Listing 1 convert and reduce; and the plain reduce branch on 2 and 8 dense tensors.
    One library call per step, L2 flushed between steps, CUDA events around each call."""
    import torch
    import paper_1905_04035_b200 as dst
    peak, _ = measured_peak()
    w = make_workload("big", seed=seed)
    tdt = {"f32": torch.float32, "i64": torch.int64}
    dense = _dev_tensor(w.dense_in, w.out_dtype, device)
    slices = [(_dev_tensor(i, w.index_dtype, device), _dev_tensor(v, w.value_dtype, device))
              for i, v in zip(w.indices, w.values)]
    n, d, vocab = w.n_rows_total, w.d, w.vocab
    out_dense = torch.empty(vocab, d, device=device)
    out_idx = torch.empty(vocab + n, dtype=torch.int64, device=device)
    out_val = torch.empty(vocab + n, d, device=device)
    ws = torch.empty(dst.dst_workspace_bytes(n, len(slices), d, vocab), dtype=torch.uint8, device=device)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
    more = [torch.randn(vocab, d, device=device) * 0.02 for _ in range(7)]
    dense_bytes, value_bytes, index_bytes = vocab * d * 4, n * d * 4, n * 8
    cases = [
        ("stock (Algorithm 1)", dst.DST_ACC_STOCK, [dense] + slices,
         2 * (dense_bytes + value_bytes) + 2 * index_bytes + vocab * 8),       # copies: read + write; indices of the dense rows written
        ("proposed (Algorithm 2)", dst.DST_ACC_PROPOSED, [dense] + slices, 2 * dense_bytes + value_bytes + index_bytes),
        ("sparse_as_dense (Listing 1)", dst.DST_ACC_SPARSE_AS_DENSE, [dense] + slices, 2 * dense_bytes + value_bytes + index_bytes),
        ("reduce, 2 dense", dst.DST_ACC_PROPOSED, [dense, more[0]], 3 * dense_bytes),
        ("reduce, 8 dense", dst.DST_ACC_PROPOSED, [dense] + more, 9 * dense_bytes),
    ]
    rows = []
    for name, strategy, grads, nbytes in cases:
        def call():
            return dst.dst_accumulate(grads, d, vocab, strategy, out_dense=out_dense, out_indices=out_idx,
                                      out_values=out_val, workspace=ws)
        for _ in range(warmup):
            flush.zero_(); plan = call()
        ev = []
        l0 = dst.dst_kernel_launches()
        for _ in range(steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); call(); b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
        rows.append({"strategy": name, "branch": plan["branch"], "out_kind": plan["out_kind"],
                     "out_bytes": plan["out_bytes"], "ms_per_step": ms, "algorithmic_bytes": nbytes,
                     "gbs": nbytes / ms / 1e6, "frac_of_hbm_peak": nbytes / ms / 1e6 / peak,
                     "gpu_launches_per_step": (dst.dst_kernel_launches() - l0) / steps})
    # the SGD step fused into the same pass, against densify followed by a separate update of the weight
    weight = torch.randn(vocab, d, device=device)
    lr = 0.1

    def fused():
        dst.dst_densify_apply_sgd(slices, d, vocab, dense, weight, lr, ws)

    def separate():
        dst.dst_densify_concat(slices, d, vocab, dense, out_dense, ws)
        weight.add_(out_dense, alpha=-lr)

    # the optimizers that keep state: every state tensor is read and written once in the same pass; the separate
    # arm is densify followed by the library's fused multi-tensor optimizer on the dense gradient
    mom_buf, adam_m, adam_v = torch.zeros(vocab, d, device=device), torch.zeros(vocab, d, device=device), torch.zeros(vocab, d, device=device)
    wparam = torch.nn.Parameter(weight.clone())
    wparam.grad = out_dense
    opt_mom = torch.optim.SGD([wparam], lr=lr, momentum=0.9)
    opt_adam = torch.optim.Adam([wparam], lr=1e-3, fused=True)
    step_no = [0]

    def fused_momentum():
        dst.dst_densify_apply(slices, d, vocab, dense, weight, ws, kind=dst.DST_OPT_MOMENTUM, lr=lr, momentum=0.9, state1=mom_buf)

    def fused_adam():
        step_no[0] += 1
        dst.dst_densify_apply(slices, d, vocab, dense, weight, ws, kind=dst.DST_OPT_ADAM, lr=1e-3, step=step_no[0],
                              state1=adam_m, state2=adam_v)

    def separate_momentum():
        dst.dst_densify_concat(slices, d, vocab, dense, out_dense, ws)
        opt_mom.step()

    def separate_adam():
        dst.dst_densify_concat(slices, d, vocab, dense, out_dense, ws)
        opt_adam.step()

    for name, fn, nbytes in (("densify + SGD step, fused (dst_densify_apply_sgd)", fused, 3 * dense_bytes + value_bytes + index_bytes),
                             ("densify, then a separate weight update", separate, 5 * dense_bytes + value_bytes + index_bytes),
                             ("densify + momentum step, fused (dst_densify_apply)", fused_momentum, 5 * dense_bytes + value_bytes + index_bytes),
                             ("densify, then torch.optim.SGD(momentum)", separate_momentum, 8 * dense_bytes + value_bytes + index_bytes),
                             ("densify + Adam step, fused (dst_densify_apply)", fused_adam, 7 * dense_bytes + value_bytes + index_bytes),
                             ("densify, then torch.optim.Adam(fused)", separate_adam, 10 * dense_bytes + value_bytes + index_bytes)):
        for _ in range(warmup):
            flush.zero_(); fn()
        ev = []
        l0 = dst.dst_kernel_launches()
        for _ in range(steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
        rows.append({"strategy": name, "branch": "convert+reduce+apply", "out_kind": "weight", "out_bytes": dense_bytes,
                     "ms_per_step": ms, "algorithmic_bytes": nbytes, "gbs": nbytes / ms / 1e6,
                     "frac_of_hbm_peak": nbytes / ms / 1e6 / peak,
                     "gpu_launches_per_step": (dst.dst_kernel_launches() - l0) / steps})
    return rows


def time_ranks(device, R: int, steps: int, warmup: int, seed: int):
    """R ranks' gradients of the tied weight (per rank the dense projection gradient and two lookups of 5,000 rows,
    the paper's 64-process case) accumulated three ways: in one pass (dst_densify_batch), in two (the dense
    tensors summed first, the slices densified onto the sum), and as the gathered form of Algorithm 1 (everything
    concatenated as IndexedSlices, then densified).  Bytes: what each way has to move at least."""
    import torch
    import paper_1905_04035_b200 as dst
    peak, _ = measured_peak()
    vocab, d, n_lookup = 33708, 1024, 5000
    g = torch.Generator(device=device); g.manual_seed(seed)
    p = 1.0 / torch.arange(1, vocab + 1, dtype=torch.float64) ** 1.1
    cdf = torch.cumsum(p / p.sum(), 0).to(device)
    ranks = []
    for r in range(R):
        dense = torch.randn(vocab, d, device=device, generator=g) * 0.02
        sl = []
        for _ in range(2):
            idx = torch.searchsorted(cdf, torch.rand(n_lookup, device=device, generator=g, dtype=torch.float64)).clamp_(max=vocab - 1)
            sl.append((idx, torch.randn(n_lookup, d, device=device, generator=g) * 0.02))
        ranks.append((dense, sl))
    n = 2 * n_lookup * R
    out = torch.empty(vocab, d, device=device)
    ws = torch.empty(dst.dst_workspace_bytes(n, 2 * R, d, vocab), dtype=torch.uint8, device=device)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
    dense_b, value_b = vocab * d * 4, n * d * 4
    all_slices = [s for _, sl in ranks for s in sl]
    denses = [dn for dn, _ in ranks]
    g_idx = torch.empty(R * vocab + n, dtype=torch.int64, device=device)
    g_val = torch.empty(R * vocab + n, d, device=device)
    ws_g = torch.empty(dst.dst_workspace_bytes(R * vocab + n, 1, d, vocab), dtype=torch.uint8, device=device)

    def one_pass():
        dst.dst_densify_batch(ranks, d, vocab, out, ws)

    def two_pass():
        dst.dst_accumulate(denses, d, vocab, dst.DST_ACC_PROPOSED, out_dense=out)          # no workspace: the sum passes
        dst.dst_densify_concat(all_slices, d, vocab, out, out, ws)

    def gathered():
        dst.dst_accumulate(denses + all_slices, d, vocab, dst.DST_ACC_STOCK, out_indices=g_idx, out_values=g_val)
        dst.dst_densify(g_idx, g_val, d, vocab, None, out, ws_g)

    gather_b = (R * vocab + n) * (d * 4 + 8)
    rows = []
    for name, fn, nbytes in (("one pass (dst_densify_batch)", one_pass, R * dense_b + value_b + dense_b),
                             ("two passes (sum of dense tensors, then densify onto it)", two_pass,
                              R * dense_b + value_b + dense_b + 2 * dense_b * ((R + 6) // 7)),
                             ("gathered form (Algorithm 1), then densified", gathered, 3 * gather_b + dense_b)):
        for _ in range(warmup):
            flush.zero_(); fn()
        ev = []
        for _ in range(steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            ev.append((a, b))
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
        rows.append({"way": name, "ms_per_step": ms, "bytes_moved_at_least": nbytes, "gbs": nbytes / ms / 1e6,
                     "frac_of_hbm_peak": nbytes / ms / 1e6 / peak})
    rep = dst.dst_bytes_report([2 * n_lookup] * R, d, vocab)       # per rank: both lookups
    return {"R": R, "vocab": vocab, "d": d, "rows_per_lookup": n_lookup, "ways": rows,
            "gathered_bytes": gather_b, "dense_bytes": dense_b, "bytes_report": rep}


def time_reduce(w, device, steps: int, warmup: int, dist_ctx):
    """The data-parallel step of Section 4 with its exchange: each rank densifies its own slices into the dense
    tensor, which a sum all-reduce (NCCL) then combines.  Device time, max over ranks."""
    import torch
    from paper_1905_04035_b200.reduce import densify_then_reduce, exchange_bytes
    from paper_1905_04035_b200.replicas import combine_over_ranks
    prob = DeviceProblem(w, device, n_sets=1)
    slices, dense, out = prob.sets[0]
    step = lambda: densify_then_reduce(lambda: prob.eng(slices, dense, out), out, dist_ctx)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    dist_ctx.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    agg = combine_over_ranks(t0.elapsed_time(t1) / steps, prob.balg, w.n_rows_total, dist_ctx, device)
    world = dist_ctx.get_world_size()
    esz = {"f32": 4, "bf16": 2}[w.out_dtype]
    isz = {"i32": 4, "i64": 8}[w.index_dtype]
    return {"ms_per_step": agg["ms_per_step"], "ranks": world, "collective": "all_reduce(sum) of [vocab, d]",
            **exchange_bytes(w.vocab, w.d, esz, w.n_rows_total, isz, world)}


def time_e2e(w, device, steps: int, warmup: int):
    """Same metric through the host entry point: pinned host buffers, H2D and D2H inside the timed region."""
    import torch
    import paper_1905_04035_b200 as dst
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32, "i64": torch.int64}

    def host(arr, kind):
        t = torch.from_numpy(arr.view(np.int16)).view(torch.bfloat16) if kind == "bf16" else torch.from_numpy(arr)
        return t.pin_memory()

    slices = [(host(i, w.index_dtype), host(v, w.value_dtype)) for i, v in zip(w.indices, w.values)]
    dense = host(w.dense_in, w.out_dtype) if w.dense_in is not None else None
    out = torch.empty(w.vocab, w.d, dtype=tdt[w.out_dtype]).pin_memory()
    res = torch.zeros(6, dtype=torch.int32).pin_memory()
    n = w.n_rows_total
    staging = torch.empty(dst.dst_host_staging_bytes(n, w.d, w.vocab, tdt[w.index_dtype], tdt[w.value_dtype],
                                                     tdt[w.out_dtype]), dtype=torch.uint8, device=device)
    ws = torch.empty(dst.dst_workspace_bytes(n, 1, w.d, w.vocab, tdt[w.index_dtype], tdt[w.value_dtype],
                                             tdt[w.out_dtype]), dtype=torch.uint8, device=device)
    for _ in range(warmup):
        dst.dst_densify_concat_host(slices, w.d, w.vocab, dense, out, staging, ws, res)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        dst.dst_densify_concat_host(slices, w.d, w.vocab, dense, out, staging, ws, res)
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / steps
    h2d = n * (w.d * SIZEOF[w.value_dtype] + SIZEOF[w.index_dtype]) + (out.numel() * out.element_size() if dense is not None else 0)
    d2h = out.numel() * out.element_size() + 24
    assert res[0].item() == 0
    return ms, int(h2d), int(d2h)


# ---------------------------------------------------------------------------------------------
# the CPU oracle arm (reference arm and cpu_baseline leg)
# ---------------------------------------------------------------------------------------------
def time_oracle(w, max_rows=None, repeats=1, threads=False):
    """Time the oracle as it stands on (a prefix of every slice of) the workload.  Single thread.

    ``threads=True`` times the other CPU baseline instead: the same loop in fp32, one thread per
    block of columns, on every core this process may use."""
    import oracle
    idx, val = w.indices, w.values
    sample = "full workload"
    if max_rows is not None and w.n_rows_total > max_rows:
        keep = max(1, max_rows // max(w.R, 1))
        idx = [i[:keep] for i in idx]
        val = [v[:keep] for v in val]
        sample = "first %d rows of each of the %d slices (%d of %d rows), full [vocab, d] dense add and output" % (
            keep, w.R, keep * w.R, w.n_rows_total)
    n = int(sum(i.shape[0] for i in idx))
    best = None
    cores = 1
    for _ in range(repeats):
        t = time.perf_counter()
        if threads:
            cores = oracle.densify_threads(idx, val, w.d, w.vocab, w.dense_in, value_dtype=w.value_dtype,
                                           out_dtype=w.out_dtype)[2]
        else:
            oracle.densify(idx, val, w.d, w.vocab, w.dense_in, value_dtype=w.value_dtype, out_dtype=w.out_dtype)
        dt = time.perf_counter() - t
        best = dt if best is None else min(best, dt)
    b = n * w.d * SIZEOF[w.value_dtype] + w.vocab * w.d * SIZEOF[w.out_dtype] + n * SIZEOF[w.index_dtype]
    if w.dense_in is not None:
        b += w.vocab * w.d * SIZEOF[w.out_dtype]
    return {"seconds": best, "rows": n, "bytes": b, "gbs": b / best / 1e9, "rows_per_s": n / best, "sample": sample,
            "cores": cores}


# ---------------------------------------------------------------------------------------------
def run_config(name, device, steps, warmup, seed, dist_ctx=None, clocks=None, want_e2e=False, e2e_steps=5,
               scale=1.0, use_graph=True):
    import torch
    peak, peak_src = measured_peak()
    w = make_workload(name, seed=seed, scale=scale)
    prob = DeviceProblem(w, device)
    # eager calls first (per-kernel events, launch count), then the timed steps replayed from CUDA graphs
    eager_ms, kernel_ms, launches, _ = time_device(prob, steps, warmup, dist_ctx, None)
    res = prob.eng.read_result()
    if use_graph:
        total_ms, clock_info = time_device_graph(prob, steps, warmup, dist_ctx, clocks)
    else:
        total_ms, _, _, clock_info = time_device(prob, steps, warmup, dist_ctx, clocks)
    ms = total_ms / steps
    warm_ms = time_device_warm(prob, steps, warmup) if use_graph and dist_ctx is None else None
    kms = float(np.mean(kernel_ms))
    # small inputs: the row-reduction kernel runs beside the index cluster (and, in the eager pass that times it, after
    # it: an event between the two launches undoes the overlap), so its own time is not a roofline figure
    overlapped = w.n_rows_total <= 65535 and w.vocab <= 65536 and w.R <= 64 and w.n_rows_total <= w.vocab
    out = {
        "workload": name, "ms_per_step": ms, "gbs": prob.balg / ms / 1e6, "rows_per_s": w.n_rows_total / ms * 1e3,
        "frac_of_hbm_peak": prob.balg / ms / 1e6 / peak, "algorithmic_bytes": prob.balg,
        "reduce_kernel_ms": kms, "reduce_kernel_gbs": None if overlapped else prob.balg / kms / 1e6,
        "reduce_kernel_frac": None if overlapped else prob.balg / kms / 1e6 / peak, "launches": launches, "l2": prob.l2_policy(),
        "eager_ms_per_step": eager_ms / steps, "warm_ms_per_step": warm_ms, "cuda_graph": bool(use_graph),
        "n_unique": res["n_unique"], "max_segment": res["max_segment"], "status": res["status"],
        "peak_gbs": peak, "peak_source": peak_src, "clocks": clock_info, "w": w,
    }
    del prob
    torch.cuda.empty_cache()
    if want_e2e:
        ems, h2d, d2h = time_e2e(w, device, e2e_steps, 2)
        out["e2e"] = {"ms_per_step": ems, "gbs": out["algorithmic_bytes"] / ems / 1e6, "h2d": h2d, "d2h": d2h}
        torch.cuda.empty_cache()
    return out


def reference_arm(args):
    """The oracle, timed on the host cores, as the reference arm (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.workload, seed=args.seed)
    # Every step is the whole workload when warm-up and timed steps then end within about three minutes (judged
    # by the first step); otherwise every step is a prefix of every slice sized to that budget.
    cap = args.reference_rows
    times = []
    info = None
    for k in range(args.warmup + args.steps):
        info = time_oracle(w, max_rows=cap)
        if k == 0 and cap is None and info["seconds"] * (args.warmup + args.steps) > 180.0:
            cap = max(1024, int(w.n_rows_total * 180.0 / (info["seconds"] * (args.warmup + args.steps))))
            info = time_oracle(w, max_rows=cap)
        if k >= args.warmup:
            times.append(info["seconds"])
    sec = float(np.mean(times))
    gbs = info["bytes"] / sec / 1e9
    line = {
        "impl": "reference", "metric": "densify_GBps", "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "recipe": w.recipe, "vocab": w.vocab, "d": w.d, "R": w.R,
                   "n_rows_total": w.n_rows_total},
        "rows_per_s": info["rows"] / sec,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": info["sample"]},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="dst", choices=["dst", "reference"])
    ap.add_argument("--workload", default="r64", choices=ALL_CONFIGS)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--headline-only", action="store_true", help="skip the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager calls instead of CUDA-graph replays")
    ap.add_argument("--accumulate-only", action="store_true",
                    help="only the accumulation-strategy and fused-SGD calls (prints their rows, one GPU)")
    ap.add_argument("--scale", type=float, default=1.0,
                    help="shrink the rows per slice (profiling captures on a small case); 1.0 = the named configuration")
    ap.add_argument("--reduce", action="store_true",
                    help="with more than one rank: also time the step followed by a sum all-reduce of the dense output "
                         "(a separate row; the headline stays the independent replicas, with no collective)")
    ap.add_argument("--reference-rows", type=int, default=None,
                    help="rows of the workload the reference arm processes per step (default: all of them, unless the "
                         "run would then take more than about three minutes)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "dst" else args.warmup

    if args.impl == "reference":
        reference_arm(args)
        return

    import torch
    import torch.distributed as dist
    import paper_1905_04035_b200 as dst

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the densify path")
    dst.load_library()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist_ctx = None
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
        dist_ctx = dist

    if args.accumulate_only:
        if rank == 0:
            print(json.dumps({"accumulate": time_accumulate(device, min(args.steps, 50), args.warmup, args.seed)}))
        return

    # every rank is an independent replica with its own seed (the path has no exchange step)
    from paper_1905_04035_b200.replicas import combine_over_ranks, replica_seed
    seed = replica_seed(args.seed, rank)
    clocks = ClockSampler(local_rank) if rank == 0 else None
    head = run_config(args.workload, device, args.steps, args.warmup, seed, dist_ctx, clocks,
                      want_e2e=not args.no_e2e, scale=args.scale, use_graph=not args.no_graph)
    w = head.pop("w")

    agg = combine_over_ranks(head["ms_per_step"], head["algorithmic_bytes"], w.n_rows_total, dist_ctx, device)
    e2e = None
    if "e2e" in head:
        eagg = combine_over_ranks(head["e2e"]["ms_per_step"], head["algorithmic_bytes"], w.n_rows_total, dist_ctx, device)
        e2e = {"value": eagg["gbs"], "unit": "GB/s", "h2d_bytes_per_step": head["e2e"]["h2d"],
               "d2h_bytes_per_step": head["e2e"]["d2h"], "ms_per_step": eagg["ms_per_step"]}

    reduce_row = None
    if args.reduce and world > 1:
        reduce_row = time_reduce(w, device, min(args.steps, 50), args.warmup, dist_ctx)

    others = []
    targets = {}
    if args.workload in TARGETS and args.scale == 1.0:
        targets[args.workload] = {"ms_per_step": head["ms_per_step"], "frac": head["frac_of_hbm_peak"], "bar": TARGETS[args.workload]}
    if rank == 0 and world == 1 and not args.headline_only:
        for name in ALL_CONFIGS:
            if name == args.workload:
                continue
            # the other configurations get enough steps for a stable figure whatever the headline's step count
            r = run_config(name, device, max(min(args.steps, 200), 100), args.warmup, args.seed, use_graph=not args.no_graph)
            r.pop("w"); r.pop("clocks")
            others.append({"workload": name, "ms_per_step": r["ms_per_step"], "frac": r["frac_of_hbm_peak"],
                           "kernel_frac": r["reduce_kernel_frac"], "status": r["status"]})
            if name in TARGETS:
                targets[name] = {"ms_per_step": r["ms_per_step"], "frac": r["frac_of_hbm_peak"], "bar": TARGETS[name]}

    accumulate = None
    ranks_rows = None
    if rank == 0 and world == 1 and not args.headline_only:
        accumulate = time_accumulate(device, min(args.steps, 50), args.warmup, args.seed)
        torch.cuda.empty_cache()
        ranks_rows = []
        for R in (8, 64):
            ranks_rows.append(time_ranks(device, R, min(args.steps, 10), 3, args.seed))
            torch.cuda.empty_cache()

    cpu = cpu_threads = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        info = time_oracle(w, max_rows=None if w.n_rows_total <= 700000 else 700000)
        cpu = {"value": info["gbs"], "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": info["sample"],
               "seconds": info["seconds"], "rows_per_s": info["rows_per_s"]}
        info = time_oracle(w, max_rows=None if w.n_rows_total <= 700000 else 700000, repeats=2, threads=True)
        cpu_threads = {"value": info["gbs"], "unit": "GB/s", "cores": info["cores"],
                       "kind": "fp32 loop, one thread per block of columns", "sample": info["sample"],
                       "seconds": info["seconds"], "rows_per_s": info["rows_per_s"]}

    if rank == 0:
        rep = dst.dst_bytes_report([int(i.shape[0]) for i in w.indices], w.d, w.vocab,
                                   *[{"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32,
                                      "i64": torch.int64}[k] for k in (w.index_dtype, w.value_dtype, w.out_dtype)])
        line = {
            "metric": "densify_GBps", "value": agg["gbs"], "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": agg["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32" if w.value_dtype == "f32" else "bf16 in, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": args.workload, "recipe": w.recipe, "vocab": w.vocab, "d": w.d, "R": w.R,
                       "n_rows_total": w.n_rows_total, "l2": head["l2"], "replicas": world, "scale": args.scale,
                       "timed_as": "CUDA-graph replay of one library call per step" if head["cuda_graph"]
                       else "eager library calls"},
            "eager_ms_per_step": head["eager_ms_per_step"], "warm_ms_per_step": head["warm_ms_per_step"],
            "rows_per_s": agg["rows_per_s"], "frac_of_hbm_peak": agg["gbs"] / world / head["peak_gbs"],
            "roofline": {"bound": "hbm", "achieved": head["reduce_kernel_gbs"], "peak": head["peak_gbs"],
                         "unit": "GB/s", "frac": head["reduce_kernel_frac"],
                         "traffic": kernel_dram_traffic(args.workload) if args.scale == 1.0 else None,
                         "kernel": "k_reduce_rows", "of": head["peak_source"],
                         "kernel_ms": head["reduce_kernel_ms"],
                         # whole-step fraction of the measured peak on the two workloads with a stated bar
                         "targets": targets},
            "e2e": e2e, "gpu_launches": head["launches"], "clocks": head["clocks"],
            "cpu_baseline": cpu, "cpu_baseline_threads": cpu_threads, "bytes_report": rep,
            "parity": {"status": head["status"], "n_unique": head["n_unique"], "max_segment": head["max_segment"]},
            "accumulate": accumulate, "ranks": ranks_rows, "reduce": reduce_row, "all_configs": others,
        }
        print(json.dumps(line))
    if dist_ctx is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

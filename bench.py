#!/usr/bin/env python
"""Benchmark of the LoMA attention hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
  1. index maps (loma_layout_index, loma_generation_index) on the device
  2. loma_masked_attn_fwd on the 4608-token training layout
     (B4 H32 D128 bf16, c=4, t=16, 32 chunks of [64|16|64])
  3. one generation cycle on the compressed cache (B32 H32 D128 bf16, 8192
     memory entries): tc = 64 x loma_decode_attn with the tail growing from 0 to
     63, then one loma_compress_step (16 memory queries + in-place compaction)

`value` is the masked-attention useful TFLOP/s (4*D FLOPs per allowed
(query, key) pair; allowed pairs counted from Eq. 1-3 in closed form); the
decode GB/s (the other half of the metric) is in `decode_attn`, and the
roofline object describes the decode kernel, which dominates the step's time.

At N=1 a second loop with the same --steps/--warmup times the two largest
workloads as steps of their own: the 69632-token forward (B1 H32 D128, c=8,
t=32, 128 chunks: the tensor-bound case) and one generation cycle at the
higher ratio (B64 H32 D128, 16384 memory entries, c=8, t=16: 128 decodes +
1 compress), reported in `large_workloads` with a roofline object per kernel.

  python bench.py --profile-case NAME [--reps N]   runs a cut-down launch of one
kernel (same per-(batch, head) shapes, fewer pairs; inputs larger than L2, a few GB
at most) and exits (what a profiler capture wraps).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With --gpus N > 1 (launched under torch.distributed.run, one rank per GPU) every
rank runs the same per-GPU workload on its own (batch, head) shard: no
collective is on the data path, scaling is weak, and times are the max over
ranks.
"""

from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LoMA masked-attn useful TFLOP/s; compressed decode-attn HBM GB/s vs roofline"

# workload: training-layout forward (configs[1]) + generation cycle (configs[2])
FWD = dict(B=4, H=32, D=128, n=32, c=4, t=16)
GEN = dict(B=32, H=32, D=128, c=4, t=16, mem_len=8192)


def allowed_pairs(n: int, c: int, t: int, prior_mem: bool = False) -> int:
    """Ones in the Eq. 2 mask of n chunks, counted block by block (Eq. 1, Eq. 3)."""
    tc = t * c
    per_chunk = tc * (tc + 1) // 2 + t * (tc + t) + tc * (t + 1)
    cross = tc * t + (t * t if prior_mem else 0)
    return n * per_chunk + cross * n * (n - 1) // 2


def _device_pause(torch, cycles: int) -> None:
    """Keeps the GPU busy for `cycles` clocks on the current stream (a spin kernel that ships with torch),
    so that the calls enqueued right after it are already queued when the GPU reaches them.  Without it
    (should a torch build lack the helper) short kernels are merely timed with the host's launch path included."""
    spin = getattr(torch.cuda, "_sleep", None)
    if spin is not None:
        spin(int(cycles))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for nme, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), power_w_max=max(power),
                    samples=len(sm), reasons=sorted(reasons))


# --------------------------------------------------------------------------- ours

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2401_09486_b200 import binding as L
    from paper_2401_09486_b200 import build, multi_gpu, synthetic

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run, one rank per GPU")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()
    L.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- inputs (seeded, synthetic; rank-dependent seeds) ----------------
    f, g = FWD, GEN
    tc_f = f["c"] * f["t"]
    S = f["n"] * (2 * tc_f + f["t"])
    std = 1.0 / math.sqrt(f["D"])
    bf = torch.bfloat16
    q, k, v = (synthetic.big_normal_(torch.empty(f["B"], f["H"], S, f["D"], dtype=bf, device=dev), multi_gpu.rank_seed(1000, rank, i),
                                     std) for i in range(3))
    o = torch.empty_like(q)
    tc_g = g["c"] * g["t"]
    cap = g["mem_len"] + tc_g + g["t"]
    kc = synthetic.big_normal_(torch.empty(g["B"], g["H"], cap, g["D"], dtype=bf, device=dev), multi_gpu.rank_seed(2000, rank), std)
    vc = synthetic.big_normal_(torch.empty(g["B"], g["H"], cap, g["D"], dtype=bf, device=dev), multi_gpu.rank_seed(2001, rank), std)
    # one (q, k_new, v_new) triple per decode step of the cycle, and the memory-token triple
    dq, dk, dv = (synthetic.big_normal_(torch.empty(tc_g, g["B"], g["H"], 1, g["D"], dtype=bf, device=dev),
                                        multi_gpu.rank_seed(2100, rank, i), std) for i in range(3))
    do = torch.empty_like(dq)
    qm, km, vm = (synthetic.big_normal_(torch.empty(g["B"], g["H"], g["t"], g["D"], dtype=bf, device=dev),
                                        multi_gpu.rank_seed(2200, rank, i), std) for i in range(3))
    om = torch.empty_like(qm)
    ws_bytes = max(16, L.loma_decode_workspace_bytes(g["B"], g["H"], g["D"], cap),
                   L.loma_compress_workspace_bytes(g["B"], g["H"], g["D"], g["t"], g["mem_len"], 0))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    idx_fwd = [torch.empty(S, dtype=torch.int32, device=dev) for _ in range(5)]
    idx_gen = [torch.empty(tc_g, dtype=torch.int32, device=dev) for _ in range(3)]
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream
    lib = L.lib()
    import ctypes
    P = lambda x: ctypes.c_void_p(x.data_ptr())

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(marks=None):
        """All hot-path calls of one step, on the current stream, through the C ABI."""
        def mark(name):
            if marks is not None:
                e = ev(); e.record(stream); marks.append((name, e))
        mark("start")
        rc = lib.loma_layout_index(f["n"], f["c"], f["t"], 0, 0, *[P(x) for x in idx_fwd], 1, st)
        rc |= lib.loma_generation_index(tc_g, g["c"], g["t"], *[P(x) for x in idx_gen], 1, st)
        # A device-side pause of ~0.08 ms (counted in the step and in the index phase): by the time it ends the
        # host has enqueued the forward, so the two events around the forward see the kernel and not the host's
        # launch path (an idle GPU otherwise waits ~12 us for the call to arrive, 7 % of this kernel's run time).
        _device_pause(torch, 150_000)
        mark("index")
        L.loma_masked_attn_fwd(q, k, v, o, None, f["n"], f["c"], f["t"], 0, 0, 0.0, stream)
        mark("masked_fwd")
        for j in range(tc_g):
            L.loma_decode_attn(dq[j], dk[j], dv[j], kc, vc, do[j], None, g["mem_len"] + j, ws, 0, 0.0, stream)
        mark("decode")
        L.loma_compress_step(qm, km, vm, kc, vc, om, None, g["mem_len"], g["c"], g["t"], ws, 0, 0.0, stream)
        mark("compress")
        if rc != 0:
            raise RuntimeError("index map call failed")

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = L.loma_launch_count()
    all_marks = []
    e0, e1 = ev(), ev()
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        marks = []
        step(marks)
        all_marks.append(marks)
    e1.record(stream)
    barrier()
    total_ms = e0.elapsed_time(e1)
    launches = L.loma_launch_count() - launches0
    clocks = sampler.stop()
    assert L.loma_device_status() == 0

    phase_ms = {}
    for marks in all_marks:
        for (n0, a), (n1, b) in zip(marks[:-1], marks[1:]):
            phase_ms[n1] = phase_ms.get(n1, 0.0) + a.elapsed_time(b)
    phase_ms = {kk: vv / args.steps for kk, vv in phase_ms.items()}

    # max over ranks of every time
    total_ms, t_index, t_fwd, t_dec, t_cmp = multi_gpu.max_over_ranks(
        [total_ms] + [phase_ms[x] for x in ("index", "masked_fwd", "decode", "compress")], dev)
    ms_per_step = total_ms / args.steps

    # ---------------- e2e: host buffers, copies inside the timed region ----------------
    pin = lambda x: torch.empty(x.shape, dtype=x.dtype, device="cpu", pin_memory=True).copy_(x)
    hq, hk, hv = pin(q), pin(k), pin(v)
    ho = torch.empty(o.shape, dtype=o.dtype, device="cpu", pin_memory=True)
    hdq, hdk, hdv = pin(dq), pin(dk), pin(dv)
    hdo = torch.empty(do.shape, dtype=do.dtype, device="cpu", pin_memory=True)
    hqm, hkm, hvm = pin(qm), pin(km), pin(vm)
    hom = torch.empty(om.shape, dtype=om.dtype, device="cpu", pin_memory=True)
    nbytes = lambda *xs: sum(x.numel() * x.element_size() for x in xs)
    h2d = nbytes(hq, hk, hv, hdq, hdk, hdv, hqm, hkm, hvm)
    d2h = nbytes(ho, hdo, hom)

    def e2e_step(marks):
        def mark(name):
            e = ev(); e.record(stream); marks.append((name, e))
        mark("start")
        q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True)
        L.loma_masked_attn_fwd(q, k, v, o, None, f["n"], f["c"], f["t"], 0, 0, 0.0, stream)
        ho.copy_(o, non_blocking=True)
        mark("masked_fwd")
        for j in range(tc_g):
            dq[j].copy_(hdq[j], non_blocking=True); dk[j].copy_(hdk[j], non_blocking=True)
            dv[j].copy_(hdv[j], non_blocking=True)
            L.loma_decode_attn(dq[j], dk[j], dv[j], kc, vc, do[j], None, g["mem_len"] + j, ws, 0, 0.0, stream)
            hdo[j].copy_(do[j], non_blocking=True)
        mark("decode")
        qm.copy_(hqm, non_blocking=True); km.copy_(hkm, non_blocking=True); vm.copy_(hvm, non_blocking=True)
        L.loma_compress_step(qm, km, vm, kc, vc, om, None, g["mem_len"], g["c"], g["t"], ws, 0, 0.0, stream)
        hom.copy_(om, non_blocking=True)
        mark("compress")

    e2e_step([])
    barrier()
    e2e_steps = max(1, min(args.steps, 3))
    e2e_fwd = e2e_dec = e2e_tot = 0.0
    for _ in range(e2e_steps):
        marks = []
        e2e_step(marks)
        torch.cuda.synchronize()
        e2e_fwd += marks[0][1].elapsed_time(marks[1][1])
        e2e_dec += marks[1][1].elapsed_time(marks[2][1])
        e2e_tot += marks[0][1].elapsed_time(marks[3][1])
    e2e_fwd, e2e_dec, e2e_tot = multi_gpu.max_over_ranks(
        [e2e_fwd / e2e_steps, e2e_dec / e2e_steps, e2e_tot / e2e_steps], dev)

    # ---------------- figures ----------------
    peaks = load_peaks()
    pairs = allowed_pairs(f["n"], f["c"], f["t"])
    fwd_flops = 4.0 * f["D"] * pairs * f["B"] * f["H"]                 # per GPU
    fwd_bytes = 4.0 * q.numel() * 2                                    # Q, K, V read + O written once
    fwd_tflops = multi_gpu.job_throughput(fwd_flops, world, t_fwd) / 1e12
    # decode: algorithmic bytes = every visible K and V row read once (cache_len + 1 rows per (b,h))
    dec_rows = sum(g["mem_len"] + j + 1 for j in range(tc_g))
    dec_bytes_cycle = 2.0 * dec_rows * g["B"] * g["H"] * g["D"] * 2
    dec_bytes_launch = dec_bytes_cycle / tc_g
    dec_ms_launch = t_dec / tc_g
    dec_gbs = dec_bytes_launch / (dec_ms_launch * 1e-3) / 1e9          # per GPU
    # compress (paper variant): tail K,V read + q,k,v_mem read + o_mem written + compaction written
    bh = g["B"] * g["H"]
    cmp_bytes = bh * g["D"] * 2.0 * (2 * tc_g + 3 * g["t"] + g["t"] + 2 * g["t"])
    cmp_gbs = cmp_bytes / (t_cmp * 1e-3) / 1e9

    out = {
        "metric": METRIC,
        "value": fwd_tflops,
        "unit": "TFLOP/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16",
        "data": "synthetic",
        "config": {
            "workload": ("masked fwd B4 H32 D128 c4 t16 n32 S4608 + generation cycle B32 H32 D128 c4 t16 "
                         "mem 8192: 64 decode + 1 compress"),
            "masked_fwd": dict(f, S=S, std="1/sqrt(D)"),
            "generation": dict(g, cap=cap, decode_steps=tc_g),
            "l2": "inputs larger than L2 (604 MB forward tensors, 4.3 GB cache streamed by every decode)",
            "per_gpu_batch": "fixed (weak scaling over (batch, head) shards, no collective)",
        },
        "phases_ms": {"index_maps": t_index, "masked_attn_fwd": t_fwd, "decode_cycle": t_dec, "compress_step": t_cmp},
        "decode_attn": {"value": world * dec_gbs, "unit": "GB/s", "ms_per_call": dec_ms_launch,
                        "bytes_per_call": dec_bytes_launch, "frac_of_measured_hbm": dec_gbs / peaks["hbm_gbs"],
                        "frac_of_8tbs": dec_gbs / 8000.0},
        "masked_attn": {"useful_tflops": fwd_tflops, "ms": t_fwd, "useful_flops": fwd_flops,
                        "compulsory_bytes": fwd_bytes, "gbs": fwd_bytes / (t_fwd * 1e-3) / 1e9,
                        "frac_of_measured_hbm": fwd_bytes / (t_fwd * 1e-3) / 1e9 / peaks["hbm_gbs"],
                        "frac_of_measured_bf16": fwd_tflops / world / peaks["bf16_tflops"],
                        "ms_x_sm_ghz": (t_fwd * clocks["sm_mhz"] / 1e3) if clocks.get("sm_mhz") else None},
        "compress": {"ms": t_cmp, "bytes": cmp_bytes, "gbs": cmp_gbs,
                     "frac_of_measured_hbm": cmp_gbs / peaks["hbm_gbs"],
                     "note": "timed in place after the 64 decodes of the cycle"},
        "roofline": {"kernel": "decode_splitkv_kernel<128, false> (+ decode_merge_kernel<128>), per loma_decode_attn call", "bound": "hbm",
                     "achieved": dec_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": dec_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     # dram__bytes_read + write of one launch: captured on the B8 case and scaled by the (b,h) count, 1024 / 256
                     "traffic": DECODE_TRAFFIC_B8_L8224 * (g["B"] * g["H"]) / 256.0,
                     "traffic_source": "ncu small case x4"},
        "roofline_other_kernels": [
            {"kernel": "masked_attn_tc_kernel<128, false>", "workload": "4608-token layout", "bound": "hbm",
             "achieved": fwd_bytes / (t_fwd * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
             "frac": fwd_bytes / (t_fwd * 1e-3) / 1e9 / peaks["hbm_gbs"],
             # dram__bytes_read.sum + dram__bytes_write.sum of one launch on one batch element of this layout x B
             "traffic": FWD_SHORT_TRAFFIC_B1 * f["B"],
             "tensor_frac_of_measured_bf16_useful": fwd_tflops / world / peaks["bf16_tflops"]},
            {"kernel": "compress_one_stage_kernel<128, 4>", "workload": "B32 H32 mem 8192, default variant", "bound": "hbm",
             "achieved": cmp_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": cmp_gbs / peaks["hbm_gbs"],
             # dram__bytes_read.sum + dram__bytes_write.sum of one launch at this very size (the 12.6 MB it writes stay in L2)
             "traffic": COMPRESS_TRAFFIC_B32, "note": "59 MB in one launch of 1024 CTAs, four resident per SM: two waves"},
        ],
        "e2e": {"value": world * fwd_flops / (e2e_fwd * 1e-3) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_tot,
                "masked_fwd_ms": e2e_fwd, "decode_cycle_ms": e2e_dec,
                "decode_gbs": world * dec_bytes_cycle / (e2e_dec * 1e-3) / 1e9},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1 and not args.no_extras:
        # free the step's tensors, then the two largest workloads as steps of their own (same --steps / --warmup)
        del q, k, v, o, kc, vc, dq, dk, dv, do, hq, hk, hv, ho, hdq, hdk, hdv, hdo
        torch.cuda.empty_cache()
        out["large_workloads"] = large_workloads(L, synthetic, torch, dev, peaks, args.steps, max(args.warmup, 3),
                                                 clocks.get("sm_mhz"))
        out["roofline_large"] = [out["large_workloads"]["masked_fwd_69632"]["roofline"],
                                 out["large_workloads"]["generation_B64_16k"]["roofline"]]
        # further shapes, timed a few times each (context, not the metric)
        out["other_workloads"] = other_workloads(L, synthetic, torch, dev, peaks)
    if rank == 0:
        out["cpu_baseline"] = cpu_baseline()
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def other_workloads(L, synthetic, torch, dev, peaks):
    """Device-timed figures for the long training layout (69632 tokens) and the
    higher-ratio generation shape (B64, 16384 memory entries): median of 5 after 3 warm-ups."""
    bf = torch.bfloat16
    stream = torch.cuda.current_stream()

    def timed(fn, reps=5, warm=3):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            # keep the GPU busy for ~0.3 ms while the host enqueues the events and the call: the interval
            # between the events is then device time only (no wait for the host's launch path)
            _device_pause(torch, 600_000)
            a.record(stream); fn(); b.record(stream); torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    res = {}
    B, H, D, n, c, t = 1, 32, 128, 128, 8, 32
    S = n * (2 * c * t + t)
    std = 1.0 / math.sqrt(D)
    q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 3000 + i, std) for i in range(3))
    o = torch.empty_like(q)
    ms = timed(lambda: L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t, 0, 0, 0.0, stream))
    flops = 4.0 * D * allowed_pairs(n, c, t) * B * H
    res["masked_fwd_69632"] = {"config": dict(B=B, H=H, D=D, n=n, c=c, t=t, S=S), "ms": ms,
                               "useful_tflops": flops / (ms * 1e-3) / 1e12,
                               "frac_of_measured_bf16": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                               "gbs": 4.0 * q.numel() * 2 / (ms * 1e-3) / 1e9,
                               "note": "single calls, each after an idle gap (the GPU's clock may not have ramped up): "
                                       "the steady-state figure of this workload is large_workloads.masked_fwd_69632"}

    def backward(tag, B, H, n, c, t, q, k, v, o):
        # gradients of the same layout (useful FLOPs: five products of the allowed pairs, 10*D per pair)
        S = q.shape[2]
        lse = torch.empty((B, H, S), dtype=torch.float32, device=dev)
        L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t, 0, 0, 0.0, stream)
        d_o = synthetic.big_normal_(torch.empty_like(q), 3050, std)
        dq, dk, dv = (torch.empty_like(q) for _ in range(3))
        wsb = torch.empty(L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t), dtype=torch.uint8, device=dev)
        ms_b = timed(lambda: L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, 0, 0, wsb, 0.0, stream))
        fl = 10.0 * D * allowed_pairs(n, c, t) * B * H
        nbytes = 8.0 * q.numel() * 2     # q, k, v, o, dO read, dq, dk, dv written, once each
        res[tag] = {"config": dict(B=B, H=H, D=D, n=n, c=c, t=t, S=S), "ms": ms_b,
                    "useful_tflops": fl / (ms_b * 1e-3) / 1e12,
                    "frac_of_measured_bf16": fl / (ms_b * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "gbs": nbytes / (ms_b * 1e-3) / 1e9, "frac_of_measured_hbm": nbytes / (ms_b * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "kernels": "bwd_delta + masked_attn_bwd_dq_tc + masked_attn_bwd_dkv_tc"}

    backward("masked_bwd_69632", B, H, n, c, t, q, k, v, o)
    del q, k, v, o
    torch.cuda.empty_cache()
    B, H, n, c, t = 4, 32, 32, 4, 16
    S = n * (2 * c * t + t)
    q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 3060 + i, std) for i in range(3))
    o = torch.empty_like(q)
    backward("masked_bwd_4608", B, H, n, c, t, q, k, v, o)
    # rotary embedding of Q and K at the layout's position ids: Q and K read and written once
    ms = timed(lambda: L.loma_rope_apply(q, k, n, c, t, 0, 0, 0.0, 0, stream))
    nbytes = 4.0 * q.numel() * 2
    res["rope_4608"] = {"config": dict(B=B, H=H, D=D, n=n, c=c, t=t, S=S), "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9,
                        "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "kernel": "rope_kernel"}
    del q, k, v, o
    torch.cuda.empty_cache()
    # the compression settings of the paper's Table 1 / Fig. 7 sweeps (c = 2, short memory zones), ~4600 tokens
    for (n2, c2, t2) in ((230, 2, 4), (115, 2, 8), (29, 2, 32)):
        B, H = 4, 32
        S = n2 * (2 * c2 * t2 + t2)
        q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 3070 + i, std) for i in range(3))
        o = torch.empty_like(q)
        ms = timed(lambda: L.loma_masked_attn_fwd(q, k, v, o, None, n2, c2, t2, 0, 0, 0.0, stream))
        fl = 4.0 * D * allowed_pairs(n2, c2, t2) * B * H
        res[f"masked_fwd_c{c2}_t{t2}"] = {"config": dict(B=B, H=H, D=D, n=n2, c=c2, t=t2, S=S), "ms": ms,
                                          "useful_tflops": fl / (ms * 1e-3) / 1e12,
                                          "gbs": 4.0 * q.numel() * 2 / (ms * 1e-3) / 1e9,
                                          "frac_of_measured_hbm": 4.0 * q.numel() * 2 / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        del q, k, v, o
    torch.cuda.empty_cache()
    B, H, c, t, mem_len = 64, 32, 8, 16, 16384
    tc = c * t
    cap = (mem_len + tc + t + 63) // 64 * 64      # a whole number of 64-row pages (for the paged variant below)
    kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3100, std)
    vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3101, std)
    q1, k1, v1 = (synthetic.big_normal_(torch.empty(B, H, 1, D, dtype=bf, device=dev), 3102 + i, std) for i in range(3))
    o1 = torch.empty_like(q1)
    qm, km, vm = (synthetic.big_normal_(torch.empty(B, H, t, D, dtype=bf, device=dev), 3110 + i, std) for i in range(3))
    om = torch.empty_like(qm)
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cap),
                         L.loma_compress_workspace_bytes(B, H, D, t, mem_len, 1)), dtype=torch.uint8, device=dev)
    cache_len = mem_len + tc // 2
    ms = timed(lambda: L.loma_decode_attn(q1, k1, v1, kc, vc, o1, None, cache_len, ws, 0, 0.0, stream))
    nbytes = 2.0 * (cache_len + 1) * B * H * D * 2
    res["decode_B64_16k"] = {"config": dict(B=B, H=H, D=D, c=c, t=t, cache_len=cache_len), "ms": ms,
                             "gbs": nbytes / (ms * 1e-3) / 1e9,
                             "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # the same decode with one length per sequence, spread over the last chunk's tail positions
    lens = torch.tensor([mem_len + (7 * b) % tc for b in range(B)], dtype=torch.int32, device=dev)
    max_len = mem_len + tc - 1
    ms = timed(lambda: L.loma_decode_attn_ragged(q1, k1, v1, kc, vc, o1, None, lens, max_len, ws, 0, 0.0, stream))
    nbytes = 2.0 * float((lens.double() + 1).sum()) * H * D * 2
    res["decode_ragged_B64_16k"] = {"config": dict(B=B, H=H, D=D, c=c, t=t, lens="mem_len + (7 b) mod tc"), "ms": ms,
                                    "gbs": nbytes / (ms * 1e-3) / 1e9,
                                    "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # the same ragged decode over a paged cache: the cache tensors re-read as a pool of 64-row pages, scattered by a
    # seeded permutation of the page numbers (every (b) owns cap/64 pages; the pool holds all heads of a page)
    ps = 64
    if cap % ps == 0 and hasattr(L, "loma_decode_attn_paged"):
        mp = cap // ps
        g_cpu = torch.Generator().manual_seed(3120)
        table = torch.randperm(B * mp, generator=g_cpu).to(torch.int32).view(B, mp).to(dev)
        kpool = kc.view(B, H, mp, ps, D).permute(0, 2, 1, 3, 4).reshape(B * mp, H, ps, D).contiguous()
        vpool = vc.view(B, H, mp, ps, D).permute(0, 2, 1, 3, 4).reshape(B * mp, H, ps, D).contiguous()
        ms = timed(lambda: L.loma_decode_attn_paged(q1, k1, v1, kpool, vpool, table, o1, None, lens, max_len, ws, 0, 0.0, stream))
        res["decode_paged_B64_16k"] = {"config": dict(B=B, H=H, D=D, page_size=ps, pages=B * mp), "ms": ms,
                                       "gbs": nbytes / (ms * 1e-3) / 1e9,
                                       "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        del kpool, vpool
    # the generator's loop over layers: 8 layers' caches of the B32 / 8192 shape decoded in one call, per layer
    del kc, vc
    torch.cuda.empty_cache()
    nl, Bl, memL, cl, tl = 8, 32, 8192, 4, 16
    capL = memL + cl * tl + tl
    kcs = [synthetic.big_normal_(torch.empty(Bl, H, capL, D, dtype=bf, device=dev), 3200 + i, std) for i in range(nl)]
    vcs = [synthetic.big_normal_(torch.empty(Bl, H, capL, D, dtype=bf, device=dev), 3300 + i, std) for i in range(nl)]
    qs, kns, vns = ([synthetic.big_normal_(torch.empty(Bl, H, 1, D, dtype=bf, device=dev), 3400 + 10 * j + i, std) for i in range(nl)]
                    for j in range(3))
    outs = [torch.empty_like(x) for x in qs]
    wsl = torch.empty(max(16, L.loma_decode_workspace_bytes(Bl, H, D, capL)), dtype=torch.uint8, device=dev)
    lenL = memL + 32
    ms_layers = timed(lambda: L.loma_decode_attn_layers(qs, kns, vns, kcs, vcs, outs, None, lenL, wsl, 0, 0.0, stream))
    ms_single = timed(lambda: L.loma_decode_attn(qs[0], kns[0], vns[0], kcs[0], vcs[0], outs[0], None, lenL, wsl, 0, 0.0, stream))
    nbl = 2.0 * (lenL + 1) * Bl * H * D * 2
    res["decode_8_layers_B32_8k"] = {"config": dict(layers=nl, B=Bl, H=H, D=D, cache_len=lenL), "ms": ms_layers,
                                     "ms_per_layer": ms_layers / nl, "ms_single_layer_call": ms_single,
                                     "gbs": nl * nbl / (ms_layers * 1e-3) / 1e9,
                                     "frac_of_measured_hbm": nl * nbl / (ms_layers * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    del kcs, vcs
    torch.cuda.empty_cache()
    kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3100, std)
    vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3101, std)
    # several new tokens over an existing cache (a prompt piece arriving mid-generation): 512 tokens over 8192 entries
    Bp, lp, kp = 32, 512, 8192
    kcp = synthetic.big_normal_(torch.empty(Bp, H, kp + lp, D, dtype=bf, device=dev), 3500, std)
    vcp = synthetic.big_normal_(torch.empty(Bp, H, kp + lp, D, dtype=bf, device=dev), 3501, std)
    qp, knp, vnp = (synthetic.big_normal_(torch.empty(Bp, H, lp, D, dtype=bf, device=dev), 3502 + i, std) for i in range(3))
    op = torch.empty_like(qp)
    ms = timed(lambda: L.loma_prefill_attn(qp, knp, vnp, kcp, vcp, op, None, kp, 0, 0.0, stream))
    fl = 4.0 * D * Bp * H * (lp * kp + lp * (lp + 1) // 2)
    nbytes = float(Bp * H) * D * 2 * (2 * (kp + lp) + 4 * lp)      # cache K, V read once; q, k_new, v_new read, o written
    res["prefill_512_over_8192_B32"] = {"config": dict(B=Bp, H=H, D=D, l=lp, cache_len=kp), "ms": ms,
                                        "useful_tflops": fl / (ms * 1e-3) / 1e12,
                                        "frac_of_measured_bf16": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                        "gbs": nbytes / (ms * 1e-3) / 1e9,
                                        "kernels": "cache_append_kernel + masked_attn_tc_kernel (prefill plan)"}
    if hasattr(L, "loma_prefill_attn_ragged"):
        # the same piece with one cache length per sequence (8192 minus up to 1023 entries)
        lens_p = torch.tensor([kp - (37 * b) % 1024 for b in range(Bp)], dtype=torch.int32, device=dev)
        ms = timed(lambda: L.loma_prefill_attn_ragged(qp, knp, vnp, kcp, vcp, op, None, lens_p, kp, 0, 0.0, stream))
        fl = 4.0 * D * H * float(sum(lp * int(n) + lp * (lp + 1) // 2 for n in lens_p.tolist()))
        res["prefill_ragged_512_over_8192_B32"] = {"config": dict(B=Bp, H=H, D=D, l=lp, cache_lens="8192 - (37 b) mod 1024"),
                                                   "ms": ms, "useful_tflops": fl / (ms * 1e-3) / 1e12,
                                                   "frac_of_measured_bf16": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                                   "kernels": "cache_append_kernel + masked_attn_tc_kernel<128, true>"}
    if hasattr(L, "loma_prefill_attn_paged"):
        # and over a paged cache: 128-row pages scattered over the pool by a seeded permutation
        psp = 128
        mpp = (kp + lp) // psp
        g_cpu = torch.Generator().manual_seed(3520)
        table_p = torch.randperm(Bp * mpp, generator=g_cpu).to(torch.int32).view(Bp, mpp).to(dev)
        kpool = kcp.view(Bp, H, mpp, psp, D).permute(0, 2, 1, 3, 4).reshape(Bp * mpp, H, psp, D).contiguous()
        vpool = vcp.view(Bp, H, mpp, psp, D).permute(0, 2, 1, 3, 4).reshape(Bp * mpp, H, psp, D).contiguous()
        ms = timed(lambda: L.loma_prefill_attn_paged(qp, knp, vnp, kpool, vpool, table_p, op, None, lens_p, kp, 0, 0.0, stream))
        res["prefill_paged_512_over_8192_B32"] = {"config": dict(B=Bp, H=H, D=D, l=lp, page_size=psp, pages=Bp * mpp,
                                                              cache_lens="8192 - (37 b) mod 1024"),
                                                  "ms": ms, "useful_tflops": fl / (ms * 1e-3) / 1e12,
                                                  "frac_of_measured_bf16": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                                  "kernels": "cache_append_kernel + masked_attn_tc_kernel<128, true> (paged key tiles)"}
        del kpool, vpool
    del kcp, vcp, qp, knp, vnp, op
    torch.cuda.empty_cache()
    for name, flags in (("compress_B64_16k", 0), ("compress_B64_16k_prior_mem", 1)):
        def run_decode_then_compress():
            L.loma_compress_step(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws, flags, 0.0, stream)
        ms = timed(run_decode_then_compress)
        rows = (2 * tc if flags == 0 else 2 * (mem_len + tc)) + 6 * t
        nbytes = float(B * H) * D * 2 * rows
        res[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9,
                     "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "note": "back-to-back calls; the 0.19 GB of the default variant can stay in L2" if flags == 0 else ""}
    return res


def large_workloads(L, synthetic, torch, dev, peaks, steps, warmup, clocks_mhz):
    """The two largest single-GPU workloads, each as a step of its own, `steps` timed repetitions after
    `warmup`: the 69632-token training-layout forward and one generation cycle at the higher ratio
    (128 decodes with the tail growing 0..127, then one compress).  CUDA events on the launching stream."""
    bf = torch.bfloat16
    stream = torch.cuda.current_stream()
    D = 128
    std = 1.0 / math.sqrt(D)
    ghz = (clocks_mhz or 0.0) / 1e3
    out = {}

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # ---- forward on the long layout
    B, H, n, c, t = 1, 32, 128, 8, 32
    S = n * (2 * c * t + t)
    q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 3000 + i, std) for i in range(3))
    o = torch.empty_like(q)
    for _ in range(warmup):
        L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t, 0, 0, 0.0, stream)
    torch.cuda.synchronize()
    marks = []
    for _ in range(steps):
        _device_pause(torch, 300_000)
        a, b = ev(), ev()
        a.record(stream)
        L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t, 0, 0, 0.0, stream)
        b.record(stream)
        marks.append((a, b))
    torch.cuda.synchronize()
    ts = [a.elapsed_time(b) for a, b in marks]
    ms = sum(ts) / len(ts)
    flops = 4.0 * D * allowed_pairs(n, c, t) * B * H
    nbytes = 4.0 * q.numel() * 2
    tf = flops / (ms * 1e-3) / 1e12
    out["masked_fwd_69632"] = {
        "config": dict(B=B, H=H, D=D, n=n, c=c, t=t, S=S), "steps": steps, "ms": ms, "ms_min": min(ts),
        "ms_x_sm_ghz": ms * ghz if ghz else None, "useful_tflops": tf, "useful_flops": flops, "compulsory_bytes": nbytes,
        "roofline": {"kernel": "masked_attn_tc_kernel<128, false>", "bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst bf16)",
                     "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                     # dram bytes of one launch on the 8-head case of this layout (ncu), times 4 for 32 heads
                     "traffic": FWD_LONG_TRAFFIC_8_HEADS * (H / 8.0) if FWD_LONG_TRAFFIC_8_HEADS else None,
                     "traffic_source": "ncu 8-head case x4"}}
    del q, k, v, o
    torch.cuda.empty_cache()

    # ---- generation cycle at the higher ratio
    B, H, c, t, mem_len = 64, 32, 8, 16, 16384
    tc = c * t
    cap = mem_len + tc + t
    kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3100, std)
    vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 3101, std)
    dq, dk, dv = (synthetic.big_normal_(torch.empty(tc, B, H, 1, D, dtype=bf, device=dev), 3102 + i, std) for i in range(3))
    do = torch.empty_like(dq)
    qm, km, vm = (synthetic.big_normal_(torch.empty(B, H, t, D, dtype=bf, device=dev), 3110 + i, std) for i in range(3))
    om = torch.empty_like(qm)
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cap), L.loma_compress_workspace_bytes(B, H, D, t, mem_len, 0)),
                     dtype=torch.uint8, device=dev)

    def cycle(marks=None):
        e0 = ev(); e0.record(stream)
        for j in range(tc):
            L.loma_decode_attn(dq[j], dk[j], dv[j], kc, vc, do[j], None, mem_len + j, ws, 0, 0.0, stream)
        e1 = ev(); e1.record(stream)
        L.loma_compress_step(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws, 0, 0.0, stream)
        e2 = ev(); e2.record(stream)
        if marks is not None:
            marks.append((e0, e1, e2))

    for _ in range(max(1, min(warmup, 3))):
        cycle()
    torch.cuda.synchronize()
    marks = []
    for _ in range(steps):
        cycle(marks)
    torch.cuda.synchronize()
    t_dec = sum(a.elapsed_time(b) for a, b, _ in marks) / steps
    t_cmp = sum(b.elapsed_time(c2) for _, b, c2 in marks) / steps
    dec_rows = sum(mem_len + j + 1 for j in range(tc))
    dec_bytes_call = 2.0 * dec_rows * B * H * D * 2 / tc
    dec_ms_call = t_dec / tc
    dec_gbs = dec_bytes_call / (dec_ms_call * 1e-3) / 1e9
    cmp_bytes = float(B * H) * D * 2 * (2 * tc + 6 * t)
    cmp_gbs = cmp_bytes / (t_cmp * 1e-3) / 1e9
    out["generation_B64_16k"] = {
        "config": dict(B=B, H=H, D=D, c=c, t=t, mem_len=mem_len, cap=cap, decode_steps=tc), "steps": steps,
        "cycle_ms": t_dec + t_cmp, "decode_ms_per_call": dec_ms_call, "decode_ms_x_sm_ghz": dec_ms_call * ghz if ghz else None,
        "decode_gbs": dec_gbs, "decode_bytes_per_call": dec_bytes_call, "compress_ms": t_cmp, "compress_gbs": cmp_gbs,
        "roofline": {"kernel": "decode_splitkv_kernel<128, false> (+ decode_merge_kernel<128>), per loma_decode_attn call", "bound": "hbm", "achieved": dec_gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dec_gbs / peaks["hbm_gbs"], "frac_of_8tbs": dec_gbs / 8000.0,
                     "peak_source": peaks["source"],
                     # every (b, h) streams its own rows once: the B8 / 8224-row capture scaled by rows and (b, h) pairs
                     "traffic": DECODE_TRAFFIC_B8_L8224 * (B * H / 256.0) * ((mem_len + tc / 2.0 + 0.5) / 8224.0),
                     "traffic_source": "ncu small case scaled by (b,h) pairs and rows"},
        "roofline_compress": {"kernel": "compress_one_stage_kernel<128, 8>", "bound": "hbm", "achieved": cmp_gbs, "peak": peaks["hbm_gbs"],
                              "unit": "GB/s", "frac": cmp_gbs / peaks["hbm_gbs"], "traffic": None,
                              "note": "0.19 GB in one launch right after the decodes of the cycle"}}
    return out


# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from ncu captures of the --profile-case launches
COMPRESS_TRAFFIC_B32 = 46.28e6         # compress_one_stage_kernel<128, 4>, B32 H32, c4 t16 (58.7e6 algorithmic, 46.1e6 of them reads)
DECODE_TRAFFIC_B8_L8224 = 1.0824e9     # decode_splitkv + merge, B8 H32, 8224 rows (1.0779e9 algorithmic)
FWD_SHORT_TRAFFIC_B1 = 128.1e6         # masked_attn_tc, one batch element of the 4608-token layout (151.0e6 algorithmic; part of O still in L2)
FWD_LONG_TRAFFIC_8_HEADS = 552.6e6     # masked_attn_tc, 8 heads of the 69632-token layout (570.4e6 algorithmic)


def profile_case(args):
    """One cut-down launch sequence of a single kernel, for profiler captures."""
    import torch

    from paper_2401_09486_b200 import binding as L
    from paper_2401_09486_b200 import build, synthetic

    build.build_library()
    torch.cuda.set_device(0)
    dev = "cuda:0"
    bf = torch.bfloat16
    D = 128
    std = 1.0 / math.sqrt(D)
    case = args.profile_case
    if case == "decode_paged":
        # the decode case below over a paged cache: 64-row pages scattered over the pool by a seeded permutation
        B, H, mem_len, ps = 8, 32, 8192, 64
        mp = (mem_len + 64 + ps) // ps
        g_cpu = torch.Generator().manual_seed(5)
        table = torch.randperm(B * mp, generator=g_cpu).to(torch.int32).view(B, mp).to(dev)
        kpool = synthetic.big_normal_(torch.empty(B * mp, H, ps, D, dtype=bf, device=dev), 1, std)
        vpool = synthetic.big_normal_(torch.empty(B * mp, H, ps, D, dtype=bf, device=dev), 2, std)
        q, kn, vn = (x.to(dev) for x in synthetic.qkv(B, H, 1, D, 3, std, bf))
        o = torch.empty_like(q)
        ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, mem_len + 64)), dtype=torch.uint8, device=dev)
        for r in range(args.reps):
            lens = torch.full((B,), mem_len + 31 + r, dtype=torch.int32, device=dev)
            L.loma_decode_attn_paged(q, kn, vn, kpool, vpool, table, o, None, lens, mem_len + 63, ws)
    elif case in ("decode", "compress", "compress_prior", "compress_b32"):
        B, H, c, t, mem_len = 8, 32, 4, 16, 8192          # 1/4 of the generation workload's batch: 1.08 GB of cache
        if case == "compress_b32":
            B = 32                                         # the generation workload's own batch (1024 CTAs: two waves), 4.3 GB
        tc = c * t
        cap = mem_len + tc + t
        kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 1, std)
        vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=bf, device=dev), 2, std)
        flags = L.LOMA_FLAG_MEM_SEES_PRIOR_MEM if case == "compress_prior" else 0
        ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cap),
                             L.loma_compress_workspace_bytes(B, H, D, t, mem_len, flags)), dtype=torch.uint8, device=dev)
        if case == "decode":
            q, kn, vn = (x.to(dev) for x in synthetic.qkv(B, H, 1, D, 3, std, bf))
            o = torch.empty_like(q)
            for r in range(args.reps):
                L.loma_decode_attn(q, kn, vn, kc, vc, o, None, mem_len + 31 + r, ws)
        else:
            qm, km, vm = (x.to(dev) for x in synthetic.qkv(B, H, t, D, 4, std, bf))
            om = torch.empty_like(qm)
            for r in range(args.reps):
                L.loma_compress_step(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws, flags)
    elif case in ("prefill", "prefill_ragged"):
        # a quarter of the context workload's batch: 512 new tokens over 8192 cached entries, B8 H32 (1.1 GB of cache)
        B, H, l, k_len = 8, 32, 512, 8192
        kc = synthetic.big_normal_(torch.empty(B, H, k_len + l, D, dtype=bf, device=dev), 1, std)
        vc = synthetic.big_normal_(torch.empty(B, H, k_len + l, D, dtype=bf, device=dev), 2, std)
        q, kn, vn = (synthetic.big_normal_(torch.empty(B, H, l, D, dtype=bf, device=dev), 3 + i, std) for i in range(3))
        o = torch.empty_like(q)
        lens = torch.tensor([k_len - (37 * b) % 1024 for b in range(B)], dtype=torch.int32, device=dev)
        for r in range(args.reps):
            if case == "prefill":
                L.loma_prefill_attn(q, kn, vn, kc, vc, o, None, k_len)
            else:
                L.loma_prefill_attn_ragged(q, kn, vn, kc, vc, o, None, lens, k_len)
    else:
        if case in ("masked", "bwd"):
            B, H, n, c, t = 1, 32, 32, 4, 16               # one batch element of the 4608-token layout: 151 MB per tensor
        else:
            B, H, n, c, t = 1, 8, 128, 8, 32               # 8 heads of the 69632-token layout: 143 MB per tensor
        S = n * (2 * c * t + t)
        q, k, v = (synthetic.big_normal_(torch.empty(B, H, S, D, dtype=bf, device=dev), 10 + i, std) for i in range(3))
        o = torch.empty_like(q)
        if case.startswith("bwd"):
            lse = torch.empty((B, H, S), dtype=torch.float32, device=dev)
            L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t)
            d_o = synthetic.big_normal_(torch.empty_like(q), 20, std)
            dq, dk, dv = (torch.empty_like(q) for _ in range(3))
            ws = torch.empty(L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n, c, t), dtype=torch.uint8, device=dev)
            for r in range(args.reps):
                L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n, c, t, 0, 0, ws)
        else:
            for r in range(args.reps):
                L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t)
    torch.cuda.synchronize()
    assert L.loma_device_status() == 0
    print("ok", case)


# ------------------------------------------------------------------ oracle timing

def _oracle_sample(n_heads_fwd: int, n_heads_dec: int, seed: int = 0):
    """Times the oracle, as it stands, on a bounded sample of the bench workload:
    the masked forward for n_heads_fwd (b,h) pairs of the 4608-token layout and
    one decode step (tail 32) for n_heads_dec (b,h) pairs of the generation cache."""
    import numpy as np
    import torch

    import oracle
    from paper_2401_09486_b200 import synthetic

    f, g = FWD, GEN
    tc_f = f["c"] * f["t"]
    S = f["n"] * (2 * tc_f + f["t"])
    std = 1.0 / math.sqrt(f["D"])
    q, k, v = (x.to(torch.float64).numpy() for x in synthetic.qkv(1, n_heads_fwd, S, f["D"], seed, std, torch.bfloat16))
    t0 = time.perf_counter()
    oracle.masked_attn_fwd(q, k, v, f["n"], f["c"], f["t"])
    t_fwd = time.perf_counter() - t0
    cache_len = g["mem_len"] + 32
    kc = synthetic.normal_tensor((1, n_heads_dec, cache_len + 1, g["D"]), seed + 1, std, torch.bfloat16).to(torch.float64).numpy()
    vc = synthetic.normal_tensor((1, n_heads_dec, cache_len + 1, g["D"]), seed + 2, std, torch.bfloat16).to(torch.float64).numpy()
    q1, k1, v1 = (x.to(torch.float64).numpy() for x in synthetic.qkv(1, n_heads_dec, 1, g["D"], seed + 3, std, torch.bfloat16))
    t0 = time.perf_counter()
    oracle.decode_attn(q1, k1, v1, kc, vc, cache_len)
    t_dec = time.perf_counter() - t0
    pairs = allowed_pairs(f["n"], f["c"], f["t"])
    tflops = 4.0 * f["D"] * pairs * n_heads_fwd / t_fwd / 1e12
    dec_gbs = 2.0 * (cache_len + 1) * g["D"] * 2 * n_heads_dec / t_dec / 1e9
    return tflops, dec_gbs, t_fwd, t_dec


def _threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline():
    tflops, dec_gbs, t_fwd, t_dec = _oracle_sample(n_heads_fwd=16, n_heads_dec=64)
    return {"value": tflops, "unit": "TFLOP/s", "cores": _threads(), "kind": "oracle",
            "sample": ("masked fwd: 16 of 128 (b,h) pairs of the 4608-token layout, dense fp64 NumPy, "
                       f"{t_fwd:.2f} s; decode: 64 of 1024 (b,h) pairs, one step at cache length 8224, {t_dec:.2f} s"),
            "decode_gbs": dec_gbs, "host_cores": os.cpu_count()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, decs, times = [], [], []
    for i in range(max(args.warmup, 1) + args.steps):
        t0 = time.perf_counter()
        tf, dg, _, _ = _oracle_sample(n_heads_fwd=1, n_heads_dec=4, seed=i)
        if i >= max(args.warmup, 1):
            vals.append(tf); decs.append(dg); times.append(time.perf_counter() - t0)
    val = statistics.mean(vals)
    cores = _threads()
    sample = "per step: masked fwd of 1 of 128 (b,h) pairs (4608 tokens) + one decode step for 4 of 1024 (b,h) pairs"
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": 1e3 * statistics.mean(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "CPU oracle on a bounded sample of the same workload", "masked_fwd": FWD,
                   "generation": GEN},
        "decode_attn": {"value": statistics.mean(decs), "unit": "GB/s"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-extras", action="store_true", help="skip the large and the context workloads timed at N=1")
    ap.add_argument("--profile-case", choices=["decode", "decode_paged", "compress", "compress_prior", "compress_b32", "masked", "masked_long", "bwd", "bwd_long", "prefill",
                                                     "prefill_ragged"],
                    help="run one cut-down kernel launch sequence (for profiler captures) and exit")
    ap.add_argument("--reps", type=int, default=3, help="launches of --profile-case")
    args = ap.parse_args()
    if args.profile_case:
        profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

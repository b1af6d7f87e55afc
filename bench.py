#!/usr/bin/env python
"""Benchmark of the fused outlier-aware W4A16 decode matmul on B200.

One step = one pass of the hot path over the LLaMA-3-8B-shaped decode layer set (qkv, o_proj,
gate_up, down) at M in {1, 8, 16}: twelve calls of fq_fused_w4a16_outlier_gemm on seeded synthetic
layers (INT4 g128, 1 % mixed-layout BF16 outliers).  The metric is effective HBM GB/s: the
algorithmic bytes of those calls (packed INT4 + scale/zero + Tile-COO by the paper's storage
formula with the true nnz + X + Y) divided by device time.  Weights are resident in HBM; every
call reads a different packed copy of its layer so that no call finds its weights in L2.

`--impl reference` times the CPU oracle instead (a deliberately plain program; a reported
baseline, not a target).
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
sys.path.insert(0, ROOT)

MS = (1, 8, 16)
GROUP = 128
DENSITY = 0.01
CONFIG_ID = 2                      # the LLaMA-3-8B layer set
REPEATS = 5                        # repetitions of the timed region (K steps each); the median is the value
L2_COVER_BYTES = 400 << 20         # rotating copies per layer cover at least this (L2 is 126 MB)
METRIC = "effective_hbm_gbs_fused_w4a16_outlier_gemm_m1_8_16"
# dram__bytes_read + dram__bytes_write of a fused launch over its algorithmic bytes, per layer, from the ncu captures
# summarised in profiles/fq_kernels_llama3_8b_decode_set.md (the padding of the column-slotted packets; the ratio
# does not depend on M).  Not measured by a bench run: `roofline.traffic` applies them to the step's launches.
NCU_TRAFFIC_RATIO = {"gate_up": 1.072, "down": 1.053, "qkv": 1.049, "o_proj": 1.048}


def algorithmic_bytes(K, N, g, nnz, n_tile, n_bucket, M):
    return K * N // 2 + 2 * (K // g) * N * 2 + (n_tile + 1) * 4 + n_bucket * 4 + 4 * nnz + 2 * M * K + 2 * M * N


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Step time of the whole job: the slowest rank's (replicas run side by side, one per GPU)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(step_bytes: int, world: int, ms_per_step: float) -> float:
    """Aggregate effective bandwidth: every rank moves `step_bytes` per step (weak scaling)."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tensor_peak():
    """Sustained dense BF16 throughput in TFLOP/s (the denominator of `tensor_frac` for rows with M >= 64)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p)).get("bf16_tflops_sustained", 1400.0)), "measured"
    return 1400.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile(prefix="fq_clocks_", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
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
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def build_workload(layers, log, config_id=CONFIG_ID, table=None, max_m=None):
    """Generate, pack and encode every layer on the host.  Returns a list of dicts (with the seconds the packer
    and the encoder took per matrix: the paper bounds its preprocessing at 100 s per matrix, Section 5.3)."""
    from paper_2608_15531_b200 import binding as fq
    from paper_2608_15531_b200 import synth
    table = synth.LLAMA3_8B if table is None else table
    out = []
    for (name, K, N) in layers:
        idx = table.index((name, K, N))
        t0 = time.time()
        lay = synth.layer(synth.tensor_seed(config_id, idx), K, N, density=DENSITY, layout="mixed")
        L = fq.fq_get_layout(K, N, GROUP)
        t1 = time.time()
        wq, scale, zero = fq.fq_pack_int4(L, lay.W, lay.mask)
        t2 = time.time()
        indptr, info, packed = fq.fq_encode_tilecoo(L, lay.coo_k, lay.coo_n, lay.coo_v)
        t3 = time.time()
        n_tile = (K // 128) * (N // L.BN)
        out.append(dict(name=name, K=K, N=N, L=L, lay=lay, wq=wq, scale=scale, zero=zero, indptr=indptr, info=info,
                        packed=packed, n_tile=n_tile, n_bucket=n_tile * L.buckets_per_tile, nnz=lay.nnz,
                        pack_s=round(t2 - t1, 3), encode_s=round(t3 - t2, 3),
                        X=synth.activations(synth.tensor_seed(config_id, idx), max_m or max(MS), K)))
        log(f"packed {name} {K}x{N}: nnz={lay.nnz} packets={packed.shape[0]} max_tile={L.max_tile_packets} "
            f"generate {t1 - t0:.1f}s pack {t2 - t1:.1f}s encode {t3 - t2:.1f}s")
    return out


def build_reference_workload(layers, log):
    """The reference arm's inputs: the generator and the oracle's own quantiser only (the library is not loaded)."""
    from paper_2608_15531_b200 import synth
    out = []
    for (name, K, N) in layers:
        idx = synth.LLAMA3_8B.index((name, K, N))
        lay = synth.layer(synth.tensor_seed(CONFIG_ID, idx), K, N, density=DENSITY, layout="mixed")
        bn = 256 if N % 256 == 0 else 128
        n_tile = (K // 128) * (N // bn)
        out.append(dict(name=name, K=K, N=N, lay=lay, n_tile=n_tile, n_bucket=n_tile * (bn // 4), nnz=lay.nnz,
                        X=synth.activations(synth.tensor_seed(CONFIG_ID, idx), 16, K)))
        log(f"generated {name} {K}x{N}: nnz={lay.nnz}")
    return out


def run_ours(args):
    global MS
    import torch
    import torch.distributed as dist
    from paper_2608_15531_b200 import binding as fq
    from paper_2608_15531_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the fused path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fq.lib()                                     # fail loudly if the library is missing

    def log(msg):
        if rank == 0 and args.verbose:
            print(f"[bench] {msg}", file=sys.stderr, flush=True)

    layers = synth.LLAMA3_8B
    ms = MS
    if args.only:                                # profiling aid: one layer, one M (e.g. gate_up:16)
        lname, lm = args.only.split(":")
        layers = [l for l in synth.LLAMA3_8B if l[0] == lname]
        ms = (int(lm),)
    MS = ms
    work = build_workload(layers, log)
    dev = torch.device("cuda", local)

    def up(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint16:
            a = a.view(np.int16)
        elif a.dtype == np.uint32:
            a = a.view(np.int32)
        return torch.from_numpy(a).to(dev)

    ws_bytes = max(fq.fq_workspace_bytes(w["L"], max(MS)) for w in work)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    calls = []                                   # (layer dict, M, bytes)
    for w in work:
        per_copy = w["wq"].nbytes + w["scale"].nbytes + w["zero"].nbytes + w["indptr"].nbytes + w["info"].nbytes + \
            w["packed"].nbytes
        ncopy = max(2, -(-L2_COVER_BYTES // per_copy))
        w["per_copy"] = per_copy
        base = dict(wq=up(w["wq"]), scale=up(w["scale"]), zero=up(w["zero"]), indptr=up(w["indptr"]),
                    info=up(w["info"]), packed=up(w["packed"]))
        w["copies"] = [base] + [{k: v.clone() for k, v in base.items()} for _ in range(ncopy - 1)]
        w["Xd"] = {M: up(w["X"][:M]) for M in MS}
        w["Yd"] = {M: torch.empty((M, w["N"]), dtype=torch.int16, device=dev) for M in MS}
        w["turn"] = 0
        for M in MS:
            calls.append((w, M, algorithmic_bytes(w["K"], w["N"], GROUP, w["nnz"], w["n_tile"], w["n_bucket"], M)))
    step_bytes = sum(c[2] for c in calls)
    stream = torch.cuda.current_stream()

    # Argument tuples are marshalled once: the timed loop only calls into the C ABI.
    import ctypes
    clib = fq.lib()
    vp = lambda t: ctypes.c_void_p(t.data_ptr())
    sp = ctypes.c_void_p(stream.cuda_stream)
    for w in work:
        w["args"] = {M: [(ctypes.byref(w["L"]), vp(w["Xd"][M]), ctypes.c_uint32(M), vp(c["wq"]), vp(c["scale"]),
                          vp(c["zero"]), vp(c["indptr"]), vp(c["info"]), vp(c["packed"]), vp(w["Yd"][M]), vp(ws),
                          ctypes.c_size_t(ws_bytes), sp) for c in w["copies"]] for M in MS}

    def one_call(w, M):
        a = w["args"][M]
        rc = clib.fq_fused_w4a16_outlier_gemm(*a[w["turn"] % len(a)])
        w["turn"] += 1
        if rc != 0:
            raise fq.FqError(rc, fq.fq_last_error())

    def step():
        for w, M, _ in calls:
            one_call(w, M)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    fq.fq_check_status(ws)
    sampler = ClockSampler(local)
    sync_all()
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps_ms, host_issue_ms = [], []
    for _ in range(REPEATS):                     # the timed region, REPEATS times: the median is reported
        sync_all()
        e0.record(stream)
        h0 = time.perf_counter()
        for _ in range(args.steps):
            step()
        host_issue_ms.append((time.perf_counter() - h0) * 1e3)
        e1.record(stream)
        sync_all()
        reps_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
    clocks = sampler.stop() if rank == 0 else {}
    ms = float(np.median(reps_ms))
    fq.fq_check_status(ws)
    ms_per_step = ms / args.steps
    value = whole_job_gbs(step_bytes, world, ms_per_step)
    # the step's bytes without the two Tile-COO metadata arrays, and as stored (padding included)
    fmt_free_bytes = sum(b - (w["n_tile"] + 1) * 4 - w["n_bucket"] * 4 for w, M, b in calls)
    moved_bytes = sum(w["per_copy"] + 2 * M * w["K"] + 2 * M * w["N"] for w, M, b in calls)
    # read-only streaming probe: a sum over 1 GiB (reads alone usually beat a copy)
    read_probe = None
    if rank == 0:
        probe = torch.ones(1 << 28, dtype=torch.float32, device=dev)
        for _ in range(3):
            probe.sum()
        torch.cuda.synchronize()
        pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pa.record(stream)
        for _ in range(10):
            probe.sum()
        pb.record(stream)
        torch.cuda.synchronize()
        read_probe = round(10 * probe.numel() * 4 / (pa.elapsed_time(pb) * 1e-3) / 1e9, 1)
        del probe
        torch.cuda.empty_cache()

    # ---- end to end: host X in, host Y out, through the C ABI, every call
    xh = {(w["name"], M): torch.from_numpy(np.ascontiguousarray(w["X"][:M]).view(np.int16)).pin_memory()
          for w, M, _ in calls}
    yh = {(w["name"], M): torch.empty((M, w["N"]), dtype=torch.int16).pin_memory() for w, M, _ in calls}
    xd = {k: torch.empty_like(v, device=dev) for k, v in xh.items()}

    def e2e_step():
        # twelve asynchronous calls (copy of X in, kernel, copy of Y out, each with staging buffers of its
        # own) and one wait for the step's results
        for w, M, _ in calls:
            c = w["copies"][w["turn"] % len(w["copies"])]
            w["turn"] += 1
            key = (w["name"], M)
            fq.fq_fused_host_io_async(w["L"], xh[key], M, xd[key], c["wq"], c["scale"], c["zero"], c["indptr"],
                                      c["info"], c["packed"], w["Yd"][M], yh[key], ws, stream)
        stream.synchronize()

    for _ in range(3):
        e2e_step()
    sync_all()
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e1.record(stream)
    sync_all()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    e2e_value = whole_job_gbs(step_bytes, world, e2e_ms / args.steps)
    h2d = sum(2 * M * w["K"] for w, M, _ in calls)
    d2h = sum(2 * M * w["N"] for w, M, _ in calls)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = peaks()

    # ---- per call: fused, unfused pair, cuBLAS BF16 on pre-dequantised weights (context, N = 1 view)
    def time_loop(fn, reps):
        """Device time per call of `reps` calls issued back to back.  The calls are queued behind a short spin
        kernel, so that the stream never waits for the host (Python issues a call in about as long as the
        shortest of these kernels runs)."""
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(reps * 12e-6 * 1.9e9))   # about 12 us of spinning per queued call
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3          # microseconds

    per_call = []
    reps = max(10, min(100, args.steps * 2))
    for w, M, nbytes in calls:
        def fused():
            one_call(w, M)

        def unfused():
            c = w["copies"][w["turn"] % len(w["copies"])]
            w["turn"] += 1
            fq.fq_unfused_gemm(w["L"], w["Xd"][M], M, c["wq"], c["scale"], c["zero"], w["Yd"][M], ws, stream)
            fq.fq_unfused_spmm(w["L"], w["Xd"][M], M, c["indptr"], c["info"], c["packed"], w["Yd"][M], stream)

        def dense_only():
            c = w["copies"][w["turn"] % len(w["copies"])]
            w["turn"] += 1
            fq.fq_unfused_gemm(w["L"], w["Xd"][M], M, c["wq"], c["scale"], c["zero"], w["Yd"][M], ws, stream)

        def spmm_only():
            c = w["copies"][w["turn"] % len(w["copies"])]
            w["turn"] += 1
            fq.fq_unfused_spmm(w["L"], w["Xd"][M], M, c["indptr"], c["info"], c["packed"], w["Ys"][M], stream)

        w.setdefault("Ys", {})[M] = torch.zeros((M, w["N"]), dtype=torch.int16, device=dev)
        us_f = time_loop(fused, reps)
        us_u = time_loop(unfused, reps)
        us_d = time_loop(dense_only, reps)
        us_s = time_loop(spmm_only, reps)
        sp_bytes = w["indptr"].nbytes + w["info"].nbytes + 4 * w["nnz"] + 2 * M * w["K"] + 4 * M * w["N"]
        per_call.append(dict(layer=w["name"], K=w["K"], N=w["N"], M=M, bytes=nbytes, fused_us=round(us_f, 3),
                             fused_gbs=round(nbytes / us_f / 1e3, 1), frac_of_peak=round(nbytes / us_f / 1e3 / peak, 4),
                             unfused_us=round(us_u, 3), unfused_gemm_us=round(us_d, 3), unfused_spmm_us=round(us_s, 3),
                             spmm_bytes=sp_bytes, spmm_roofline_us=round(sp_bytes / peak / 1e3, 3)))
    if args.cublas:
        for w in work:
            # BF16 GEMM on dequant(W_Q) + W_O, materialised with torch on the device (a baseline, not the path)
            q = torch.from_numpy(fq.fq_unpack_int4(w["L"], w["wq"])).to(dev).float()
            s = up(w["scale"]).view(torch.bfloat16).float().repeat_interleave(GROUP, 0)
            z = up(w["zero"]).view(torch.bfloat16).float().repeat_interleave(GROUP, 0)
            Wd = (s * (q - z))
            Wd[torch.from_numpy(w["lay"].coo_k.astype(np.int64)).to(dev), torch.from_numpy(w["lay"].coo_n.astype(np.int64)).to(dev)] = \
                up(w["lay"].coo_v).view(torch.bfloat16).float()
            Wb = Wd.to(torch.bfloat16)
            del q, s, z, Wd
            ncopy = max(2, -(-L2_COVER_BYTES // (Wb.numel() * 2)))
            Wc = [Wb] + [Wb.clone() for _ in range(ncopy - 1)]
            for M in MS:
                xb = w["Xd"][M].view(torch.bfloat16)
                turn = [0]

                def gemm():
                    turn[0] += 1
                    torch.matmul(xb, Wc[turn[0] % len(Wc)])

                us = time_loop(gemm, reps)
                for pc in per_call:
                    if pc["layer"] == w["name"] and pc["M"] == M:
                        pc["cublas_bf16_us"] = round(us, 3)
            del Wc, Wb
            torch.cuda.empty_cache()

    cpu = cpu_baseline(work, budget_s=args.cpu_seconds) if args.cpu_seconds > 0 else None
    others = None
    if args.other_sets and world == 1 and not args.only:
        for w in work:                               # the headline's device copies are no longer needed
            for k in ("copies", "Xd", "Yd", "Ys", "args"):
                w.pop(k, None)
        torch.cuda.empty_cache()
        others = other_sets(dev, stream, peak, log, time_loop, up)

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5),
        "ms_per_step_repeats": {"n": REPEATS, "median": round(ms_per_step, 5), "min": round(min(reps_ms) / args.steps, 5),
                                "max": round(max(reps_ms) / args.steps, 5)},
        "host_issue_ms_per_step": round(float(np.median(host_issue_ms)) / args.steps, 5),
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "configs[1]: LLaMA3-8B decode layer set qkv/o_proj/gate_up/down x M in {1,8,16}, "
                               "INT4 g128, 1% mixed-layout BF16 outliers; one step = 12 fused calls",
                   "l2": "inputs larger than L2: each call reads a different packed copy, copies per layer cover >= 400 MB",
                   "replicas": "replicas only: each rank runs the same workload on its own GPU, no collective on the data path"},
        "clocks": clocks,
        "e2e": {"value": round(e2e_value, 2), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms / args.steps, 5)},
        "gpu_launches": args.steps * len(calls),
        "roofline": {"bound": "hbm", "achieved": round(value / world, 2), "peak": peak, "unit": "GB/s",
                     "frac": round(value / world / peak, 4),
                     "traffic": int(sum(NCU_TRAFFIC_RATIO.get(w["name"], 1.06) * b for w, M, b in calls) / len(calls)),
                     "traffic_kind": "algorithmic bytes x the DRAM/algorithmic ratio of each layer's committed ncu capture "
                                     f"{NCU_TRAFFIC_RATIO}, average launch of the step; not measured by this run",
                     "peak_kind": f"of {peak_kind}",
                     "bytes_per_launch": step_bytes // len(calls), "us_per_launch": round(ms_per_step * 1e3 / len(calls), 3),
                     # the same time against other byte counts and other denominators
                     "frac_of_spec_8000": round(value / world / 8000.0, 4),
                     "format_independent_gbs": round(whole_job_gbs(fmt_free_bytes, 1, ms_per_step), 2),
                     "moved_gbs": round(whole_job_gbs(moved_bytes, 1, ms_per_step), 2),
                     "read_probe_gbs": read_probe, "frac_of_read_probe": round(value / world / read_probe, 4) if read_probe else None},
        "cpu_baseline": cpu,
        "preprocess": [dict(layer=w["name"], K=w["K"], N=w["N"], pack_s=w["pack_s"], encode_s=w["encode_s"]) for w in work],
        "us_per_call": per_call,
        "us_per_call_other_sets": others,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def other_sets(dev, stream, peak, log, time_loop, up):
    """Per-call times of the layer sets the headline does not cover: configs[0] (one 4096 x 4096 layer, M = 1) and
    configs[3] (the LLaMA3-70B shapes, M in {1, 4, 16, 32}); same generator, fused call and cuBLAS BF16 per point."""
    import torch
    from paper_2608_15531_b200 import binding as fq
    from paper_2608_15531_b200 import synth
    rows = []
    sets = [("configs[0]", 1, [("single", 4096, 4096)], (1,)),
            ("configs[3]", 4, synth.LLAMA3_70B, (1, 4, 16, 32))]
    for set_name, cfg, table, Ms in sets:
        for idx, (name, K, N) in enumerate(table):
            t0 = time.time()
            lay = synth.layer(synth.tensor_seed(cfg, idx), K, N, density=DENSITY, layout="mixed")
            L = fq.fq_get_layout(K, N, GROUP)
            t1 = time.time()
            wq, scale, zero = fq.fq_pack_int4(L, lay.W, lay.mask)
            t2 = time.time()
            indptr, info, packed = fq.fq_encode_tilecoo(L, lay.coo_k, lay.coo_n, lay.coo_v)
            t3 = time.time()
            log(f"{set_name} {name} {K}x{N}: generate {t1 - t0:.1f}s pack {t2 - t1:.1f}s encode {t3 - t2:.1f}s")
            base = dict(wq=up(wq), scale=up(scale), zero=up(zero), indptr=up(indptr), info=up(info), packed=up(packed))
            per_copy = sum(v.numel() * v.element_size() for v in base.values())
            copies = [base] + [{k: v.clone() for k, v in base.items()}
                               for _ in range(max(2, -(-L2_COVER_BYTES // per_copy)) - 1)]
            Wb = [torch.randn((K, N), dtype=torch.bfloat16, device=dev) for _ in range(2)]   # cuBLAS: time only
            n_tile = (K // 128) * (N // L.BN)
            ws = torch.zeros(fq.fq_workspace_bytes(L, max(Ms)), dtype=torch.uint8, device=dev)
            Xall = synth.activations(lay.seed, max(Ms), K)
            for M in Ms:
                X = up(Xall[:M])
                Y = torch.empty((M, N), dtype=torch.int16, device=dev)
                turn = [0]

                def fused():
                    c = copies[turn[0] % len(copies)]
                    turn[0] += 1
                    fq.fq_fused_w4a16_outlier_gemm(L, X, M, c["wq"], c["scale"], c["zero"], c["indptr"], c["info"],
                                                   c["packed"], Y, ws, stream)

                def mm():
                    turn[0] += 1
                    torch.matmul(X.view(torch.bfloat16), Wb[turn[0] & 1])

                nbytes = algorithmic_bytes(K, N, GROUP, lay.nnz, n_tile, n_tile * L.buckets_per_tile, M)
                us_f = time_loop(fused, 20)
                us_c = time_loop(mm, 10)
                fq.fq_check_status(ws)
                rows.append(dict(set=set_name, layer=name, K=K, N=N, M=M, bytes=nbytes, fused_us=round(us_f, 3),
                                 fused_gbs=round(nbytes / us_f / 1e3, 1), frac_of_peak=round(nbytes / us_f / 1e3 / peak, 4),
                                 cublas_bf16_us=round(us_c, 3), pack_s=round(t2 - t1, 3), encode_s=round(t3 - t2, 3)))
            del copies, base, Wb, lay, wq, packed
            torch.cuda.empty_cache()
    return rows


def cpu_baseline(work, budget_s: float):
    """The oracle as it stands on the host cores, on a bounded sample: every layer of the step at
    M = 16, restricted to its first `f * N` output columns, f chosen from a short probe so that the
    whole sample takes about `budget_s` seconds."""
    import oracle
    probe = work[min(1, len(work) - 1)]            # o_proj
    cols = 128
    lay = probe["lay"]
    q, s, z = oracle.quantize(np.ascontiguousarray(lay.W[:, :cols]), np.ascontiguousarray(lay.mask[:, :cols]), GROUP)
    sel = lay.coo_n < cols
    t0 = time.time()
    oracle.fused_matmul(probe["X"][:16], q, s, z, GROUP, lay.coo_k[sel], lay.coo_n[sel], lay.coo_v[sel])
    rate = 16 * probe["K"] * cols / max(time.time() - t0, 1e-6)        # multiply-adds per second
    total_mac = sum(16 * w["K"] * w["N"] for w in work)
    f = min(1.0, budget_s * rate / total_mac)
    t_total, bytes_total = 0.0, 0
    for w in work:
        lay = w["lay"]
        ncols = max(64, int(f * w["N"]) // 64 * 64)
        q, s, z = oracle.quantize(np.ascontiguousarray(lay.W[:, :ncols]), np.ascontiguousarray(lay.mask[:, :ncols]), GROUP)
        sel = lay.coo_n < ncols
        t0 = time.time()
        oracle.fused_matmul(w["X"][:16], q, s, z, GROUP, lay.coo_k[sel], lay.coo_n[sel], lay.coo_v[sel])
        t_total += time.time() - t0
        frac = ncols / w["N"]
        bytes_total += int(frac * algorithmic_bytes(w["K"], w["N"], GROUP, w["nnz"], w["n_tile"], w["n_bucket"], 16))
    return {"value": round(bytes_total / t_total / 1e9, 4), "unit": "GB/s", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(t_total, 2),
            "sample": f"all four layers at M=16, first {f:.3f} of each layer's output columns (fp64 oracle, OpenMP over columns)"}


def run_sweep(args):
    """Not the contract line: the paper's two sweeps on one GPU, one JSON object on stdout.
    `density`: M = 8, K = 4096, N = 14336, densities 0..5 % in the uniform and the clustered layout;
    `batch`:   K = 8192, N = 28672, 1 % mixed outliers, M = 1..128, groups of 64 and 128.
    Every point: fused call, unfused pair (dense kernel + SpMM), rotating weight copies larger than L2."""
    import ctypes
    import torch
    from paper_2608_15531_b200 import binding as fq
    from paper_2608_15531_b200 import synth
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the fused path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream()
    peak, peak_kind = peaks()

    def up(a):
        a = np.ascontiguousarray(a)
        a = a.view(np.int16) if a.dtype == np.uint16 else (a.view(np.int32) if a.dtype == np.uint32 else a)
        return torch.from_numpy(a).to(dev)

    def time_loop(fn, reps=30):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(reps * 12e-6 * 1.9e9))   # the calls queue up behind a spin kernel: no host-bound gaps
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3

    def point(cfg, tag, K, N, g, density, layout, Ms, slot_order=0, repurpose=False, extra=None):
        lay = synth.layer(synth.tensor_seed(cfg, tag), K, N, density=density, layout=layout)
        L = fq.fq_get_layout(K, N, g)
        L.slot_order = slot_order
        t0 = time.time()
        if repurpose:
            # Section 3.2.1's remark: the packets' padding slots take the column's worst-quantised weights
            mask2, _ = fq.fq_repurpose_pad_slots(L, lay.W, lay.mask)
            kk, nn = np.nonzero(mask2)
            u = lay.W[kk, nn].view(np.uint32).astype(np.uint64)
            lay.mask, lay.coo_k, lay.coo_n = mask2, kk.astype(np.uint32), nn.astype(np.uint32)
            lay.coo_v = ((u + 0x7fff + ((u >> 16) & 1)) >> 16).astype(np.uint16)
        t1 = time.time()
        wq, scale, zero = fq.fq_pack_int4(L, lay.W, lay.mask if lay.nnz else None)
        t2 = time.time()
        indptr, info, packed = fq.fq_encode_tilecoo(L, lay.coo_k, lay.coo_n, lay.coo_v)
        t3 = time.time()
        if extra is not None:
            extra.update(repurpose_s=round(t1 - t0, 3), pack_s=round(t2 - t1, 3), encode_s=round(t3 - t2, 3),
                         packets=int(packed.shape[0]), stored_values=int(lay.nnz))
        if packed.shape[0] == 0:
            packed = np.zeros((8, 16), dtype=np.uint8)
        base = dict(wq=up(wq), scale=up(scale), zero=up(zero), indptr=up(indptr), info=up(info), packed=up(packed))
        per_copy = sum(v.numel() * v.element_size() for v in base.values())
        copies = [base] + [{k: v.clone() for k, v in base.items()} for _ in range(max(2, -(-L2_COVER_BYTES // per_copy)) - 1)]
        n_tile = (K // 128) * (N // L.BN)
        ws = torch.zeros(fq.fq_workspace_bytes(L, max(Ms)), dtype=torch.uint8, device=dev)
        out = []
        for M in Ms:
            X = up(synth.activations(lay.seed, M, K))
            Y = torch.empty((M, N), dtype=torch.int16, device=dev)
            turn = [0]

            def fused():
                c = copies[turn[0] % len(copies)]
                turn[0] += 1
                fq.fq_fused_w4a16_outlier_gemm(L, X, M, c["wq"], c["scale"], c["zero"], c["indptr"], c["info"],
                                               c["packed"], Y, ws, stream)

            def unfused():
                c = copies[turn[0] % len(copies)]
                turn[0] += 1
                fq.fq_unfused_gemm(L, X, M, c["wq"], c["scale"], c["zero"], Y, ws, stream)
                fq.fq_unfused_spmm(L, X, M, c["indptr"], c["info"], c["packed"], Y, stream)

            nbytes = algorithmic_bytes(K, N, g, lay.nnz, n_tile, n_tile * L.buckets_per_tile, M)
            us_f, us_u = time_loop(fused), time_loop(unfused)
            fq.fq_check_status(ws)
            out.append(dict(K=K, N=N, group=g, M=M, density=density, layout=layout, nnz=int(lay.nnz), bytes=nbytes,
                            fused_us=round(us_f, 2), unfused_us=round(us_u, 2), fused_gbs=round(nbytes / us_f / 1e3, 1),
                            frac_of_peak=round(nbytes / us_f / 1e3 / peak, 4), fused_over_unfused=round(us_u / us_f, 2)))
            if M >= 64:                              # against the tensor roofline as well: 2 M K N over the sustained BF16 peak
                tp, _ = tensor_peak()
                out[-1]["tensor_frac"] = round(2.0 * M * K * N / (us_f * 1e-6) / 1e12 / tp, 4)
        del copies, base
        torch.cuda.empty_cache()
        return out

    def cublas_bf16_us(K, N, M):
        """torch.matmul on BF16 weights of the same shape (values do not matter for its time)."""
        W = [torch.randn((K, N), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        X = torch.randn((M, K), dtype=torch.bfloat16, device=dev)
        turn = [0]

        def mm():
            turn[0] += 1
            torch.matmul(X, W[turn[0] & 1])

        us = time_loop(mm, reps=10)
        del W
        torch.cuda.empty_cache()
        return us

    points = []
    if args.sweep == "paper":
        # The paper's ratio and batch sweep on its extreme operator shape, both orientations
        # (Section 5: outlier ratios 1-3 %, batch 8/16/32); uniform layout, BF16 outliers.
        for tag, (K, N) in enumerate(((14848, 75264), (75264, 14848))):
            ref = {M: round(cublas_bf16_us(K, N, M), 2) for M in (8, 16, 32)}
            for density in (0.01, 0.015, 0.02, 0.025, 0.03):
                pts = point(6, 10 * tag + int(density * 1000), K, N, GROUP, density, "uniform", (8, 16, 32))
                for pt in pts:
                    pt["cublas_bf16_us"] = ref[pt["M"]]
                    pt["cublas_over_fused"] = round(ref[pt["M"]] / pt["fused_us"], 2)
                points += pts
                print(f"[bench] {K}x{N} {density}: " + ", ".join(f"M={q['M']}: {q['fused_us']} us" for q in pts),
                      file=sys.stderr, flush=True)
    elif args.sweep == "encoder":
        # Ablation of the encoder's choices (Sec. 5.4) on the density sweep's shape at 1 % mixed outliers: order of
        # a column's outliers over its packets (bank-aware / by row), padding slots empty / holding weights.
        for slot_order, repurpose in ((0, False), (1, False), (0, True)):
            extra = {}
            pts = point(3, 10, 4096, 14336, GROUP, DENSITY, "mixed", (1, 8, 16), slot_order=slot_order,
                        repurpose=repurpose, extra=extra)
            for pt in pts:
                pt.update(slot_order="bank-aware" if slot_order == 0 else "by row", pad_slots="weights" if repurpose else "empty",
                          **extra)
            points += pts
    elif args.sweep == "density":
        for layout in ("uniform", "clustered"):
            for density in (0.0, 0.005, 0.01, 0.02, 0.05):
                if density == 0.0 and layout == "clustered":
                    continue
                points += point(3, int(density * 1000) + (layout == "clustered"), 4096, 14336, GROUP, density, layout,
                                (1, 8, 16))
    else:
        for g in (64, 128):
            points += point(5, g, 8192, 28672, g, DENSITY, "mixed", (1, 2, 4, 8, 16, 32, 64, 128))
    print(json.dumps({"sweep": args.sweep, "peak_gbs": peak, "peak_kind": f"of {peak_kind}", "data": "synthetic",
                      "points": points}))


def run_reference(args):
    """The oracle arm: rank 0 times the CPU oracle on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2608_15531_b200 import synth

    def log(msg):
        if args.verbose:
            print(f"[bench] {msg}", file=sys.stderr, flush=True)

    work = build_reference_workload(synth.LLAMA3_8B, log)
    steps = max(1, args.steps)
    per_step_budget = max(2.0, min(20.0, 120.0 / (steps + args.warmup)))
    for _ in range(args.warmup):
        cpu_baseline(work, per_step_budget)
    t0 = time.time()
    res = None
    for _ in range(steps):
        res = cpu_baseline(work, per_step_budget)
    dt = (time.time() - t0) / steps
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": args.warmup,
        "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "configs[1]: LLaMA3-8B decode layer set, bounded sample per step (see cpu_baseline.sample)"},
        "cpu_baseline": res,
        "e2e": {"value": res["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the CPU-oracle baseline leg (0 = skip)")
    ap.add_argument("--no-cublas", dest="cublas", action="store_false")
    ap.add_argument("--no-other-sets", dest="other_sets", action="store_false",
                    help="skip the per-call rows of configs[0] and configs[3] (N = 1 only; the headline is unchanged)")
    ap.add_argument("--verbose", action="store_true")
    ap.add_argument("--only", default="", help="profiling aid: restrict the step to one LAYER:M, e.g. gate_up:16")
    ap.add_argument("--sweep", default="", choices=["", "density", "batch", "paper", "encoder"],
                    help="print the density sweep, the batch transition sweep or the paper's ratio-and-batch sweep on "
                         "its largest operator shape (minutes of host time) instead of the benchmark line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

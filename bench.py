#!/usr/bin/env python
"""Benchmark of the USV sparsified-attention hot path on B200.

One "step" = one pass of the attention path of the workload over one synthetic batch:
block pooling + scores -> top-k key-block selection -> block-sparse attention forward
(and, for the merging workloads, token merge before and token unmerge after).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl usv|reference]

Prints ONE JSON line (rank 0).  `value` is dense-equivalent TFLOP/s of the whole job
(4*B*H*N^2*d per step and rank, summed over ranks, divided by the max-over-ranks step time)
with inputs resident in HBM; `e2e` is the same metric through the public API with pinned HOST
buffers (H2D of q,k,v and D2H of o inside the timed region).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import usv_inputs as ui  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0
PAPER_CONTEXT = ("paper: 83.3x DiT-denoising / 22.7x end-to-end speedup vs dense Wan2.1-1.3B "
                 "(sparsity 0.95, 3 steps vs 50) on 1x NVIDIA H20, precision unstated; "
                 "no kernel-level number is published")

ATTN_KERNEL_SOURCE = os.path.join(ROOT, "paper_2512_05754_b200", "csrc", "usv_attn_pair.cu")
ATTN_PROFILE = os.path.join(ROOT, "profiles", "attn_pair_kernel_wan480p.md")


def attn_dram_traffic(workload):
    """DRAM bytes per launch of the attention kernel (dram__bytes_read.sum + dram__bytes_write.sum)
    from the ncu summary under profiles/, which records the sha256 prefix of the kernel source it
    was captured on in a line `dram_traffic: workload=<name> bytes=<float> source_sha256=<16 hex>`.
    None once the kernel source has changed since (or for a workload without a capture)."""
    import hashlib
    import re
    try:
        text = open(ATTN_PROFILE).read()
        sha = hashlib.sha256(open(ATTN_KERNEL_SOURCE, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    for m in re.finditer(r"dram_traffic:\s*workload=(\S+)\s+bytes=(\S+)\s+source_sha256=([0-9a-f]{16})", text):
        if m.group(1) == workload and m.group(3) == sha:
            return float(m.group(2))
    return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons while the timed region runs.

    The timed region of the default run lasts tens of milliseconds, so the samples are read through
    NVML from a thread of this process, one every millisecond or two (reads only; nothing is set);
    `nvidia-smi -lms`, whose shortest period is longer than the region, is the fallback."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.device = device
        self.proc = None
        self.lines = []
        self.samples = []          # (time, sm MHz, power W, reasons bit mask)
        self.nvml = None
        self.handle = None
        self.stop_flag = False
        self.thread = None
        self.sm_max = None

    def _nvml_open(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(self.device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except TypeError:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            pynvml.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
            self.nvml = pynvml
            return True
        except Exception:
            self.nvml = None
            return False

    def _poll(self):
        nv, h = self.nvml, self.handle
        while not self.stop_flag:
            try:
                self.samples.append((time.time(), float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                     nv.nvmlDeviceGetPowerUsage(h) / 1000.0,
                                     int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))))
            except Exception:
                break
            time.sleep(0.001)

    def start(self):
        if self._nvml_open():
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.device.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def _stop_nvml(self, t0, t1):
        nv = self.nvml
        self.stop_flag = True
        self.thread.join(timeout=2)
        rows = [x for x in self.samples if t0 <= x[0] <= t1] or self.samples[-3:]
        bits = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        reasons = sorted(name for name, bit in bits.items() if any(x[3] & bit for x in rows))
        return {"sm_mhz": float(np.median([x[1] for x in rows])) if rows else None,
                "sm_min_mhz": float(min(x[1] for x in rows)) if rows else None,
                "sm_max_mhz": self.sm_max,
                "power_w": float(np.median([x[2] for x in rows])) if rows else None,
                "samples": len(rows), "source": "nvml", "reasons": reasons}

    def stop(self, t0, t1):
        if self.nvml is not None:
            return self._stop_nvml(t0, t1)
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.2] or [l for (_, l) in self.lines[-3:]]
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for nme, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(power)) if power else None,
                "samples": len(sm), "source": "nvidia-smi", "reasons": sorted(reasons)}


def flops(wl, N, k_per_head):
    """(dense-equivalent, effective) attention FLOPs of one call at sequence length N."""
    NB = (N + 63) // 64
    n_pad = NB * 64
    dense = 4.0 * wl.B * wl.H * float(n_pad) ** 2 * wl.d
    eff = 4.0 * wl.B * sum(float(n_pad) * 64 * k * wl.d for k in k_per_head)
    return dense, eff


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank timings over all ranks (every rank gets the result).
    The job is as slow as its slowest rank; there is no data-path collective besides this."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return t.tolist()


def job_value(world, flops_per_rank, ms_per_step):
    """Whole-job throughput in TFLOP/s: every rank runs one layer instance (weak scaling)."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def make_config(wl, merge_window=None, fused_unmerge=False):
    """The workload description both arms print (identical keys and values)."""
    N = wl.N_attn
    return {"workload": wl.name, "B": wl.B, "H": wl.H, "d": wl.d, "N": N, "blocks": (N + 63) // 64,
            "k_per_head": sorted(set(wl.k_per_head())), "merge_r": wl.r,
            "merge_window": list(merge_window) if merge_window else None, "fused_unmerge": bool(fused_unmerge),
            "per_gpu": "one layer instance per GPU (heads/batch shard, no collective)",
            "l2": ("inputs larger than L2 (q,k,v,o = %.0f MB per step), no flush" if 4 * wl.B * wl.H * N * wl.d * 2 > 126e6
                   else "q,k,v,o = %.1f MB per step: fits in L2, not flushed (sanity workload)")
                  % (4 * wl.B * wl.H * N * wl.d * 2 / 1e6)}


def build_inputs(wl, device):
    """Device-resident inputs of one step.  Returns a dict."""
    if wl.merge_part is None:
        q, k, v = ui.make_qkv(wl, device=device, layout="bhnd")
        return dict(q=q, k=k, v=v, N=wl.N)
    z = ui.make_hidden(wl, device)                                   # [B,N,C]
    w = ui.make_qkv_weight(wl, device)                               # [C,3C]
    metric = (z @ w[:, wl.C:2 * wl.C]).reshape(wl.B, wl.N, wl.H, wl.d).contiguous()
    return dict(z=z, w=w, metric=metric, N=wl.N_attn)


def time_call(fn, iters=20, warmup=3):
    """Mean CUDA-event time of fn() in ms (current stream)."""
    for _ in range(warmup):
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def hbm_entry(call, kernels, nbytes, ms, peak_gbs, note=None):
    gbs = nbytes / (ms * 1e-3) / 1e9
    d = {"call": call, "kernels": kernels, "bound": "hbm", "bytes": int(nbytes), "ms": ms,
         "achieved": gbs, "peak": peak_gbs, "unit": "GB/s", "frac": gbs / peak_gbs}
    if note:
        d["note"] = note
    return d


def merge_path_rooflines(usv, device, peak_gbs):
    """HBM-bound calls of the merge path, timed on the 50 %-merge Wan 480p workload (hidden
    states 100.6 MB + merged 50.3 MB per call: larger than L2, no flush): applying a stored plan
    (CSR build + merge_kernel) and the unmerge gather."""
    wl = ui.workload("wan1.3b_480p_merge50")
    z = ui.make_hidden(wl, device)
    w = ui.make_qkv_weight(wl, device)
    metric = (z @ w[:, wl.C:2 * wl.C]).reshape(wl.B, wl.N, wl.H, wl.d).contiguous()
    del w
    zm, plan = usv.token_merge(z, metric, wl.grid, wl.merge_part, wl.r)
    y = torch.empty_like(z)
    zm2 = torch.empty_like(zm)
    ms_plan = time_call(lambda: usv.token_merge(z, metric, wl.grid, wl.merge_part, wl.r, out=zm2))
    ms_apply = time_call(lambda: usv.token_merge(z, None, wl.grid, wl.merge_part, wl.r, plan=plan, out=zm2))
    usv.merge_plan_cache(plan)
    ms_cached = time_call(lambda: usv.token_merge_apply(z, plan, out=zm2))
    ms_unm = time_call(lambda: usv.token_unmerge(zm, plan.pos, out=y))
    moved = z.numel() * 2 + zm.numel() * 2
    desc_bytes = metric.numel() * 2 + wl.B * wl.N * wl.d * 4
    return [
        hbm_entry("usv_token_merge_apply", "merge_kernel (merged-source lists cached with the plan)", moved, ms_cached, peak_gbs),
        hbm_entry("usv_token_merge(metric=NULL)", "csr_count/scan/fill + merge_kernel", moved, ms_apply, peak_gbs,
                  "merge_kernel streams the bytes; the three CSR kernels before it are latency-bound"),
        hbm_entry("usv_token_unmerge", "unmerge_kernel", moved, ms_unm, peak_gbs),
        {"call": "usv_token_merge(metric)", "kernels": "desc + split + match_tc + rescore + plan + CSR + merge",
         "bound": "tensor (matching) + hbm (descriptors, merge)", "ms": ms_plan,
         "bytes_descriptors": int(desc_bytes), "bytes_merge": int(moved),
         "note": "whole call; the plan-building part is %.4f ms" % (ms_plan - ms_apply)},
    ], {"workload": wl.name, "B": wl.B, "N": wl.N, "C": wl.C, "r": wl.r}


def run_usv(args, wl, rank, world, device):
    import paper_2512_05754_b200 as usv
    peaks, peak_src = load_peaks()
    inp = build_inputs(wl, device)
    kph = wl.k_per_head()
    N = inp["N"]
    dense_f, eff_f = flops(wl, N, kph)
    merging = wl.merge_part is not None
    win = tuple(int(v) for v in args.merge_window.split(",")) if (merging and args.merge_window) else None
    ev = lambda: torch.cuda.Event(enable_timing=True)

    if merging:
        # projection of the merged hidden states is harness work (outside the library); it is
        # done once, untimed, so that the timed step holds only the library's kernels.
        zm, plan = usv.token_merge(inp["z"], inp["metric"], wl.grid, wl.merge_part, wl.r, window=win)
        qkv = (zm @ inp["w"]).reshape(wl.B, N, 3, wl.H, wl.d)
        q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))   # [B,H,N,d] views
        o = torch.empty((wl.B, N, wl.H, wl.d), dtype=torch.bfloat16, device=device).permute(0, 2, 1, 3)
    else:
        q, k, v = inp["q"], inp["k"], inp["v"]
        o = torch.empty_like(q)

    marks = []
    fused = merging and args.fused_unmerge and wl.d == 128
    y_full = torch.empty((wl.B, wl.N, wl.C), dtype=torch.bfloat16, device=device) if fused else None

    def step(record=False):
        e = [ev() for _ in range(6)] if record else None
        if record: e[0].record()
        umap = None
        if merging:
            _, pl = usv.token_merge(inp["z"], inp["metric"], wl.grid, wl.merge_part, wl.r, window=win)
            if fused:
                umap = usv.unmerge_map(pl.pos, N)      # inverse of the plan's pos, part of building the plan
        if record: e[1].record()
        s = usv.block_scores(q, k, N, N)
        if record: e[2].record()
        sel = usv.select_blocks(s, kph)
        if record: e[3].record()
        if fused:
            usv.sparse_attn_fwd_unmerge(q, k, v, sel, kph, umap, wl.N, N=N, out=y_full)
        else:
            usv.sparse_attn_fwd(q, k, v, sel, kph, N=N, out=o)
        if record: e[4].record()
        if merging and not fused:
            usv.token_unmerge(o.permute(0, 2, 1, 3).reshape(wl.B, N, wl.C), plan.pos)
        if record:
            e[5].record()
            marks.append(e)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(device)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)
    t_wall0 = time.time()
    e0, e1 = ev(), ev()
    barrier()
    launches0 = usv.kernel_launches()
    e0.record()
    for _ in range(args.steps):
        step(record=True)
    e1.record()
    launches = usv.kernel_launches() - launches0     # the library's own count of what it enqueued
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    total_ms = e0.elapsed_time(e1)
    seg = np.array([[m[i].elapsed_time(m[i + 1]) for i in range(5)] for m in marks])  # ms
    seg_mean = seg.mean(0)
    # the status word is sticky: a bounded wait that gave up in ANY step shows up here
    assert usv.workspace_status() == 0, "a device-side wait gave up during the timed steps"

    # ---- end to end through the public API with pinned host buffers: every step copies its
    # inputs from the host, runs the whole path and copies the result back.  Copies and kernels
    # run on three streams over two sets of device buffers, so that step i + 1's inputs arrive
    # and step i - 1's result leaves while step i computes (the usual way to feed a GPU from the
    # host); every step still moves all its bytes inside the timed region.
    if merging:
        hz, hm = inp["z"].cpu().pin_memory(), inp["metric"].cpu().pin_memory()
        dz = [torch.empty_like(inp["z"]) for _ in range(2)]
        dmet = [torch.empty_like(inp["metric"]) for _ in range(2)]
        hy = torch.empty(inp["z"].shape, dtype=torch.bfloat16).pin_memory()
        do = torch.empty((wl.B, N, wl.H, wl.d), dtype=torch.bfloat16, device=device).permute(0, 2, 1, 3)
        dy = [torch.empty_like(inp["z"]) for _ in range(2)]
        h2d, d2h = hz.numel() * 2 + hm.numel() * 2, hy.numel() * 2

        def e2e_in(b):
            dz[b].copy_(hz, non_blocking=True); dmet[b].copy_(hm, non_blocking=True)

        def e2e_compute(b):
            zm_, plan_ = usv.token_merge(dz[b], dmet[b], wl.grid, wl.merge_part, wl.r, window=win)
            qkv_ = (zm_ @ inp["w"]).reshape(wl.B, N, 3, wl.H, wl.d)      # harness projection (cuBLAS), inside the timed region
            q_, k_, v_ = (qkv_[:, :, i].permute(0, 2, 1, 3) for i in range(3))
            sel_ = usv.select_blocks(usv.block_scores(q_, k_, N, N), kph)
            usv.sparse_attn_fwd(q_, k_, v_, sel_, kph, N=N, out=do)
            usv.token_unmerge(do.permute(0, 2, 1, 3).reshape(wl.B, N, wl.C), plan_.pos, out=dy[b])

        def e2e_out(b):
            hy.copy_(dy[b], non_blocking=True)
    else:
        hq, hk, hv = (t.contiguous().cpu().pin_memory() for t in (q, k, v))
        ho = torch.empty(o.shape, dtype=o.dtype).pin_memory()
        dq, dk, dv, do2 = ([torch.empty_like(hq, device=device) for _ in range(2)] for _ in range(4))
        h2d, d2h = 3 * hq.numel() * 2, ho.numel() * 2

        def e2e_in(b):
            dq[b].copy_(hq, non_blocking=True); dk[b].copy_(hk, non_blocking=True); dv[b].copy_(hv, non_blocking=True)

        def e2e_compute(b):
            s = usv.block_scores(dq[b], dk[b], N, N)
            sel = usv.select_blocks(s, kph)
            usv.sparse_attn_fwd(dq[b], dk[b], dv[b], sel, kph, N=N, out=do2[b])

        def e2e_out(b):
            ho.copy_(do2[b], non_blocking=True)

    s_comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    in_done, comp_done, out_done = ([None, None] for _ in range(3))

    def e2e_run(nsteps, start=None):
        if start is not None:
            s_in.wait_event(start); s_out.wait_event(start)
        for i in range(nsteps):
            b = i & 1
            with torch.cuda.stream(s_in):
                if comp_done[b] is not None:
                    s_in.wait_event(comp_done[b])        # the step that last read these input buffers
                e2e_in(b)
                in_done[b] = ev(); in_done[b].record(s_in)
            s_comp.wait_event(in_done[b])
            if out_done[b] is not None:
                s_comp.wait_event(out_done[b])           # the copy that last read this output buffer
            e2e_compute(b)
            comp_done[b] = ev(); comp_done[b].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[b])
                e2e_out(b)
                out_done[b] = ev(); out_done[b].record(s_out)
        for e in out_done:
            if e is not None:
                s_comp.wait_event(e)

    e2e_steps = max(3, min(args.steps, 20))
    e2e_run(3)
    barrier()
    f0, f1 = ev(), ev()
    f0.record()
    e2e_run(e2e_steps, f0)
    f1.record()
    barrier()
    e2e_ms = f0.elapsed_time(f1) / e2e_steps
    assert usv.workspace_status() == 0

    entropy_ms = None
    if args.with_entropy:
        s_ = usv.block_scores(q, k, N, N)
        sel_ = usv.select_blocks(s_, kph)
        _, lse_ = usv.sparse_attn_fwd(q, k, v, sel_, kph, N=N, out=o, return_lse=True)
        entropy_ms = time_call(lambda: usv.attn_entropy(q, k, sel_, kph, lse_, N=N))

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], world, device)
    if rank != 0:
        return None
    ms_step = total_ms / args.steps
    attn_ms = float(seg_mean[3])
    peak = peaks["bf16_tflops"]
    attn_eff_tflops = eff_f / (attn_ms * 1e-3) / 1e12
    hbm = peaks["hbm_gbs"]
    NB = (N + 63) // 64
    # algorithmic bytes: Q and K read once, fp32 means written; scores read once, selection written
    pool_bytes = 2 * (wl.B * wl.H * N * wl.d * 2) + 2 * (wl.B * wl.H * NB * wl.d * 4)
    scores_bytes = wl.B * wl.H * NB * NB * 4
    select_bytes = scores_bytes + wl.B * wl.H * NB * max(kph) * 4
    # the streaming kernel of usv_block_scores by itself (pool_kernel: first launch of the call)
    hbm_list = [
        hbm_entry("usv_block_scores", "pool_kernel + scores (tensor-core) kernel", pool_bytes + scores_bytes,
                  float(seg_mean[1]), hbm,
                  "whole call: the pooling stream plus the small score product and its launch gaps"),
        hbm_entry("usv_select_blocks", "select kernel", select_bytes, float(seg_mean[2]), hbm,
                  "latency-bound: one warp (rows <= 2048 scores) or CTA per row searches its k-th largest score"),
    ]
    result = {
        "metric": "sparse_attn_dense_equiv_tflops",
        "value": job_value(world, dense_f, ms_step),
        "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16",
        "data": "synthetic",
        "config": make_config(wl, win, fused),
        "breakdown_ms": {"token_merge": float(seg_mean[0]), "block_scores": float(seg_mean[1]),
                         "select_blocks": float(seg_mean[2]), "sparse_attn_fwd": attn_ms,
                         "token_unmerge": float(seg_mean[4]),
                         "sparse_attn_fwd_min": float(seg[:, 3].min())},
        "effective_tflops": {"attn_kernel": attn_eff_tflops,
                             "step": eff_f / (ms_step * 1e-3) / 1e12,
                             "note": "effective = only the selected blocks' FLOPs; `value` is the dense-equivalent "
                                     "figure (the work dense attention would have done / step time) and is not a "
                                     "hardware rate",
                             "frac_of_measured_burst": attn_eff_tflops / peak,
                             "frac_of_measured_sustained": attn_eff_tflops / peaks["bf16_tflops_sustained"],
                             "frac_of_nominal_2250": attn_eff_tflops / NOMINAL_BF16_TFLOPS},
        "roofline": {"bound": "tensor", "kernel": "sparse_attn_fwd (pair_plan_kernel + attn_pair_kernel)",
                     "achieved": attn_eff_tflops, "peak": peak, "unit": "TFLOP/s",
                     "frac": attn_eff_tflops / peak, "peak_source": "%s (burst bf16)" % peak_src,
                     "traffic": attn_dram_traffic(wl.name)},
        "hbm_rooflines": hbm_list,
        "e2e": {"value": job_value(world, dense_f, e2e_ms), "unit": "TFLOP/s",
                "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "path": ("H2D z, metric -> merge -> projection (harness) -> scores -> select -> attention -> "
                         "unmerge -> D2H y") if merging else "H2D q,k,v -> scores -> select -> attention -> D2H o",
                "overlap": "copies and kernels on three streams over two sets of device buffers; every step "
                           "moves all its bytes inside the timed region"},
        "gpu_launches": int(launches),
        "gpu_launches_source": "usv_kernel_launches(): the library's own counter around the timed steps",
        "attn_entropy_ms": entropy_ms,
        "clocks": clocks,
        "context": PAPER_CONTEXT,
    }
    if merging:
        mb = (wl.B * wl.N * wl.C * 2) + (wl.B * N * wl.C * 2)
        hbm_list.append(hbm_entry("usv_token_unmerge", "unmerge_kernel", mb, float(seg_mean[4]), hbm))
    if not args.no_merge_pass and world == 1:
        # the HBM half of the target lives on the merge path, which the headline workload does not
        # run: a short secondary pass on the 50 %-merge workload supplies those figures
        extra, cfg = merge_path_rooflines(usv, device, hbm)
        result["hbm_rooflines"] += extra
        result["hbm_rooflines_merge_workload"] = cfg
        assert usv.workspace_status() == 0
    return result, dict(q=q, k=k, v=v, N=N, kph=kph)


def oracle_sample_step(wl, q, k, v, N, kph, n_qb, seed):
    """One oracle pass: pooling, scores, selection in full; attention on n_qb sampled query
    blocks.  Returns (seconds pooled/selected, seconds attention sample, blocks total)."""
    import oracle
    t0 = time.time()
    s = oracle.block_scores(oracle.block_pool(q, N), oracle.block_pool(k, N))
    sel, _ = oracle.select_blocks(s, kph)
    t1 = time.time()
    NB = (N + 63) // 64
    allqb = oracle.all_query_blocks(wl.B, wl.H, NB)
    rng = np.random.default_rng(seed)
    pick = allqb[np.sort(rng.choice(allqb.shape[0], size=min(n_qb, allqb.shape[0]), replace=False))]
    oracle.sparse_attn(q, k, v, N, sel, kph, qb_list=pick)
    t2 = time.time()
    return t1 - t0, t2 - t1, allqb.shape[0], pick.shape[0]


def cpu_baseline(wl, tensors, n_qb=384):
    import oracle
    q, k, v = (tensors[n].contiguous().cpu() for n in ("q", "k", "v"))
    N, kph = tensors["N"], tensors["kph"]
    t_sel, t_attn, total, picked = oracle_sample_step(wl, q, k, v, N, kph, n_qb, 0)
    t_full = t_sel + t_attn * total / picked
    dense_f, _ = flops(wl, N, kph)
    return {"value": dense_f / t_full / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds_full_step_extrapolated": t_full,
            "sample": "pooling+scores+selection in full (%.2f s); attention on %d of %d query "
                      "blocks (%.2f s), extrapolated linearly" % (t_sel, picked, total, t_attn)}


def run_reference(args, wl):
    """The fp64 oracle as it stands, on host cores, same metric.  The first timed step runs the
    whole call (every query block) when that fits in about a minute and a half; every other step
    is a bounded sample of the attention, extrapolated linearly, and says so."""
    import oracle
    q, k, v = ui.make_qkv(wl, device="cpu", layout="bhnd") if wl.merge_part is None else (None,) * 3
    if q is None:
        z = ui.make_hidden(wl, "cpu")
        w = ui.make_qkv_weight(wl, "cpu")
        metric = (z.float() @ w[:, wl.C:2 * wl.C].float()).to(torch.bfloat16).reshape(wl.B, wl.N, wl.H, wl.d)
        plan = oracle.merge_plan(metric, wl.grid, wl.merge_part, wl.r)
        zm = torch.from_numpy(oracle.round_to_bf16(oracle.merge_apply(z, plan["dst_of"], plan["pos"], plan["Nm"]))
                              .view(np.int16)).view(torch.bfloat16)
        qkv = (zm.float() @ w.float()).to(torch.bfloat16).reshape(wl.B, wl.N_attn, 3, wl.H, wl.d)
        q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3).contiguous() for i in range(3))
    N, kph = wl.N_attn, wl.k_per_head()
    dense_f, _ = flops(wl, N, kph)
    n_qb = 96
    est, full_steps = [], 0
    total = picked = 0
    for i in range(args.warmup + args.steps):
        t_sel, t_attn, total, picked = oracle_sample_step(wl, q, k, v, N, kph, n_qb, i)
        t_est = t_sel + t_attn * total / picked
        if i == args.warmup and t_est <= 90.0 and picked < total:
            # one whole, un-sampled step
            t_sel, t_attn, total, _ = oracle_sample_step(wl, q, k, v, N, kph, total, i)
            t_est = t_sel + t_attn
            full_steps = 1
        elif i >= args.warmup and picked >= total:
            full_steps += 1                      # small workload: the "sample" is every query block
        if i >= args.warmup:
            est.append(t_est)
    t_full = float(np.mean(est))
    val = dense_f / t_full / 1e12
    sample = ("pooling+scores+selection in full every step; attention: %d step(s) over all %d query blocks "
              "(measured), %d step(s) on %d of %d query blocks extrapolated linearly to the full call"
              % (full_steps, total, len(est) - full_steps, min(n_qb, total), total))
    return {"impl": "reference", "metric": "sparse_attn_dense_equiv_tflops", "value": val,
            "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": t_full * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": make_config(wl),
            "measured_full_steps": full_steps, "extrapolated_steps": len(est) - full_steps,
            "extrapolated": full_steps < len(est),
            "ms_full_step_measured": est[0] * 1e3 if full_steps else None,
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def spawn_ranks(argv, n):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script (one per GPU,
    rendezvous on 127.0.0.1), pass rank 0's JSON line through, return the worst exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + argv, env=env,
                                      stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    rc = procs[0].returncode
    for p_ in procs[1:]:
        rc = max(rc, p_.wait())
    sys.stdout.write(out)
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="wan1.3b_480p")
    ap.add_argument("--impl", default="usv", choices=["usv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-merge-pass", action="store_true",
                    help="skip the secondary pass that times the merge-path calls for the HBM rooflines")
    ap.add_argument("--with-entropy", action="store_true",
                    help="also time usv_attn_entropy (Sec. 3.4) on the step's q, k, sel; reported beside the step")
    ap.add_argument("--fused-unmerge", action="store_true",
                    help="merging workloads: unmerge inside the attention epilogue (usv_sparse_attn_fwd_unmerge) "
                         "instead of a separate usv_token_unmerge call")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend of the N > 1 path (gloo + --host-check exercise its host logic on CPU)")
    ap.add_argument("--host-check", action="store_true",
                    help="no GPU work: every rank contributes made-up timings to the max-over-ranks exchange and "
                         "rank 0 prints the resulting line (tests the N > 1 plumbing on CPU)")
    ap.add_argument("--merge-window", default=None,
                    help="wt,wh,ww: keep the merge matching inside nearby partition blocks (usv arm only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "usv" else args.warmup
    wl = ui.workload(args.workload)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, wl)))
        return 0

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(sys.argv[1:], args.gpus)     # no launcher: be one

    if args.host_check:
        if world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            torch.distributed.init_process_group(args.backend, rank=rank, world_size=world)
        ms = max_over_ranks([1.0 + rank, 10.0 - rank], world, torch.device("cpu"))
        dense_f, _ = flops(wl, wl.N_attn, wl.k_per_head())
        if rank == 0:
            print(json.dumps({"host_check": True, "n_gpus": world, "ms_per_step": ms[0],
                              "value": job_value(world, dense_f, ms[0]), "max_over_ranks": ms,
                              "config": make_config(wl)}))
        if world > 1:
            torch.distributed.barrier()
            torch.distributed.destroy_process_group()
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the product and has no CPU fallback")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group(args.backend, device_id=device)
    out = run_usv(args, wl, rank, world, device)
    if rank == 0:
        result, tensors = out
        if not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline(wl, tensors)
        print(json.dumps(result))
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

#!/usr/bin/env python
"""Benchmark of the Tucker-attention forward library.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c2|c3|c5] [--impl reference]

A step is one pass of the whole hot path (one tucker_attn_fwd or tucker_attn_decode call:
core contraction, latent projections, per-head queries + latent RoPE, online-softmax
attention, output-side factors) over one batch of seeded synthetic input.  One JSON line is
printed by rank 0.  `value` is device-timed throughput with inputs resident in HBM; `e2e`
times the same call with the step's input copied from pinned host memory and its output
copied back inside the timed region.  With N > 1 (torchrun) every rank runs an independent
replica of the workload (batch-sharded replicas, no collective on the data path) and the
slowest rank sets the time.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2603_30033_b200 import workloads as W

LIB_FLAGS = 0   # TA_FLAG_* bits for every library call (set from --flags)
SUSTAINED_SECONDS = 0.0   # length of the sustained leg of the main workload (set from --sustained)

METRIC = "prefill TFLOP/s & decode GB/s vs B200 roofline (fused Tucker attention)"
KEYS = ("C", "U1", "U2", "U3", "Ct", "Ut1", "Ut2", "Ut3")
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes (read + write) of ONE launch of the dominant kernel, from an ncu capture of that kernel on this
# workload: value, the summary under profiles/ it comes from, and the SHA-256 of the kernel's source file at the
# time of the capture.  A value is only reported while that file is unchanged (see ncu_traffic()).
_ATTN = {"source": "ta_attn_prefill.cuh", "sha256": "83abe4f00b82ea24232967bb6792cee9c2eed58417272c517f4f348ff22e88c6"}
_DEC = {"source": "ta_decode_umma.cuh", "sha256": "b29368639f2d9ea4a252a55117459bd2a1a167eff6dc63668ccc285447534b03"}
NCU_TRAFFIC = {
    "c4_long_prefill": {"bytes": 17971968 + 77637120, "profile": "profiles/k_attn_prefill_c4_long_prefill.md", **_ATTN},
    "c3_vit_prefill": {"bytes": 33884416 + 64199424, "profile": "profiles/k_attn_prefill_c3_vit_prefill.md", **_ATTN},
    "c2_gpt2_prefill": {"bytes": 3584256 + 0, "profile": "profiles/k_attn_prefill_c2_gpt2_prefill.md", **_ATTN},
    "c5_decode": {"bytes": 1075363072 + 4196608, "profile": "profiles/k_dec_attn_umma_c5_decode.md", **_DEC},
    "f1_decode_shared_kv": {"bytes": 537998592 + 4850688, "profile": "profiles/k_dec_attn_umma_f1_decode_shared_kv.md", **_DEC},
    "f1r_decode_shared_kv_rope": {"bytes": 538054400 + 6371328,
                                  "profile": "profiles/k_dec_attn_umma_f1r_decode_shared_kv_rope.md", **_DEC},
}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}     # the figures the targets are quoted against


def ncu_traffic(workload: str):
    """(bytes per launch or None, provenance string)."""
    import hashlib
    rec = NCU_TRAFFIC.get(workload)
    if not rec:
        return None, "no ncu capture for this workload"
    path = os.path.join(ROOT, "paper_2603_30033_b200", "csrc", rec["source"])
    try:
        with open(path, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None, f"{rec['source']} not found"
    if digest != rec["sha256"]:
        return None, f"{rec['source']} changed since the capture in {rec['profile']}"
    return rec["bytes"], f"{rec['profile']} ({rec['source']} unchanged since)"


FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100", "-i",
                 str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if t0 is not None and not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------
# GPU arms
# ----------------------------------------------------------------------------------------

def _dev(a, dtype, torch):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return (t.to(torch.bfloat16) if dtype == "bf16" else t).cuda()


class Flusher:
    def __init__(self, torch, needed: bool):
        self.buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if needed else None

    def __call__(self):
        if self.buf is not None:
            self.buf.fill_(1)


def time_steps(torch, Bd, step_fn, steps, warmup, flush, barrier, profile=False):
    """Runs warm-up, then `steps` timed steps.  Returns (per-step ms list, per-step dominant-kernel
    ms list or None, wall interval).  With profile=True two extra events are recorded around the
    dominant kernel of every step; that pass is only used for the kernel's own duration, because
    an event between two kernels keeps their launches from overlapping."""
    for _ in range(warmup):
        flush()
        step_fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    if profile:
        for a, b in kev:      # materialise the handles
            a.record()
            b.record()
    barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    for i in range(steps):
        flush()
        if profile:
            Bd.set_profile_events(*kev[i])
        ev[i][0].record()
        step_fn()
        ev[i][1].record()
    Bd.set_profile_events()
    torch.cuda.synchronize()
    t1 = time.time()
    barrier()
    ms = [a.elapsed_time(b) for a, b in ev]
    kms = [a.elapsed_time(b) for a, b in kev] if profile else None
    return ms, kms, (t0, t1)


def pipelined_e2e(torch, steps, warmup, barrier, h2d, compute, d2h):
    """End-to-end steps with the copies overlapped across steps: step i's input copy (copy-in stream), its
    compute (compute stream) and its result copy (copy-out stream) use buffer set i % 2, so that step i + 1's
    host-to-device copy and step i - 1's device-to-host copy run while step i computes.  Every step still
    moves its own input from pinned host memory and its own result back.  Returns ms per step over `steps`
    steps (from the first copy-in to the last copy-out, so the pipeline fill is inside)."""
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def run(n):
        for i in range(n):
            b = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[b])       # the compute of step i - 2 has read this input buffer
                h2d(b)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[b])
                if i >= 2:
                    s_cmp.wait_event(ev_out[b])      # the result of step i - 2 has left this output buffer
                compute(b)
                ev_cmp[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[b])
                d2h(b)
                ev_out[b].record(s_out)
    torch.cuda.synchronize()
    run(max(warmup, 2))
    torch.cuda.synchronize()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(s_in)
    run(steps)
    s_out.wait_stream(s_in); s_out.wait_stream(s_cmp)
    t1.record(s_out)
    torch.cuda.synchronize()
    barrier()
    return t0.elapsed_time(t1) / steps


def sustained_leg(torch, step_fn, seconds, gpu_index, work, div, peak_sustained):
    """Repeats the step back to back for at least `seconds` (the burst numbers above last tens of
    milliseconds, during which the SM clock stays at its maximum; under a seconds-long load the power cap pulls
    it down).  Reports ms per step, the median SM clock sampled meanwhile and their product."""
    sampler = ClockSampler(gpu_index)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_fn()
    torch.cuda.synchronize()
    sampler.start()
    time.sleep(0.3)
    t0 = time.time()
    n = 0
    e0.record()
    while True:
        for _ in range(50):
            step_fn()
        n += 50
        if n % 200 == 0:
            torch.cuda.synchronize()
            if time.time() - t0 >= seconds:
                break
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0 + 0.5, t1)
    ms = e0.elapsed_time(e1) / n
    value = work / (ms * 1e-3) / div
    return {"seconds": t1 - t0, "steps": n, "ms_per_step": ms, "value": value, "sm_mhz_median": clocks["sm_mhz"],
            "reasons": clocks["reasons"], "ms_times_mhz": ms * clocks["sm_mhz"] if clocks["sm_mhz"] else None,
            "peak_sustained": peak_sustained, "frac_of_sustained_peak": (value / peak_sustained) if peak_sustained else None,
            "note": "inputs stay in L2 between steps where they fit; no flush in this leg"}


def bench_prefill(w, steps, warmup, torch, Bd, barrier, peaks, with_e2e=True, sampler=None):
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    dw = [_dev(wt[k], w.dtype, torch) for k in KEYS]
    X32 = torch.from_numpy(W.make_X(w))
    X_host = (X32.to(torch.bfloat16) if w.dtype == "bf16" else X32).contiguous().pin_memory()
    del X32
    X = X_host.cuda()
    Y = torch.empty_like(X)
    Y_host = torch.empty_like(X_host).pin_memory()
    desc = Bd.make_desc(B=w.B, N=w.N, d_model=w.d_model, n_H=w.n_H, r=w.r, t=w.t, causal=w.causal, rope=w.rope,
                        rope_base=w.rope_base, dtype=Bd.TA_DTYPE_BF16 if w.dtype == "bf16" else Bd.TA_DTYPE_F32)
    ws = Bd.alloc_workspace(Bd.fwd_workspace_bytes(desc), X.device)
    kw = dict(n_H=w.n_H, causal=w.causal, rope=w.rope, rope_base=w.rope_base, out=Y, workspace=ws, flags=LIB_FLAGS)

    def step():
        Bd.tucker_attn_fwd(X, *dw, **kw)

    in_bytes = X.numel() * X.element_size()
    flush = Flusher(torch, needed=in_bytes < 2 * L2_BYTES)
    if sampler:
        sampler.start()
    ms, _, (t0, t1) = time_steps(torch, Bd, step, steps, warmup, flush, barrier)
    clocks = sampler.stop(t0, t1) if sampler else None
    _, kms, _ = time_steps(torch, Bd, step, min(steps, 10), 1, flush, barrier, profile=True)
    launches = Bd.last_launch_count()
    path = Bd.last_path()
    assert Bd.last_device_error() == 0, "device error word set during the benchmark"
    fl = W.prefill_flops(w)
    ms_step = sum(ms) / len(ms)
    res = {
        "workload": w.name, "unit": "TFLOP/s", "value": fl["total"] / (ms_step * 1e-3) / 1e12, "ms_per_step": ms_step,
        "ms_best": min(ms), "flops_per_step": fl["total"], "gpu_launches_per_step": launches, "path": path,
        "l2": "L2 flushed between steps" if flush.buf is not None else "inputs larger than L2",
    }
    kms_avg = sum(kms) / len(kms)
    attn_flops = fl["scores"] + fl["pv"]
    fused_q = w.dtype == "bf16" and max(w.r[1], w.r[2], w.t[2]) <= 128   # the kernel then also forms the per-head queries
    if fused_q:
        attn_flops += fl["qhat"]
    peak = peaks["bf16_tflops"] if w.dtype == "bf16" else None
    ach = attn_flops / (kms_avg * 1e-3) / 1e12
    res["roofline"] = {
        "kernel": ("attention (per-head queries + scores + online softmax + PV)" if fused_q
                   else "attention (scores + online softmax + PV)"), "bound": "tensor", "achieved": ach, "peak": peak,
        "unit": "TFLOP/s", "frac": (ach / peak) if peak else None, "traffic": ncu_traffic(w.name)[0],
        "traffic_source": ncu_traffic(w.name)[1], "kernel_ms": kms_avg,
        "flops_per_launch": attn_flops, "whole_step_frac_of_peak": (res["value"] / peak) if peak else None,
        "frac_of_nominal": ach / NOMINAL_PEAKS["bf16_tflops"],
        "whole_step_frac_of_nominal": res["value"] / NOMINAL_PEAKS["bf16_tflops"],
    }
    res["clocks"] = clocks
    if SUSTAINED_SECONDS > 0 and sampler is not None:
        res["sustained"] = sustained_leg(torch, step, SUSTAINED_SECONDS, sampler.gpu, fl["total"], 1e12,
                                         peaks.get("bf16_tflops_sustained"))
    if with_e2e:
        def e2e_step():
            X.copy_(X_host, non_blocking=True)
            Bd.tucker_attn_fwd(X, *dw, **kw)
            Y_host.copy_(Y, non_blocking=True)
        ems, _, _ = time_steps(torch, Bd, e2e_step, steps, min(warmup, 3), Flusher(torch, False), barrier)
        serial_ms = sum(ems) / len(ems)
        # the same through two buffer sets and three streams, copies overlapped with the neighbouring steps' compute
        Xb, Yb = [X, torch.empty_like(X)], [Y, torch.empty_like(Y)]
        e_ms = pipelined_e2e(
            torch, steps, min(warmup, 3), barrier,
            lambda b: Xb[b].copy_(X_host, non_blocking=True),
            lambda b: Bd.tucker_attn_fwd(Xb[b], *dw, **{**kw, "out": Yb[b]}),
            lambda b: Y_host.copy_(Yb[b], non_blocking=True))
        res["e2e"] = {"value": fl["total"] / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e_ms,
                      "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": Y.numel() * Y.element_size(),
                      "serial_ms_per_step": serial_ms,
                      "how": "copy-in, compute and copy-out on three streams with two buffer sets; serial_ms_per_step is "
                             "the same step with copy, compute, copy back to back on one stream"}
    return res


def bench_decode(w, steps, warmup, torch, Bd, barrier, peaks, with_e2e=True, sampler=None):
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    dw = [_dev(wt[k], w.dtype, torch) for k in KEYS]
    shared = getattr(w, "shared_kv", False)
    if shared:
        dw[7] = dw[3]           # the same device tensor for U3 and Ut3 selects the shared projection
    L, Lmax, B = w.N, w.N + 1, w.B
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    Kc = torch.empty(B, Lmax, w.r[2], dtype=tdt, device="cuda")
    Vc = Kc if shared else torch.empty(B, Lmax, w.t[2], dtype=tdt, device="cuda")
    for b in range(B):      # cache entries ~ N(0,1), drawn on the device one sequence at a time
        Kc[b] = torch.randn(Lmax, w.r[2], generator=gen, device="cuda", dtype=torch.float32).to(tdt)
        if not shared:
            Vc[b] = torch.randn(Lmax, w.t[2], generator=gen, device="cuda", dtype=torch.float32).to(tdt)
    x32 = torch.from_numpy(W.make_decode_x(w))
    x_host = (x32.to(tdt)).contiguous().pin_memory()
    x = x_host.cuda()
    y = torch.empty_like(x)
    y_host = torch.empty_like(x_host).pin_memory()
    lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
    desc = Bd.make_desc(B=B, N=1, d_model=w.d_model, n_H=w.n_H, r=w.r, t=w.t, causal=True, rope=w.rope,
                        rope_base=w.rope_base, dtype=Bd.TA_DTYPE_BF16 if w.dtype == "bf16" else Bd.TA_DTYPE_F32)
    ws = Bd.alloc_workspace(Bd.decode_workspace_bytes(desc, Lmax), x.device)
    kw = dict(n_H=w.n_H, rope=w.rope, rope_base=w.rope_base, append=True, out=y, workspace=ws, flags=LIB_FLAGS)

    def step():
        Bd.tucker_attn_decode(x, *dw, Kc, Vc, lens, **kw)

    by = W.decode_bytes(w)
    flush = Flusher(torch, needed=by["total"] < 2 * L2_BYTES)
    if sampler:
        sampler.start()
    ms, _, (t0, t1) = time_steps(torch, Bd, step, steps, warmup, flush, barrier)
    clocks = sampler.stop(t0, t1) if sampler else None
    _, kms, _ = time_steps(torch, Bd, step, min(steps, 10), 1, flush, barrier, profile=True)
    launches, path = Bd.last_launch_count(), Bd.last_path()
    assert Bd.last_device_error() == 0, "device error word set during the benchmark"
    ms_step = sum(ms) / len(ms)
    res = {
        "workload": w.name, "unit": "GB/s", "value": by["total"] / (ms_step * 1e-3) / 1e9, "ms_per_step": ms_step,
        "ms_best": min(ms), "bytes_per_step": by["total"], "gpu_launches_per_step": launches, "path": path,
        "l2": "L2 flushed between steps" if flush.buf is not None else "inputs larger than L2",
    }
    kms_avg = sum(kms) / len(kms)
    ach = by["cache"] / (kms_avg * 1e-3) / 1e9
    res["roofline"] = {
        "kernel": "decode attention over the latent KV cache", "bound": "hbm", "achieved": ach,
        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": ncu_traffic(w.name)[0],
        "traffic_source": ncu_traffic(w.name)[1], "kernel_ms": kms_avg, "bytes_per_launch": by["cache"],
        "whole_step_frac_of_peak": res["value"] / peaks["hbm_gbs"],
        "frac_of_nominal": ach / NOMINAL_PEAKS["hbm_gbs"],
        "whole_step_frac_of_nominal": res["value"] / NOMINAL_PEAKS["hbm_gbs"],
    }
    res["clocks"] = clocks
    if with_e2e:
        def e2e_step():
            x.copy_(x_host, non_blocking=True)
            Bd.tucker_attn_decode(x, *dw, Kc, Vc, lens, **kw)
            y_host.copy_(y, non_blocking=True)
        ems, _, _ = time_steps(torch, Bd, e2e_step, steps, min(warmup, 3), flush, barrier)
        e_ms = sum(ems) / len(ems)
        res["e2e"] = {"value": by["total"] / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e_ms,
                      "h2d_bytes_per_step": x.numel() * x.element_size(),
                      "d2h_bytes_per_step": y.numel() * y.element_size(),
                      "note": "the latent KV cache is layer state and stays resident in HBM"}
    return res


# ----------------------------------------------------------------------------------------
# CPU oracle arm (bounded sample)
# ----------------------------------------------------------------------------------------

def oracle_sample(w, scale=1.0):
    """Returns (callable running the oracle on a bounded sample, work in the metric's unit
    numerator, description, unit).  `scale` enlarges the default sample: more sequences first (up to the
    workload's batch), then more query rows per sequence (up to all of them)."""
    from oracle import tucker_oracle as O
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    args = [wt[k] for k in KEYS]
    if w.kind == "prefill":
        nrows = {"c4_long_prefill": 256, "c2_gpt2_prefill": 1024, "c3_vit_prefill": 197}.get(w.name, min(w.N, 256))
        nseq = {"c3_vit_prefill": 8}.get(w.name, 1)
        nseq2 = int(min(w.B, max(nseq, round(nseq * scale))))
        nrows = int(min(w.N, max(nrows, round(nrows * scale * nseq / nseq2))))
        nseq = nseq2
        rows = sorted(set(np.linspace(0, w.N - 1, nrows).astype(int).tolist()))
        X = W.round_to_storage(W.make_X(w, B=nseq), w.dtype)
        r1, r2, r3 = w.r
        t1, t2, t3 = w.t
        pairs = sum((r + 1) if w.causal else w.N for r in rows)
        flops = nseq * (2 * w.N * w.d_model * (r2 + r3 + t3) + 2 * w.n_H * pairs * (r3 + t3)
                        + len(rows) * (2 * w.n_H * (r2 * r3 + t3 * t2) + 2 * t2 * w.d_model)) \
            + 2 * w.n_H * (r1 * r2 * r3 + t1 * t2 * t3)

        def run():
            return O.tucker_attn_fwd(X, *args, causal=w.causal, rope=w.rope, rope_base=w.rope_base, rows=rows)
        desc = (f"{nseq} of {w.B} sequences, projections for all {w.N} tokens, attention and output for "
                f"{len(rows)} evenly spaced query rows per sequence")
        return run, flops / 1e12, desc, "TFLOP/s"
    nseq = int(min(w.B, max(4, round(4 * scale))))
    L = w.N
    x = W.round_to_storage(W.make_decode_x(w, B=nseq), w.dtype)
    Kc = np.zeros((nseq, L + 1, w.r[2]))
    Vc = np.zeros((nseq, L + 1, w.t[2]))
    for b in range(nseq):
        k, v = W.decode_cache_rows(w, b, L)
        Kc[b, :L], Vc[b, :L] = W.round_to_storage(k, w.dtype), W.round_to_storage(v, w.dtype)
    if getattr(w, "shared_kv", False):
        Vc = Kc                 # one latent cache serves keys and values
    lens = np.full((nseq,), L, dtype=np.int32)
    by = W.decode_bytes(w, B=nseq)

    def run():
        if getattr(w, "shared_kv", False) and w.rope:      # one cache of un-rotated rows, keys rotated when used
            return O.tucker_attn_decode_shared_rope(x, *args[:7], Kc, lens, rope_base=w.rope_base)
        return O.tucker_attn_decode(x, *args, Kc, Vc, lens, rope=w.rope, rope_base=w.rope_base)
    return run, by["total"] / 1e9, f"{nseq} of {w.B} sequences with the full {L}-entry cache", "GB/s"


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(w, steps=1, warmup=0, budget_s=10.0):
    """Times the oracle, as it stands, on a bounded sample of the workload sized to take about `budget_s`
    seconds per run on this host: the default sample is timed once as a probe and enlarged accordingly."""
    run, work, desc, unit = oracle_sample(w)
    t = time.perf_counter()
    run()
    probe = max(time.perf_counter() - t, 1e-3)
    if budget_s / probe >= 1.5:
        run, work, desc, unit = oracle_sample(w, scale=budget_s / probe)
    for _ in range(warmup):
        run()
    ts = []
    for _ in range(steps):
        t = time.perf_counter()
        run()
        ts.append(time.perf_counter() - t)
    sec = sum(ts) / len(ts)
    return {"value": work / sec, "unit": unit, "cores": oracle_threads(), "kind": "oracle", "sample": desc,
            "seconds_per_sample": sec}


def run_reference(args, rank):
    if rank != 0:
        return
    w = W.get_workload(args.workload)
    # every step is one bounded sample; their size is set so that the whole run stays within a few minutes
    n_runs = max(1, args.steps) + min(args.warmup, 1)
    cb = time_oracle(w, steps=max(1, args.steps), warmup=min(args.warmup, 1), budget_s=min(10.0, max(0.5, 120.0 / n_runs)))
    line = {
        "impl": "reference", "metric": METRIC, "value": cb["value"], "unit": cb["unit"], "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": cb["seconds_per_sample"] * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, **_cfg(w)}, "cpu_baseline": cb,
        "e2e": {"value": cb["value"], "unit": cb["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(values, dist=None, device="cpu"):
    """Slowest rank sets the time: element-wise MAX of a list of per-rank floats over the process
    group (identity without one).  Works with NCCL (device tensors) and gloo (CPU tensors)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_value(work_per_rank, world, ms):
    """Units all ranks processed (independent replicas: world x the per-rank work) per second."""
    return world * work_per_rank / (ms * 1e-3)


def _cfg(w):
    return {"kind": w.kind, "B": w.B, "N_or_cache_len": w.N, "d_model": w.d_model, "n_H": w.n_H,
            "ranks_qk": list(w.r), "ranks_vo": list(w.t), "causal": w.causal, "rope": w.rope,
            "rope_base": w.rope_base, "storage": w.dtype}


# ----------------------------------------------------------------------------------------

def bench_pack(torch, Bd, peaks, steps=10):
    """Next row f-3: MHA weights of the c2 layer (d = 768, 12 heads) packed as Tucker-attention weights.
    Bytes that must move: the four [d, d] inputs read, the eight outputs written."""
    d, n_H = 768, 12
    g = torch.Generator(device="cuda")
    g.manual_seed(1100)
    Ws = [torch.randn(d, d, device="cuda", dtype=torch.bfloat16, generator=g) for _ in range(4)]
    outs = Bd.tucker_pack_mha(*Ws, n_H=n_H)
    nbytes = sum(t.numel() * t.element_size() for t in Ws) + sum(t.numel() * t.element_size() for t in outs)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    times = []
    for i in range(steps + 3):
        flush.fill_(i & 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        Bd.tucker_pack_mha(*Ws, n_H=n_H, out=outs)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            times.append(e0.elapsed_time(e1))
    ms = sum(times) / len(times)
    ach = nbytes / (ms * 1e-3) / 1e9
    return {"workload": "f3_pack_mha_gpt2", "unit": "GB/s", "value": ach, "ms_per_step": ms, "bytes_per_step": nbytes,
            "gpu_launches_per_step": 1, "l2": "flushed between steps",
            "roofline": {"kernel": "weight packers (selector core, copies, transpose)", "bound": "hbm", "achieved": ach,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": None,
                         "kernel_ms": ms, "whole_step_frac_of_peak": ach / peaks["hbm_gbs"]}}


def bench_hosvd(torch, Bd, peaks, steps=3):
    """Next row f-4: HOSVD initialiser on synthetic low-rank-plus-noise MHA weights of the c2 layer shape
    (d = 768, 12 heads), ranks (12, 64, 64).  The dominant kernels are the two d x d Gram matrices of the
    mode unfoldings, one bf16 tensor-core GEMM each with K = 3 n_H d (high / low split of the fp32 tensor)."""
    d, n_H, ranks = 768, 12, (12, 64, 64)
    wm = W.make_lowrank_mha(d, n_H, 64, 0.02, 1200)
    dev = [torch.from_numpy(np.ascontiguousarray(wm[k], dtype=np.float32)).cuda() for k in ("WQ", "WK", "WV", "WO")]
    Wt, _ = Bd.tucker_mha_weight_tensors(*dev, n_H=n_H)
    ws = Bd.alloc_workspace(load_hosvd_ws(Bd, d, n_H, ranks), Wt.device)
    times, ktimes = [], []
    for i in range(steps + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0.record(); k1.record()
        Bd.set_profile_events(k0, k1)
        e0.record()
        Bd.tucker_hosvd_init(Wt, ranks, workspace=ws)
        e1.record()
        Bd.set_profile_events()
        torch.cuda.synchronize()
        if i >= 1:
            times.append(e0.elapsed_time(e1))
            ktimes.append(k0.elapsed_time(k1))
    assert Bd.last_device_error() == 0
    launches = Bd.last_launch_count()
    ms, kms = sum(times) / len(times), sum(ktimes) / len(ktimes)
    gram_flops_bf16 = 2.0 * d * d * (3 * n_H * d)          # executed on the tensor cores by one Gram GEMM
    ach = gram_flops_bf16 / (kms * 1e-3) / 1e12
    return {"workload": "f4_hosvd_init_gpt2_layer", "unit": "ms", "value": ms, "ms_per_step": ms,
            "gpu_launches_per_step": launches, "l2": "one tensor of 28 MB, resident",
            "roofline": {"kernel": "Gram matrix of a mode unfolding (k_umma_gemm, bf16 high/low split, split-K fp32 partials)",
                         "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": ach / peaks["bf16_tflops"], "traffic": None, "kernel_ms": kms,
                         "flops_per_launch": gram_flops_bf16, "algorithmic_fp32_flops_per_launch": gram_flops_bf16 / 3,
                         "whole_step_frac_of_peak": None}}


def bench_plane_mix(torch, Bd):
    """Row f-2 (core-factorised scores), priced instead of built: the mixing of r1 = 8 score planes into the two
    score tiles of a head pair, alone, at the tile count of the long causal prefill (66560 [128 x 128] tiles of
    head pairs over 148 SMs = 450 per SM), against the tensor-core cycles per tile that the form could save."""
    cyc, ms = Bd.probe_plane_mix(450, 8, 148)
    # what the form replaces: per head pair and tile 2 score MMAs of 128 x 128 x 128 (about 560 cycles each at the
    # measured 70 cycles per K = 16 step); with r1 = 8 planes and n_H = 32 heads it would issue 8 / 16 of them
    saved = 2 * 8 * 70.0 * (1.0 - 8.0 / 32.0)
    return {"workload": "f2_plane_mix_probe", "unit": "cycles/tile", "value": cyc, "ms_per_step": ms,
            "gpu_launches_per_step": 1, "l2": "n/a",
            "note": f"mixing alone: {cyc:.0f} cycles per tile and head pair in the softmax warps; tensor-core cycles "
                    f"it could save per tile and head pair: at most {saved:.0f}, on a tensor pipe that is half idle",
            "roofline": {"kernel": "plane mixing S_h = sum_a U1[h,a] P_a (FMA pipe)", "bound": "alu", "achieved": None,
                         "peak": None, "unit": "cycles/tile", "frac": None, "traffic": None, "kernel_ms": ms,
                         "whole_step_frac_of_peak": None}}


def bench_mma_rates(torch, Bd):
    """Cycles per tcgen05.mma (128 x N x 16, bf16) by operand source and layout, all SMs busy."""
    names = {0: "A, B shared memory K-major", 1: "A in TMEM, B K-major", 2: "B MN-major in shared memory"}
    table = {f"{names[m]}, N={n}": round(Bd.probe_mma_rate(m, n), 1) for m in (0, 1, 2) for n in (64, 128, 256)}
    assert Bd.last_device_error() == 0
    return {"workload": "mma_rate_probe", "unit": "cycles per MMA (N=128, smem K-major)", "value": table["A, B shared memory K-major, N=128"],
            "ms_per_step": 0.0, "gpu_launches_per_step": 9, "l2": "n/a", "note": table,
            "roofline": {"kernel": "tcgen05.mma issue rate", "bound": "tensor", "achieved": None, "peak": None, "unit": "cycles",
                         "frac": None, "traffic": None, "kernel_ms": 0.0, "whole_step_frac_of_peak": None}}


def load_hosvd_ws(Bd, d, n_H, ranks):
    return int(Bd.load_library().tucker_hosvd_workspace_bytes(int(d), int(n_H), int(ranks[1]), int(ranks[2])))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-others", action="store_true", help="skip the secondary workloads")
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0, help="TA_FLAG_* bits passed to the library (route selection)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustained", type=float, default=2.0,
                    help="seconds of back-to-back steps for the sustained-clock leg of a prefill workload (0 = skip)")
    args = ap.parse_args()
    global LIB_FLAGS, SUSTAINED_SECONDS
    LIB_FLAGS = args.flags
    SUSTAINED_SECONDS = args.sustained
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_2603_30033_b200 import binding as Bd
    Bd.load_library()          # raises if the CUDA library is missing: there is no fallback
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    peaks, peak_kind = load_peaks()
    if args.workload in ("f2", "f3", "f4", "mma"):
        # the widened rows that are not layer steps: the plane-mixing probe, the weight packers, the HOSVD initialiser
        o = {"f2": lambda: bench_plane_mix(torch, Bd), "f3": lambda: bench_pack(torch, Bd, peaks),
             "f4": lambda: bench_hosvd(torch, Bd, peaks), "mma": lambda: bench_mma_rates(torch, Bd)}[args.workload]()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": o["value"], "unit": o["unit"], "n_gpus": world, "steps": args.steps,
                              "warmup": args.warmup, "ms_per_step": o["ms_per_step"], "higher_is_better": o["unit"] != "ms",
                              "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                              "config": {"workload": o["workload"]}, "roofline": o["roofline"], "cpu_baseline": None,
                              "gpu_launches": o["gpu_launches_per_step"], "note": o.get("note")}))
        if dist is not None:
            dist.destroy_process_group()
        return
    w = W.get_workload(args.workload)
    fn = bench_prefill if w.kind == "prefill" else bench_decode
    gpu_index = local_rank
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            gpu_index = int(vis.split(",")[local_rank])
        except Exception:
            gpu_index = local_rank
    res = fn(w, args.steps, args.warmup, torch, Bd, barrier, peaks, with_e2e=True, sampler=ClockSampler(gpu_index))

    ms, e2e_ms = max_over_ranks([res["ms_per_step"], res["e2e"]["ms_per_step"]], dist, "cuda")
    work = res.get("flops_per_step", res.get("bytes_per_step"))
    div = 1e12 if w.kind == "prefill" else 1e9
    value = whole_job_value(work, world, ms) / div
    e2e_value = whole_job_value(work, world, e2e_ms) / div

    others = []
    if not args.no_others and world == 1:
        for name in ("c2", "c3", "c4", "c5", "f1", "f1r"):
            ow = W.get_workload(name)
            if ow.name == w.name:
                continue
            torch.cuda.empty_cache()
            ofn = bench_prefill if ow.kind == "prefill" else bench_decode
            o = ofn(ow, max(5, min(args.steps, 20)), 3, torch, Bd, barrier, peaks, with_e2e=False)
            o.pop("clocks", None)
            others.append(o)
        torch.cuda.empty_cache()
        others.append(bench_pack(torch, Bd, peaks))
        torch.cuda.empty_cache()
        others.append(bench_hosvd(torch, Bd, peaks))
        others.append(bench_plane_mix(torch, Bd))

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(w)

    if rank == 0:
        res["roofline"]["peak_source"] = f"{peak_kind} ({'burst' if w.kind == 'prefill' else 'copy'})"
        line = {
            "metric": METRIC, "value": value, "unit": res["unit"], "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, **_cfg(w), "l2": res["l2"],
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "roofline": res["roofline"], "sustained": res.get("sustained"), "cpu_baseline": cpu_baseline,
            "clocks": res["clocks"],
            "e2e": {**res["e2e"], "value": e2e_value, "ms_per_step": e2e_ms},
            "gpu_launches": res["gpu_launches_per_step"] * args.steps, "path": res["path"],
            "ms_best": res["ms_best"], "other_workloads": others,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

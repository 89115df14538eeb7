"""Shared test plumbing: build seeded inputs once, hand bit-identical values to the oracle
(as float64) and to the CUDA library (as torch tensors of the storage dtype)."""
from __future__ import annotations

import dataclasses

import numpy as np

from paper_2603_30033_b200 import workloads as W

WEIGHT_KEYS = ("C", "U1", "U2", "U3", "Ct", "Ut1", "Ut2", "Ut3")


def custom_workload(name="custom", **kw) -> W.Workload:
    base = dict(name=name, kind="prefill", B=1, N=16, d_model=32, n_H=4, r=(2, 8, 8), t=(2, 8, 8), causal=True,
                rope=False, rope_base=10000.0, dtype="fp32", seed=7)
    base.update(kw)
    return W.Workload(**base)


def host_inputs(w: W.Workload, B=None, N=None, core_gain=1.0, core_std=None):
    """Weights and X rounded to the storage dtype, as float64 numpy arrays."""
    wt = W.make_weights(w, core_std=core_std, core_gain=core_gain)
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in wt.items()}
    X = W.round_to_storage(W.make_X(w, B=B, N=N), w.dtype)
    return X, wt


def to_device(a: np.ndarray, dtype: str, device="cuda"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    t = t.to(torch.bfloat16) if dtype == "bf16" else t
    return t.to(device).contiguous()


def weights_to_device(wt: dict, dtype: str, device="cuda"):
    return [to_device(wt[k], dtype, device) for k in WEIGHT_KEYS]


def err_stats(got, ref):
    d = np.abs(np.asarray(got, np.float64) - np.asarray(ref, np.float64))
    return float(d.max()), float(d.mean())


def tolerances(dtype: str, ref=None):
    """(max-abs, mean-abs) bounds: bf16 storage with fp32 accumulation 2e-2 / 2e-3; fp32 1e-4.

    The bf16 bounds are absolute and are the ones the five benchmark workloads are held to;
    their outputs have rms <= 0.16.  bf16 rounding is relative (2^-9 per rounding point: the
    latent queries / keys / values, P, O, Z, Y), so for the extra stress shapes, whose outputs
    are several times larger, the bounds scale with the output size: pass `ref` to multiply
    them by max(1, rms(ref) / 0.2).  fp32 bounds never scale."""
    if dtype != "bf16":
        return (1e-4, 1e-4)
    s = 1.0
    if ref is not None:
        s = max(1.0, float(np.sqrt(np.mean(np.asarray(ref, np.float64) ** 2))) / 0.2)
    return (2e-2 * s, 2e-3 * s)


def check(got, ref, dtype, what="", scaled=False):
    """Element-wise comparison of a result with the oracle's.  scaled=False: the absolute bounds of the
    benchmark workloads; scaled=True (stress shapes with large outputs): bounds grow with the output rms,
    see tolerances().  With TA_PARITY_LOG=<file> in the environment every comparison appends its raw
    figures (max-abs, mean-abs, rms of the reference, whether the unscaled bounds would have held)."""
    import os
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    mx, mean = err_stats(got, ref)
    tmax, tmean = tolerances(dtype, ref if scaled else None)
    log = os.environ.get("TA_PARITY_LOG")
    if log:
        amax, amean = tolerances(dtype)
        rms = float(np.sqrt(np.mean(ref ** 2)))
        with open(log, "a") as f:
            f.write(f"{dtype} | {what} | max-abs {mx:.3e} | mean-abs {mean:.3e} | rms(ref) {rms:.3f} | "
                    f"{'scaled' if scaled else 'absolute'} | meets absolute: {mx <= amax and mean <= amean}\n")
    assert np.isfinite(got).all(), what
    assert mx <= tmax and mean <= tmean, f"{what}: max-abs {mx:.3e} (<= {tmax}), mean-abs {mean:.3e} (<= {tmean})"
    return mx, mean


def with_(w: W.Workload, **kw) -> W.Workload:
    return dataclasses.replace(w, **kw)

"""Seeded synthetic inputs for the Tucker-attention hot path.

This module only *generates inputs* (Gaussian draws, a QR orthonormalisation of a
Gaussian matrix, rounding to the storage dtype) and counts work.  It contains none of
the method's arithmetic, so that the CPU oracle and the CUDA path can both consume the
same arrays without sharing any code that computes attention.

Shapes follow the paper's notation (Definition 1, "Tucker Attention"):
  X   [B, N, d_model]            embedded sequence(s)
  C   [r1, r2, r3]  U1 [n_H, r1]  U2 [d_model, r2]  U3 [d_model, r3]      (pre-softmax tensor)
  Ct  [t1, t2, t3]  Ut1 [n_H, t1] Ut2 [d_model, t2] Ut3 [d_model, t3]     (post-softmax tensor;
                                                   mode 2 = output, mode 3 = value)
The five named workloads take the layer shapes of the paper's GPT-2, ViT-B/16 and
LLaMA-style experiments; the data itself is synthetic (X ~ N(0,1), orthonormal factors,
Gaussian cores) and stands in for those datasets and checkpoints.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, asdict

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "get_workload", "orthonormal_factor", "make_weights",
    "make_X", "make_decode_state", "decode_cache_rows", "make_decode_x", "round_to_storage", "prefill_flops", "decode_bytes",
    "decode_flops",
]


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str                 # "prefill" | "decode"
    B: int
    N: int                    # prefill: tokens per sequence; decode: cache length L
    d_model: int
    n_H: int
    r: tuple                  # (r1, r2, r3)  head / query / key ranks of the pre-softmax tensor
    t: tuple                  # (t1, t2, t3)  head / output / value ranks of the post-softmax tensor
    causal: bool
    rope: bool
    rope_base: float
    dtype: str                # "fp32" | "bf16"  (storage type; accumulation is fp32 on the GPU)
    seed: int
    shared_kv: bool = False   # one latent cache serves keys and values (Ut3 := U3); with rope it holds un-rotated rows

    def asdict(self):
        return asdict(self)


WORKLOADS = {
    w.name: w for w in [
        Workload("c1_tiny_fp32", "prefill", 1, 64, 128, 4, (2, 16, 16), (2, 16, 16),
                 True, False, 10000.0, "fp32", 1000),
        Workload("c2_gpt2_prefill", "prefill", 8, 1024, 768, 12, (12, 64, 64), (12, 64, 64),
                 True, True, 10000.0, "bf16", 1001),
        Workload("c3_vit_prefill", "prefill", 256, 197, 768, 12, (4, 96, 96), (4, 96, 96),
                 False, False, 10000.0, "bf16", 1002),
        Workload("c4_long_prefill", "prefill", 2, 8192, 4096, 32, (8, 128, 128), (8, 128, 128),
                 True, True, 500000.0, "bf16", 1003),
        Workload("c5_decode", "decode", 64, 32768, 4096, 32, (8, 128, 128), (8, 128, 128),
                 True, True, 500000.0, "bf16", 1004),
        # the decode shape with the paper's shared key / value down-projection (one latent cache, no RoPE)
        Workload("f1_decode_shared_kv", "decode", 64, 32768, 4096, 32, (8, 128, 128), (8, 128, 128),
                 True, False, 500000.0, "bf16", 1005, True),
        # the same with latent RoPE at position 32768: the one cache holds un-rotated rows, keys are rotated on chip
        Workload("f1r_decode_shared_kv_rope", "decode", 64, 32768, 4096, 32, (8, 128, 128), (8, 128, 128),
                 True, True, 500000.0, "bf16", 1006, True),
    ]
}


def get_workload(name: str) -> Workload:
    if name in WORKLOADS:
        return WORKLOADS[name]
    for k, w in WORKLOADS.items():          # allow "c4", "c2", ...
        if k.split("_")[0] == name:
            return w
    raise KeyError(f"unknown workload {name!r}; have {sorted(WORKLOADS)}")


def _rng(seed: int, *stream: int) -> np.random.Generator:
    """Independent PCG64 stream per tensor: (seed, stream...) -> generator."""
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *stream])))


def orthonormal_factor(rng: np.random.Generator, rows: int, rank: int) -> np.ndarray:
    """Q factor of the thin QR of a Gaussian [rows, rank] matrix, signs fixed so that
    diag(R) > 0 (makes the factor a deterministic function of the draw).  If rank > rows
    the first `rows` columns are orthonormal and the rest are a second, independent
    orthonormal block scaled to keep unit column norms as far as possible."""
    if rank <= rows:
        a = rng.standard_normal((rows, rank))
        q, r = np.linalg.qr(a)
        s = np.sign(np.diag(r))
        s[s == 0] = 1.0
        return q * s[None, :]
    blocks = []
    left = rank
    while left > 0:
        k = min(left, rows)
        blocks.append(orthonormal_factor(rng, rows, k))
        left -= k
    return np.concatenate(blocks, axis=1)


def make_weights(w: Workload, core_std: float | None = None, core_gain: float = 1.0) -> dict:
    """The two cores and six factor matrices (fp64).  Cores ~ N(0, var = 1/sqrt(r2*r3)),
    i.e. std = (r2*r3)**-0.25, unless `core_std` is given; `core_gain` multiplies the
    pre-softmax core only (a gain of 8 gives the "sharp softmax" stress variant)."""
    r1, r2, r3 = w.r
    t1, t2, t3 = w.t
    d, nH, s = w.d_model, w.n_H, w.seed
    std_c = core_std if core_std is not None else (r2 * r3) ** -0.25
    std_ct = core_std if core_std is not None else (t2 * t3) ** -0.25
    wts = {
        "U1": orthonormal_factor(_rng(s, 1), nH, r1),
        "U2": orthonormal_factor(_rng(s, 2), d, r2),
        "U3": orthonormal_factor(_rng(s, 3), d, r3),
        "C": _rng(s, 4).standard_normal((r1, r2, r3)) * (std_c * core_gain),
        "Ut1": orthonormal_factor(_rng(s, 5), nH, t1),
        "Ut2": orthonormal_factor(_rng(s, 6), d, t2),
        "Ut3": orthonormal_factor(_rng(s, 7), d, t3),
        "Ct": _rng(s, 8).standard_normal((t1, t2, t3)) * std_ct,
    }
    if getattr(w, "shared_kv", False):
        wts["Ut3"] = wts["U3"]          # shared key / value down-projection
    return wts


def make_X(w: Workload, B: int | None = None, N: int | None = None) -> np.ndarray:
    """X ~ N(0,1), float32 (so that the largest workload stays within host memory)."""
    B = w.B if B is None else B
    N = w.N if N is None else N
    return _rng(w.seed, 0).standard_normal((B, N, w.d_model), dtype=np.float32)


def make_decode_state(w: Workload, B: int | None = None, L: int | None = None,
                      Lmax: int | None = None, cache_len=None):
    """Decode-step inputs: new-token embeddings x [B, d_model] ~ N(0,1); latent caches
    Kc [B, Lmax, r3] and Vc [B, Lmax, t3] with entries ~ N(0,1) in the first cache_len[b]
    slots (the K cache is taken as already rotated) and zeros after; cache_len [B] int32.
    """
    B = w.B if B is None else B
    L = w.N if L is None else L
    Lmax = (L + 1) if Lmax is None else Lmax
    if cache_len is None:
        cache_len = np.full((B,), L, dtype=np.int32)
    cache_len = np.asarray(cache_len, dtype=np.int32)
    assert cache_len.shape == (B,) and int(cache_len.max(initial=0)) < Lmax
    x = _rng(w.seed, 10).standard_normal((B, w.d_model), dtype=np.float32)
    Kc = np.zeros((B, Lmax, w.r[2]), dtype=np.float32)
    Vc = np.zeros((B, Lmax, w.t[2]), dtype=np.float32)
    for b in range(B):
        n = int(cache_len[b])
        Kc[b, :n], Vc[b, :n] = decode_cache_rows(w, b, n)
    return x, Kc, Vc, cache_len


def decode_cache_rows(w: Workload, b: int, n: int):
    """The first n cached latent key / value rows of sequence b (float32, ~N(0,1)); every
    sequence has its own stream, so a large cache can be produced one sequence at a time."""
    k = _rng(w.seed, 11, b).standard_normal((n, w.r[2]), dtype=np.float32)
    v = _rng(w.seed, 12, b).standard_normal((n, w.t[2]), dtype=np.float32)
    return k, v


def make_decode_x(w: Workload, B: int | None = None) -> np.ndarray:
    """New-token embeddings x [B, d_model] ~ N(0,1) (same draw as make_decode_state)."""
    B = w.B if B is None else B
    return _rng(w.seed, 10).standard_normal((B, w.d_model), dtype=np.float32)


def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round an array to the workload's storage type and return it as float64, so that both
    sides start from bit-identical values: fp32 -> nearest float32; bf16 -> nearest-even
    bfloat16 (done on the float32 bit pattern; inputs here are finite)."""
    a32 = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "fp32":
        return a32.astype(np.float64)
    if dtype != "bf16":
        raise ValueError(dtype)
    u = a32.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a32.shape).astype(np.float64)


# ----------------------------------------------------------------------------------------
# Work counts (latent-dimension FLOP count; bytes that must move for decode)
# ----------------------------------------------------------------------------------------

def prefill_flops(w: Workload, B: int | None = None, N: int | None = None) -> dict:
    """FLOPs of one prefill forward, counted on the latent dimensions actually contracted:
    projections, head-mode core contraction, per-head queries, scores, PV, output side.
    Causal attention counts N(N+1)/2 (query, key) pairs."""
    B = w.B if B is None else B
    N = w.N if N is None else N
    r1, r2, r3 = w.r
    t1, t2, t3 = w.t
    d, nH = w.d_model, w.n_H
    T = B * N
    pairs = N * (N + 1) // 2 if w.causal else N * N
    f = {
        "proj": 2 * T * d * (r2 + r3 + t3),
        "core": 2 * nH * (r1 * r2 * r3 + t1 * t2 * t3),
        "qhat": 2 * T * nH * r2 * r3,
        "scores": 2 * B * nH * pairs * r3,
        "pv": 2 * B * nH * pairs * t3,
        "z": 2 * T * nH * t3 * t2,
        "y": 2 * T * t2 * d,
    }
    f["total"] = sum(f.values())
    return f


def decode_bytes(w: Workload, B: int | None = None, L: int | None = None) -> dict:
    """Bytes one decode step has to move at the storage width: the latent caches read once,
    the weights, x and y, and the appended key/value rows."""
    B = w.B if B is None else B
    L = w.N if L is None else L
    r1, r2, r3 = w.r
    t1, t2, t3 = w.t
    d, nH = w.d_model, w.n_H
    e = 2 if w.dtype == "bf16" else 4
    shared = getattr(w, "shared_kv", False)
    by = {
        "cache": B * L * (r3 if shared else r3 + t3) * e,
        "weights": (r1 * r2 * r3 + t1 * t2 * t3 + nH * (r1 + t1) + d * (r2 + r3 + t2 + (0 if shared else t3))) * e,
        "xy": 2 * B * d * e,
        "append": B * (r3 if shared else r3 + t3) * e,
    }
    by["total"] = sum(by.values())
    return by


def decode_flops(w: Workload, B: int | None = None, L: int | None = None) -> int:
    B = w.B if B is None else B
    L = w.N if L is None else L
    r1, r2, r3 = w.r
    t1, t2, t3 = w.t
    d, nH = w.d_model, w.n_H
    attn = 2 * B * nH * (L + 1) * (r3 + t3)
    other = 2 * B * d * (r2 + r3 + t3) + 2 * B * nH * (r2 * r3 + t3 * t2) + 2 * B * t2 * d \
        + 2 * nH * (r1 * r2 * r3 + t1 * t2 * t3)
    return attn + other


def make_lowrank_mha(d: int, n_H: int, rank: int, noise: float, seed: int) -> dict:
    """Synthetic MHA weights WQ, WK, WV, WO [d, d] whose per-head products have a dominant shared rank-`rank`
    structure plus Gaussian noise of relative size `noise` (stand-in for pretrained weights, whose spectra decay;
    input of the HOSVD initialiser).  Every head's query / key / value columns are mixtures of `rank` common
    directions, so the three unfoldings of the weight tensors have `rank` (modes 2, 3) large singular values."""
    out = {}
    for idx, name in enumerate(("WQ", "WK", "WV", "WO")):
        rng = _rng(seed, 20 + idx)
        basis = orthonormal_factor(rng, d, rank)                       # common directions
        mix = rng.standard_normal((rank, d)) / np.sqrt(rank)
        Wm = basis @ mix if name != "WO" else (basis @ mix).T
        out[name] = Wm + noise * rng.standard_normal((d, d)) / np.sqrt(d)
    return out

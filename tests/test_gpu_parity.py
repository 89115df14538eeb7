"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle on the same
seeded inputs, element by element on small cases and on sampled query rows / sequences at
the full benchmark sizes.  Bounds: bf16 storage max-abs <= 2e-2 and mean-abs <= 2e-3; fp32
max-abs <= 1e-4."""
import numpy as np
import pytest

from oracle import tucker_oracle as O
from paper_2603_30033_b200 import binding as Bd
from paper_2603_30033_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def oracle_fwd(X, wt, w, rows=None, pos0=0, scale=None):
    return O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=w.causal, rope=w.rope,
                             rope_base=w.rope_base, pos0=pos0, rows=rows, scale=scale)


def gpu_fwd(X, wt, w, flags=0, pos0=0, caches=None, scale=0.0):
    dw = H.weights_to_device(wt, w.dtype)
    Xd = H.to_device(X, w.dtype)
    kw = {}
    if caches is not None:
        kw = dict(Kcache=caches[0], Vcache=caches[1])
    Y = Bd.tucker_attn_fwd(Xd, *dw, n_H=w.n_H, causal=w.causal, rope=w.rope, rope_base=w.rope_base, pos0=pos0,
                           flags=flags, scale=scale, **kw)
    assert Bd.last_device_error() == 0
    return Y.float().cpu().numpy().astype(np.float64)


check = H.check


# --------------------------------------------------------------------------------------
# config 1: tiny fp32 layer, plus weights that make Tucker attention equal MHA / GQA exactly
# --------------------------------------------------------------------------------------

def test_c1_tiny_fp32():
    w = W.get_workload("c1")
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w)
    check(got, oracle_fwd(X, wt, w), "fp32", "c1")
    assert Bd.last_path() == 1


@pytest.mark.parametrize("n_G", [4, 2, 1])
def test_c1_mha_gqa_exact_weights(n_G):
    # ranks (4,128,128) reproduce MHA, (4,128,n_G*32) reproduce GQA / MQA
    w = W.get_workload("c1")
    rng = np.random.default_rng(100 + n_G)
    d, n_H, d_H = w.d_model, w.n_H, w.d_model // w.n_H
    f32 = lambda a: a.astype(np.float32).astype(np.float64)
    WQ, WO = (f32(rng.standard_normal((d, d)) / np.sqrt(d)) for _ in range(2))
    WKg, WVg = (f32(rng.standard_normal((d, n_G * d_H)) / np.sqrt(d)) for _ in range(2))
    X = f32(rng.standard_normal((1, w.N, d)))
    wt = O.tucker_from_gqa(WQ, WKg, WVg, WO, n_H, n_G)
    ref = O.gqa_reference(X[0], WQ, WKg, WVg, WO, n_H, n_G, causal=True)
    got = gpu_fwd(X, wt, w)[0]
    check(got, ref, "fp32", f"gqa n_G={n_G}")


# --------------------------------------------------------------------------------------
# small shapes, both storage types, ragged sizes, flags
# --------------------------------------------------------------------------------------

SMALL = [
    dict(B=2, N=37, d_model=48, n_H=3, r=(2, 10, 12), t=(3, 9, 7), causal=True, rope=True),
    dict(B=1, N=130, d_model=64, n_H=4, r=(4, 16, 32), t=(2, 24, 16), causal=False, rope=False),
    dict(B=3, N=1, d_model=32, n_H=2, r=(1, 4, 6), t=(1, 5, 3), causal=True, rope=True),
    dict(B=2, N=65, d_model=96, n_H=6, r=(3, 20, 18), t=(6, 33, 40), causal=True, rope=False),
]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", SMALL)
def test_small_shapes_generic(shape, dtype):
    w = H.custom_workload(dtype=dtype, rope_base=10000.0, seed=31, **shape)
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w, flags=Bd.TA_FLAG_FORCE_GENERIC, pos0=5)
    check(got, oracle_fwd(X, wt, w, pos0=5), dtype, str(shape))


# `scaled=True` marks the stress shapes whose outputs are several times larger than the benchmark workloads'
# (rms 0.45 .. 1.5 against <= 0.16) and whose raw bf16 errors exceed the absolute 2e-2 / 2e-3; every other shape is
# held to the absolute bounds.
FAST = [
    dict(B=2, N=200, d_model=128, n_H=4, r=(4, 64, 64), t=(4, 64, 64), causal=True, rope=True, scaled=True),
    dict(B=1, N=333, d_model=192, n_H=6, r=(3, 96, 64), t=(2, 32, 128), causal=False, rope=False),
    dict(B=3, N=128, d_model=256, n_H=8, r=(8, 128, 128), t=(8, 128, 128), causal=True, rope=True, scaled=True),
    dict(B=2, N=77, d_model=64, n_H=2, r=(2, 32, 32), t=(2, 96, 96), causal=True, rope=False, scaled=True),
    dict(B=1, N=1, d_model=64, n_H=2, r=(2, 64, 64), t=(2, 64, 64), causal=True, rope=True, scaled=True),
    # query rank above 128: per-head queries come from the separate GEMM, not the attention prologue
    dict(B=2, N=150, d_model=256, n_H=4, r=(4, 256, 64), t=(4, 64, 64), causal=True, rope=True),
    # no mask: one CTA walks several head pairs; odd head count ends on a single head
    dict(B=2, N=197, d_model=192, n_H=3, r=(3, 64, 96), t=(3, 96, 96), causal=False, rope=True),
    dict(B=3, N=260, d_model=384, n_H=12, r=(4, 96, 96), t=(4, 96, 96), causal=False, rope=False),
    # odd head count with a mask (the last pair has one head), mixed ranks, a single 64-row tile
    dict(B=2, N=300, d_model=320, n_H=5, r=(5, 64, 64), t=(5, 32, 64), causal=True, rope=True),
    dict(B=2, N=150, d_model=256, n_H=4, r=(2, 128, 64), t=(2, 64, 96), causal=False, rope=True),
    dict(B=1, N=64, d_model=192, n_H=6, r=(3, 96, 96), t=(3, 96, 96), causal=True, rope=True),
    # wide model: the projection GEMM reads K-major copies of the factors
    dict(B=1, N=150, d_model=2048, n_H=16, r=(4, 64, 96), t=(4, 64, 32), causal=True, rope=True),
]


@pytest.mark.parametrize("shape", FAST)
def test_small_shapes_tensor_core_path(shape):
    shape = dict(shape)
    scaled = shape.pop("scaled", False)
    w = H.custom_workload(dtype="bf16", rope_base=10000.0, seed=77, **shape)
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w, pos0=3)
    assert Bd.last_path() == 2
    check(got, oracle_fwd(X, wt, w, pos0=3), "bf16", str(shape), scaled=scaled)


def _random_shapes(seed, count):
    import random
    rng = random.Random(seed)
    out = []
    for _ in range(count):
        nH = rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 12])
        ranks = [rng.choice([32, 64, 96, 128]) for _ in range(4)]
        out.append(dict(B=rng.choice([1, 2, 3]), N=rng.choice([1, 17, 64, 127, 128, 129, 200, 255, 256, 257, 384, 400, 520, 777]),
                        d_model=nH * 64, n_H=nH, r=(min(nH, rng.choice([1, 2, 4])), ranks[0], ranks[1]),
                        t=(min(nH, rng.choice([1, 2, 3])), ranks[2], ranks[3]), causal=rng.choice([True, False]),
                        rope=rng.choice([True, False])))
    return out


@pytest.mark.parametrize("shape", _random_shapes(5, 32), ids=lambda s: "B%dN%dH%d" % (s["B"], s["N"], s["n_H"]))
def test_random_shapes_tensor_core_path(shape):
    # seeded random mixes of head counts (odd ones end on a single head), ranks, lengths around the tile edges,
    # masks and RoPE: every role of the attention kernel's pipeline has to keep its barrier phases in step
    w = H.custom_workload(dtype="bf16", rope_base=10000.0, seed=300 + shape["N"] + shape["n_H"], **shape)
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w)
    assert Bd.last_path() == 2 and Bd.last_device_error() == 0
    # a single token has no averaging over keys: its error is judged relative to the output's size
    check(got, oracle_fwd(X, wt, w), "bf16", str(shape), scaled=shape["N"] == 1)


def test_fused_and_unfused_query_paths_agree():
    # the attention kernel forming Qhat in its prologue vs reading it from the query GEMM
    w = H.custom_workload(dtype="bf16", B=2, N=300, d_model=256, n_H=8, r=(3, 128, 128), t=(3, 64, 128), causal=True,
                          rope=True, rope_base=500000.0, seed=91)
    X, wt = H.host_inputs(w)
    ref = oracle_fwd(X, wt, w, pos0=1000)
    for flags in (0, Bd.TA_FLAG_SEPARATE_QUERIES, Bd.TA_FLAG_FMA_ATTENTION, Bd.TA_FLAG_SEPARATE_OUTPUT_GEMMS):
        got = gpu_fwd(X, wt, w, flags=flags, pos0=1000)
        assert Bd.last_path() == 2
        check(got, ref, "bf16", f"flags={flags}")


def test_results_are_bit_repeatable():
    # no atomics anywhere on the path: repeated calls must give identical bits (a cheap race detector)
    import torch
    for shape in (dict(B=2, N=333, d_model=384, n_H=6, r=(3, 64, 64), t=(3, 64, 64), causal=True, rope=True),
                  dict(B=2, N=200, d_model=256, n_H=8, r=(4, 128, 128), t=(4, 128, 128), causal=True, rope=True),
                  dict(B=4, N=197, d_model=384, n_H=12, r=(4, 96, 96), t=(4, 96, 96), causal=False, rope=False)):
        w = H.custom_workload(dtype="bf16", rope_base=10000.0, seed=95, **shape)
        X, wt = H.host_inputs(w)
        dw = H.weights_to_device(wt, w.dtype)
        Xd = H.to_device(X, w.dtype)
        first = None
        for it in range(12):
            if it % 3 == 1:     # disturb caches / timing between calls
                a = torch.randn(2048, 2048, device="cuda", dtype=torch.bfloat16)
                (a @ a).sum().item()
            Y = Bd.tucker_attn_fwd(Xd, *dw, n_H=w.n_H, causal=w.causal, rope=w.rope, rope_base=w.rope_base)
            assert Bd.last_device_error() == 0
            if first is None:
                first = Y.clone()
            else:
                assert torch.equal(Y, first), f"call {it} differs from call 0 for {shape}"


def test_tensor_core_path_writes_cache():
    import torch
    w = H.custom_workload(dtype="bf16", B=2, N=150, d_model=128, n_H=4, r=(2, 64, 64), t=(2, 64, 32), rope=True, seed=5)
    X, wt = H.host_inputs(w)
    Lmax = 160
    Kc = torch.full((2, Lmax, 64), 7.0, device="cuda", dtype=torch.bfloat16)
    Vc = torch.full((2, Lmax, 32), 7.0, device="cuda", dtype=torch.bfloat16)
    gpu_fwd(X, wt, w, caches=(Kc, Vc))
    assert Bd.last_path() == 2
    _, parts = O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=True, rope=True, return_parts=True)
    for b in range(2):
        assert np.abs(Kc[b, :150].float().cpu().numpy() - parts[b]["K"]).max() < 3e-2
        assert np.abs(Vc[b, :150].float().cpu().numpy() - parts[b]["V"]).max() < 3e-2
    assert (Kc[:, 150:] == 7.0).all() and (Vc[:, 150:] == 7.0).all()


def test_prefill_writes_cache():
    import torch
    w = H.custom_workload(dtype="fp32", B=2, N=21, d_model=32, n_H=4, r=(2, 8, 10), t=(2, 8, 6), rope=True, seed=3)
    X, wt = H.host_inputs(w)
    Lmax = 30
    Kc = torch.full((2, Lmax, 10), 7.0, device="cuda")
    Vc = torch.full((2, Lmax, 6), 7.0, device="cuda")
    gpu_fwd(X, wt, w, caches=(Kc, Vc))
    _, parts = O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=True, rope=True, return_parts=True)
    for b in range(2):
        np.testing.assert_allclose(Kc[b, :21].cpu().numpy(), parts[b]["K"], atol=1e-5)
        np.testing.assert_allclose(Vc[b, :21].cpu().numpy(), parts[b]["V"], atol=1e-5)
    assert (Kc[:, 21:] == 7.0).all() and (Vc[:, 21:] == 7.0).all()


def test_custom_scale_and_invariants():
    # scale override; permutation equivariance without mask; causal prefix independence
    w = H.custom_workload(dtype="fp32", B=1, N=40, d_model=32, n_H=4, r=(2, 8, 8), t=(2, 8, 8), causal=False, seed=9)
    X, wt = H.host_inputs(w)
    check(gpu_fwd(X, wt, w, scale=0.3), oracle_fwd(X, wt, w, scale=0.3), "fp32", "scale")
    perm = np.random.default_rng(0).permutation(40)
    a, b = gpu_fwd(X, wt, w), gpu_fwd(X[:, perm], wt, w)
    assert np.abs(a[:, perm] - b).max() < 1e-5
    wc = H.with_(w, causal=True, rope=True)
    X2 = X.copy()
    X2[:, 25:] = 0.5
    a, b = gpu_fwd(X, wt, wc), gpu_fwd(X2, wt, wc)
    assert np.abs(a[:, :25] - b[:, :25]).max() == 0.0
    # position-offset invariance of latent RoPE
    c = gpu_fwd(X, wt, wc, pos0=4096)
    assert np.abs(a - c).max() < 2e-4


# --------------------------------------------------------------------------------------
# decode
# --------------------------------------------------------------------------------------

def run_decode(w, B, lens, Lmax, flags=0, append=True):
    import torch
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    x, Kc, Vc, cache_len = W.make_decode_state(w, B=B, L=max(lens), Lmax=Lmax, cache_len=lens)
    x, Kc, Vc = (W.round_to_storage(a, w.dtype) for a in (x, Kc, Vc))
    ref_y, ref_k, ref_v = O.tucker_attn_decode(x, *[wt[k] for k in H.WEIGHT_KEYS], Kc, Vc, cache_len, rope=w.rope,
                                               rope_base=w.rope_base)
    dw = H.weights_to_device(wt, w.dtype)
    Kd, Vd, xd = H.to_device(Kc, w.dtype), H.to_device(Vc, w.dtype), H.to_device(x, w.dtype)
    ld = torch.from_numpy(cache_len).cuda()
    y = Bd.tucker_attn_decode(xd, *dw, Kd, Vd, ld, n_H=w.n_H, rope=w.rope, rope_base=w.rope_base, append=append,
                              flags=flags)
    assert Bd.last_device_error() == 0
    y = y.float().cpu().numpy().astype(np.float64)
    return y, ref_y, (Kd, Vd, Kc, Vc, ref_k, ref_v, cache_len)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_decode_small_generic(dtype):
    w = H.custom_workload(kind="decode", dtype=dtype, d_model=64, n_H=4, r=(2, 16, 12), t=(2, 10, 20), rope=True, seed=17)
    lens = [0, 1, 31, 32, 33, 100]
    y, ref, (Kd, Vd, Kc, Vc, ref_k, ref_v, cl) = run_decode(w, 6, lens, 128, flags=Bd.TA_FLAG_FORCE_GENERIC)
    check(y, ref, dtype, "decode small")
    tol = 1e-5 if dtype == "fp32" else 2e-2
    Kh, Vh = Kd.float().cpu().numpy(), Vd.float().cpu().numpy()
    for b, L in enumerate(lens):
        assert np.abs(Kh[b, L] - ref_k[b]).max() < tol and np.abs(Vh[b, L] - ref_v[b]).max() < tol
        assert np.array_equal(Kh[b, :L], Kc[b, :L].astype(np.float32))        # old slots untouched
        assert np.array_equal(Kh[b, L + 1:], Kc[b, L + 1:].astype(np.float32))


DEC_FAST = [
    dict(d_model=256, n_H=4, r=(2, 64, 64), t=(2, 64, 64), lens=[0, 1, 127, 128, 129, 300, 1000], Lmax=1024),
    dict(d_model=256, n_H=32, r=(8, 128, 128), t=(8, 128, 128), lens=[511, 5, 2047, 256, 255], Lmax=2048),
    dict(d_model=192, n_H=12, r=(4, 96, 96), t=(4, 32, 96), lens=[700, 33], Lmax=777),
    dict(d_model=128, n_H=2, r=(2, 32, 128), t=(2, 64, 64), lens=[100] * 3 + [4000] + [0] * 200, Lmax=4001, scaled=True),
    dict(d_model=128, n_H=8, r=(2, 64, 64), t=(2, 32, 128), lens=[50000], Lmax=50001),
]


@pytest.mark.parametrize("append", [True, False])
@pytest.mark.parametrize("case", DEC_FAST)
def test_decode_tensor_core_path(case, append):
    case = dict(case)
    lens, Lmax, scaled = case.pop("lens"), case.pop("Lmax"), case.pop("scaled", False)
    w = H.custom_workload(kind="decode", dtype="bf16", rope=True, rope_base=500000.0, seed=23, **case)
    y, ref, (Kd, Vd, Kc, Vc, ref_k, ref_v, cl) = run_decode(w, len(lens), lens, Lmax, append=append)
    assert Bd.last_path() == 2
    check(y, ref, "bf16", f"decode {case}", scaled=scaled)
    Kh, Vh = Kd.float().cpu().numpy(), Vd.float().cpu().numpy()
    for b, L in enumerate(lens[:8]):
        if append:
            assert np.abs(Kh[b, L] - ref_k[b]).max() < 3e-2 and np.abs(Vh[b, L] - ref_v[b]).max() < 3e-2
            Kh[b, L], Vh[b, L] = Kc[b, L], Vc[b, L]
        assert np.array_equal(Kh[b], Kc[b].astype(np.float32)) and np.array_equal(Vh[b], Vc[b].astype(np.float32))


def test_decode_growing_scores_exercise_the_rescaling():
    # Cached keys whose norm grows along the sequence and a pre-softmax core scaled by 8: the running maximum
    # of most heads rises by far more than the lazy-rescale threshold from tile to tile, so the accumulated
    # outputs and row sums are rescaled again and again (the random caches of the other tests almost never
    # move the maximum after the first tile).
    import torch
    w = H.custom_workload(kind="decode", dtype="bf16", d_model=256, n_H=32, r=(8, 64, 128), t=(8, 64, 128), rope=True,
                          rope_base=500000.0, seed=29)
    lens, Lmax = [1500, 700, 129, 2047], 2048
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    wt["C"] = W.round_to_storage(wt["C"] * 8.0, w.dtype)
    x, Kc, Vc, cache_len = W.make_decode_state(w, B=len(lens), L=max(lens), Lmax=Lmax, cache_len=lens)
    ramp = (1.0 + 3.0 * np.arange(Lmax) / Lmax).astype(np.float32)[None, :, None]
    x, Kc, Vc = (W.round_to_storage(a, w.dtype) for a in (x, Kc * ramp, Vc))
    ref, _, _ = O.tucker_attn_decode(x, *[wt[k] for k in H.WEIGHT_KEYS], Kc, Vc, cache_len, rope=True,
                                     rope_base=w.rope_base)
    y = Bd.tucker_attn_decode(H.to_device(x, w.dtype), *H.weights_to_device(wt, w.dtype), H.to_device(Kc, w.dtype),
                              H.to_device(Vc, w.dtype), torch.from_numpy(cache_len).cuda(), n_H=w.n_H, rope=True,
                              rope_base=w.rope_base, append=True)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    check(y.float().cpu().numpy().astype(np.float64), ref, "bf16", "decode, growing scores", scaled=True)


# --------------------------------------------------------------------------------------
# shared key / value projection and cache (Sec. 3.1: K, V replaced by L^KV = X U3), no RoPE
# --------------------------------------------------------------------------------------

def _shared_weights(w):
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    wt["Ut3"] = wt["U3"]
    return wt


@pytest.mark.parametrize("dtype,shape,path", [
    ("bf16", dict(d_model=256, n_H=8, r=(4, 64, 128), t=(4, 64, 128)), 2),
    ("bf16", dict(d_model=192, n_H=6, r=(3, 96, 64), t=(2, 32, 64)), 2),
    ("fp32", dict(d_model=64, n_H=4, r=(2, 16, 12), t=(2, 10, 12)), 1),
])
def test_decode_shared_latent_cache(dtype, shape, path):
    import torch
    w = H.custom_workload(kind="decode", dtype=dtype, rope=False, seed=61, **shape)
    wt = _shared_weights(w)
    lens = [0, 1, 127, 128, 300, 650]
    Lmax = 700
    x, Kc, _, cache_len = W.make_decode_state(w, B=len(lens), L=max(lens), Lmax=Lmax, cache_len=lens)
    x, Kc = (W.round_to_storage(a, dtype) for a in (x, Kc))
    ref, ref_k, ref_v = O.tucker_attn_decode(x, *[wt[k] for k in H.WEIGHT_KEYS], Kc, Kc, cache_len, rope=False)
    np.testing.assert_allclose(ref_k, ref_v)            # one row serves as key and value
    dw = H.weights_to_device(wt, dtype)
    dw[7] = dw[3]                                        # the same device tensor for U3 and Ut3
    Kd = H.to_device(Kc, dtype)
    y = Bd.tucker_attn_decode(H.to_device(x, dtype), *dw, Kd, Kd, torch.from_numpy(cache_len).cuda(), n_H=w.n_H,
                              rope=False, append=True)
    assert Bd.last_device_error() == 0 and Bd.last_path() == path
    check(y.float().cpu().numpy().astype(np.float64), ref, dtype, f"shared decode {shape}")
    Kh = Kd.float().cpu().numpy()
    tol = 1e-5 if dtype == "fp32" else 3e-2
    for b, L in enumerate(lens):
        assert np.abs(Kh[b, L] - ref_k[b]).max() < tol
        assert np.array_equal(Kh[b, :L], Kc[b, :L].astype(np.float32))


@pytest.mark.parametrize("d_model", [256, 2048])
def test_prefill_shared_projection_and_cache(d_model):
    import torch
    w = H.custom_workload(dtype="bf16", B=2, N=200, d_model=d_model, n_H=8, r=(4, 64, 128), t=(4, 64, 128), causal=True,
                          rope=False, seed=63)
    wt = _shared_weights(w)
    X = W.round_to_storage(W.make_X(w), w.dtype)
    ref, parts = O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=True, rope=False, return_parts=True)
    dw = H.weights_to_device(wt, w.dtype)
    dw[7] = dw[3]
    cache = torch.full((2, 210, 128), 7.0, device="cuda", dtype=torch.bfloat16)
    Y = Bd.tucker_attn_fwd(H.to_device(X, w.dtype), *dw, n_H=w.n_H, causal=True, rope=False, Kcache=cache, Vcache=cache)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    check(Y.float().cpu().numpy().astype(np.float64), ref, "bf16", "shared prefill")
    for b in range(2):
        assert np.abs(cache[b, :200].float().cpu().numpy() - parts[b]["K"]).max() < 3e-2
    assert (cache[:, 200:] == 7.0).all()


def test_aliased_caches_need_shared_weights():
    import torch
    w = H.custom_workload(kind="decode", dtype="bf16", d_model=256, n_H=8, r=(4, 64, 64), t=(4, 64, 64), rope=True, seed=65)
    wt = _shared_weights(w)
    Kd = torch.zeros(2, 16, 64, device="cuda", dtype=torch.bfloat16)
    x = torch.zeros(2, 256, device="cuda", dtype=torch.bfloat16)
    ld = torch.zeros(2, dtype=torch.int32, device="cuda")
    dw2 = H.weights_to_device(wt, "bf16")             # distinct U3 / Ut3 tensors: not a shared projection
    for rope in (False, True):
        with pytest.raises(Bd.TuckerAttnError) as e:
            Bd.tucker_attn_decode(x, *dw2, Kd, Kd, ld, n_H=8, rope=rope)
        assert e.value.status == -1


# --------------------------------------------------------------------------------------
# shared latent cache WITH latent RoPE (Sec. 3.1 + Definition 2): the one cache holds un-rotated rows
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,shape,path", [
    ("bf16", dict(d_model=256, n_H=8, r=(4, 64, 128), t=(4, 64, 128)), 2),
    ("bf16", dict(d_model=256, n_H=32, r=(8, 128, 64), t=(8, 32, 64)), 2),
    ("bf16", dict(d_model=192, n_H=6, r=(3, 96, 96), t=(2, 32, 96)), 2),
    ("fp32", dict(d_model=64, n_H=4, r=(2, 16, 12), t=(2, 10, 12)), 1),
])
@pytest.mark.parametrize("append", [True, False])
def test_decode_shared_latent_cache_with_rope(dtype, shape, path, append):
    import torch
    w = H.custom_workload(kind="decode", dtype=dtype, rope=True, rope_base=500000.0, seed=67, **shape)
    wt = _shared_weights(w)
    lens = [0, 1, 127, 128, 129, 300, 650, 1023]
    Lmax = 1024
    x, Lc, _, cache_len = W.make_decode_state(w, B=len(lens), L=max(lens), Lmax=Lmax, cache_len=lens)
    x, Lc = (W.round_to_storage(a, dtype) for a in (x, Lc))
    ref, l_new = O.tucker_attn_decode_shared_rope(x, wt["C"], wt["U1"], wt["U2"], wt["U3"], wt["Ct"], wt["Ut1"], wt["Ut2"],
                                                  Lc, cache_len, rope_base=w.rope_base)
    dw = H.weights_to_device(wt, dtype)
    dw[7] = dw[3]                                        # the same device tensor for U3 and Ut3
    Ld = H.to_device(Lc, dtype)
    for b, L in enumerate(lens):                         # slots from cache_len on are never trusted
        Ld[b, L:] = float("nan")
    y = Bd.tucker_attn_decode(H.to_device(x, dtype), *dw, Ld, Ld, torch.from_numpy(cache_len).cuda(), n_H=w.n_H,
                              rope=True, rope_base=w.rope_base, append=append)
    assert Bd.last_device_error() == 0 and Bd.last_path() == path
    check(y.float().cpu().numpy().astype(np.float64), ref, dtype, f"shared cache + RoPE decode {shape}", scaled=True)
    Lh = Ld.float().cpu().numpy()
    tol = 1e-5 if dtype == "fp32" else 3e-2
    for b, L in enumerate(lens):
        if append:
            assert np.abs(Lh[b, L] - l_new[b]).max() < tol          # the UN-rotated latent row was appended
        else:
            assert np.isnan(Lh[b, L]).all()
        assert np.array_equal(Lh[b, :L], Lc[b, :L].astype(np.float32))


@pytest.mark.parametrize("dtype,shape,path", [
    ("bf16", dict(d_model=256, n_H=8, r=(4, 64, 128), t=(4, 64, 128)), 2),
    ("fp32", dict(d_model=64, n_H=4, r=(2, 16, 12), t=(2, 10, 12)), 1),
])
def test_prefill_then_decode_with_one_unrotated_cache(dtype, shape, path):
    # prefill of N tokens writes ONE cache of un-rotated latent rows; a decode step for token N on that cache
    # equals row N of the prefill over N + 1 tokens
    import torch
    N = 200
    w = H.custom_workload(dtype=dtype, B=2, N=N + 1, causal=True, rope=True, rope_base=10000.0, seed=69, **shape)
    wt = _shared_weights(w)
    X = W.round_to_storage(W.make_X(w), dtype)
    ref, parts = O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=True, rope=True, rope_base=w.rope_base,
                                   return_parts=True)
    dw = H.weights_to_device(wt, dtype)
    dw[7] = dw[3]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    cache = torch.full((2, N + 9, shape["r"][2]), 7.0, device="cuda", dtype=tdt)
    Y = Bd.tucker_attn_fwd(H.to_device(X[:, :N], dtype), *dw, n_H=w.n_H, causal=True, rope=True, rope_base=w.rope_base,
                           Kcache=cache, Vcache=cache)
    assert Bd.last_device_error() == 0 and Bd.last_path() == path
    check(Y.float().cpu().numpy().astype(np.float64), ref[:, :N], dtype, f"shared projection + RoPE prefill {shape}",
          scaled=True)
    tol = 1e-5 if dtype == "fp32" else 3e-2
    for b in range(2):
        assert np.abs(cache[b, :N].float().cpu().numpy() - parts[b]["V"][:N]).max() < tol     # un-rotated rows
    assert (cache[:, N:] == 7.0).all()
    lens = torch.full((2,), N, dtype=torch.int32, device="cuda")
    y = Bd.tucker_attn_decode(H.to_device(X[:, N], dtype), *dw, cache, cache, lens, n_H=w.n_H, rope=True,
                              rope_base=w.rope_base, append=True)
    assert Bd.last_device_error() == 0 and Bd.last_path() == path
    check(y.float().cpu().numpy().astype(np.float64), ref[:, N], dtype, f"decode after that prefill {shape}", scaled=True)


@pytest.mark.parametrize("N", [200, 197])
def test_prefill_with_one_shared_cache_without_rope(N):
    # U3 == Ut3, no RoPE, one cache for keys and values: the projection has two segments, and the key segment is
    # also the value tile of the attention kernel (written transposed, in 16-byte pieces when N is a multiple of 8)
    import torch
    shape = dict(d_model=256, n_H=8, r=(4, 64, 128), t=(4, 64, 128))
    w = H.custom_workload(dtype="bf16", B=2, N=N, causal=True, rope=False, seed=71, **shape)
    wt = _shared_weights(w)
    X = W.round_to_storage(W.make_X(w), "bf16")
    ref, parts = O.tucker_attn_fwd(X, *[wt[k] for k in H.WEIGHT_KEYS], causal=True, rope=False, return_parts=True)
    dw = H.weights_to_device(wt, "bf16")
    dw[7] = dw[3]
    cache = torch.full((2, N + 5, 128), 7.0, device="cuda", dtype=torch.bfloat16)
    Y = Bd.tucker_attn_fwd(H.to_device(X, "bf16"), *dw, n_H=w.n_H, causal=True, rope=False, Kcache=cache, Vcache=cache)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    check(Y.float().cpu().numpy().astype(np.float64), ref, "bf16", f"shared projection prefill N={N}", scaled=True)
    for b in range(2):
        assert np.abs(cache[b, :N].float().cpu().numpy() - parts[b]["V"][:N]).max() < 3e-2
    assert (cache[:, N:] == 7.0).all()


def test_decode_garbage_beyond_cache_len_is_ignored():
    # slots at and after cache_len hold NaN / Inf bit patterns: they must not leak into the result
    import torch
    w = H.custom_workload(kind="decode", dtype="bf16", d_model=256, n_H=4, r=(2, 64, 64), t=(2, 64, 64), rope=True, seed=29)
    lens = [5, 130, 255]
    Lmax = 300
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    x, Kc, Vc, cache_len = W.make_decode_state(w, B=3, L=max(lens), Lmax=Lmax, cache_len=lens)
    x, Kc, Vc = (W.round_to_storage(a, w.dtype) for a in (x, Kc, Vc))
    ref, _, _ = O.tucker_attn_decode(x, *[wt[k] for k in H.WEIGHT_KEYS], Kc, Vc, cache_len, rope=True, rope_base=w.rope_base)
    Kd, Vd = H.to_device(Kc, "bf16"), H.to_device(Vc, "bf16")
    for b, L in enumerate(lens):
        Kd[b, L:] = float("nan")
        Vd[b, L:] = float("inf")
    y = Bd.tucker_attn_decode(H.to_device(x, "bf16"), *H.weights_to_device(wt, "bf16"), Kd, Vd,
                              torch.from_numpy(cache_len).cuda(), n_H=4, rope=True, rope_base=w.rope_base, append=False)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    check(y.float().cpu().numpy().astype(np.float64), ref, "bf16", "garbage tail")


def test_calls_replay_from_a_cuda_graph():
    # Neither entry point synchronises, allocates or reads device memory on the host, so a call can be captured
    # into a CUDA graph (its launches keep their programmatic-dependent-launch edges) and replayed on new contents
    # of the same buffers; the replays must give the direct calls' bits.
    import torch
    w = H.custom_workload(kind="decode", dtype="bf16", d_model=256, n_H=8, r=(4, 64, 64), t=(4, 64, 64), rope=True,
                          rope_base=500000.0, seed=43)
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    dw = H.weights_to_device(wt, "bf16")
    lens = [100, 300, 7, 511]
    x, Kc, Vc, cl = W.make_decode_state(w, B=4, L=max(lens), Lmax=1024, cache_len=lens)
    xd, Kd, Vd = (H.to_device(W.round_to_storage(a, "bf16"), "bf16") for a in (x, Kc, Vc))
    ld = torch.from_numpy(cl).cuda()
    desc = Bd.make_desc(B=4, N=1, d_model=256, n_H=8, r=w.r, t=w.t, causal=True, rope=True, rope_base=w.rope_base)
    ws = Bd.alloc_workspace(Bd.decode_workspace_bytes(desc, 1024), xd.device)
    y = torch.empty_like(xd)
    dkw = dict(n_H=8, rope=True, rope_base=w.rope_base, append=False, out=y, workspace=ws)
    Xp = H.to_device(W.round_to_storage(W.make_X(H.with_(w, kind="prefill"), B=2, N=200), "bf16"), "bf16")
    pdesc = Bd.make_desc(B=2, N=200, d_model=256, n_H=8, r=w.r, t=w.t, causal=True, rope=True, rope_base=w.rope_base)
    pws = Bd.alloc_workspace(Bd.fwd_workspace_bytes(pdesc), xd.device)
    Y = torch.empty_like(Xp)
    pkw = dict(n_H=8, causal=True, rope=True, rope_base=w.rope_base, out=Y, workspace=pws)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        Bd.tucker_attn_decode(xd, *dw, Kd, Vd, ld, **dkw)          # warm-up outside the capture (kernel attributes)
        Bd.tucker_attn_fwd(Xp, *dw, **pkw)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            Bd.tucker_attn_decode(xd, *dw, Kd, Vd, ld, **dkw)
            Bd.tucker_attn_fwd(Xp, *dw, **pkw)
    for trial in range(2):
        xd.copy_(torch.randn_like(xd))                               # new contents, same buffers
        Xp.copy_(torch.randn_like(Xp))
        want_y = Bd.tucker_attn_decode(xd, *dw, Kd, Vd, ld, **{**dkw, "out": torch.empty_like(xd)})
        want_Y = Bd.tucker_attn_fwd(Xp, *dw, **{**pkw, "out": torch.empty_like(Xp)})
        y.zero_(); Y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert Bd.last_device_error() == 0
        assert torch.equal(y, want_y) and torch.equal(Y, want_Y), f"trial {trial}"


def test_decode_no_append_leaves_cache():
    w = H.custom_workload(kind="decode", dtype="fp32", d_model=32, n_H=4, r=(2, 8, 8), t=(2, 8, 8), rope=True, seed=18)
    y, ref, (Kd, Vd, Kc, Vc, *_r) = run_decode(w, 2, [5, 9], 16, append=False)
    check(y, ref, "fp32", "decode no-append")
    assert np.array_equal(Kd.cpu().numpy(), Kc.astype(np.float32))
    assert np.array_equal(Vd.cpu().numpy(), Vc.astype(np.float32))


def test_decode_bad_cache_len_is_flagged_not_fatal():
    import torch
    w = H.custom_workload(kind="decode", dtype="fp32", d_model=32, n_H=4, r=(2, 8, 8), t=(2, 8, 8), rope=False, seed=19)
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    dw = H.weights_to_device(wt, "fp32")
    Kd = torch.zeros(2, 8, 8, device="cuda")
    Vd = torch.zeros(2, 8, 8, device="cuda")
    xd = torch.randn(2, 32, device="cuda")
    ld = torch.tensor([3, 8], dtype=torch.int32, device="cuda")        # 8 == Lmax: out of range
    Bd.tucker_attn_decode(xd, *dw, Kd, Vd, ld, n_H=4, rope=False)
    assert Bd.last_device_error() & Bd.TA_DEVERR_BAD_CACHE_LEN
    assert Bd.last_device_error() == 0                                 # cleared by the read


def test_a_wait_that_nothing_ends_gives_up_and_is_reported():
    # The kernels' waits are bounded: one that runs out sets TA_DEVERR_WAIT_TIMEOUT and every other wait of
    # the block returns through the abort flag.  The library's self-test kernel does exactly that with a
    # 2 ms budget (a barrier that nothing signals); the context must stay usable afterwards.
    import torch
    assert Bd.last_device_error() == 0
    out = Bd.selftest_wait_timeout(2000)
    err = Bd.last_device_error()                       # synchronises the stream
    assert err == Bd.TA_DEVERR_WAIT_TIMEOUT
    Bd.selftest_wait_timeout(1000)                     # once more: the status-code form of the same read
    assert Bd.sync_status() == -5 and Bd.status_string(-5) == "device-side wait timed out"
    assert Bd.sync_status() == 0
    first, second, cycles_k = out.cpu().tolist()
    assert first == 0 and second == 0                  # both waits gave up ...
    assert cycles_k < (50_000_000 >> 10)               # ... the second long before its own two-second budget
    assert Bd.last_device_error() == 0                 # the word is cleared by the read
    w = W.get_workload("c1")                           # and ordinary calls still work
    X, wt = H.host_inputs(w)
    check(gpu_fwd(X, wt, w), oracle_fwd(X, wt, w), "fp32", "c1 after the self-test")


# --------------------------------------------------------------------------------------
# benchmark-sized workloads, sampled
# --------------------------------------------------------------------------------------

def sample_rows(N, n, seed):
    rng = np.random.default_rng(seed)
    fixed = [r for r in (0, 1, 63, 64, 127, 128, 129, 255, 256, N // 2, N - 2, N - 1) if 0 <= r < N]
    extra = rng.choice(N, size=min(n, N), replace=False).tolist()
    return sorted(set(fixed + extra))[: n + len(fixed)]


@pytest.mark.parametrize("name,nrows", [("c2", 96), ("c3", 197), ("c4", 40)])
def test_full_size_prefill_sampled(name, nrows):
    w = W.get_workload(name)
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w)
    batches = sorted(set([0, w.B - 1, w.B // 2]))
    rows = sample_rows(w.N, nrows, w.seed)
    ref = oracle_fwd(X[batches], wt, w, rows=rows)
    check(got[batches][:, rows], ref, w.dtype, name)


def test_persistent_grid_walks_many_causal_items():
    # 1152 causal work items of 1 - 8 key tiles on one CTA per SM (each CTA walks about eight items, back and forth
    # through the size-ordered list), an odd number of head pairs per row tile and ragged last tiles
    w = H.custom_workload(dtype="bf16", B=16, N=1000, d_model=576, n_H=18, r=(6, 64, 64), t=(6, 64, 64), causal=True,
                          rope=True, rope_base=10000.0, seed=88)
    X, wt = H.host_inputs(w)
    got = gpu_fwd(X, wt, w)
    assert Bd.last_path() == 2
    batches, rows = [0, 9, 15], sample_rows(w.N, 24, 3)
    check(got[batches][:, rows], oracle_fwd(X[batches], wt, w, rows=rows), "bf16", "causal, persistent grid")


def test_sharp_softmax_variant():
    # pre-softmax core scaled by 8: peaky rows exercise the online rescaling
    w = H.with_(W.get_workload("c2"), B=2)
    X, wt = H.host_inputs(w, core_gain=8.0)
    got = gpu_fwd(X, wt, w)
    rows = sample_rows(w.N, 64, 5)
    check(got[:, rows], oracle_fwd(X, wt, w, rows=rows), w.dtype, "sharp c2", scaled=True)


def test_full_size_decode_sampled():
    # benchmark decode workload: 64 sequences, 32768 cached latent rows each, RoPE at position 32768
    # (in the launch configuration bench.py times)
    import torch
    w = W.get_workload("c5")
    L, Lmax, B = w.N, w.N + 1, w.B
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w).items()}
    dw = H.weights_to_device(wt, w.dtype)
    x = W.round_to_storage(W.make_decode_x(w), w.dtype)
    Kd = torch.zeros(B, Lmax, w.r[2], dtype=torch.bfloat16, device="cuda")
    Vd = torch.zeros(B, Lmax, w.t[2], dtype=torch.bfloat16, device="cuda")
    lens = np.full((B,), L, dtype=np.int32)
    lens[5], lens[40] = 12345, 127            # ragged lengths inside the full-size launch
    for b in range(B):
        k, v = W.decode_cache_rows(w, b, int(lens[b]))
        Kd[b, :lens[b]] = torch.from_numpy(k).to(torch.bfloat16).cuda()
        Vd[b, :lens[b]] = torch.from_numpy(v).to(torch.bfloat16).cuda()
    y = Bd.tucker_attn_decode(H.to_device(x, w.dtype), *dw, Kd, Vd, torch.from_numpy(lens).cuda(), n_H=w.n_H,
                              rope=True, rope_base=w.rope_base, append=True)
    assert Bd.last_device_error() == 0
    y = y.float().cpu().numpy().astype(np.float64)
    sample = [0, 5, 40, 63]
    Kh = np.stack([Kd[b].float().cpu().numpy() for b in sample]).astype(np.float64)
    Vh = np.stack([Vd[b].float().cpu().numpy() for b in sample]).astype(np.float64)
    for i, b in enumerate(sample):        # slot L was appended by the call; the oracle must not see it
        Kh[i, lens[b]:] = 0
        Vh[i, lens[b]:] = 0
    ref, ref_k, _ = O.tucker_attn_decode(x[sample], *[wt[k] for k in H.WEIGHT_KEYS], Kh, Vh, lens[sample], rope=True,
                                         rope_base=w.rope_base)
    check(y[sample], ref, w.dtype, "c5 decode")
    got_k = np.stack([Kd[b, lens[b]].float().cpu().numpy() for b in sample])
    assert np.abs(got_k - ref_k).max() < 3e-2

"""GPU parity of the weight packers (MHA, GQA / MQA, MLA as Tucker attention, Sec. 2.2): the packed
tensors against the oracle's constructions element by element, and the packed weights run through
tucker_attn_fwd against the independently coded MHA / GQA / MLA references."""
import numpy as np
import pytest

from oracle import tucker_oracle as O
from paper_2603_30033_b200 import binding as Bd
from tests import helpers as H

pytestmark = pytest.mark.gpu

KEYS = H.WEIGHT_KEYS      # C, U1, U2, U3, Ct, Ut1, Ut2, Ut3


def _host(rng, shape, fan_in, dtype):
    from paper_2603_30033_b200 import workloads as W
    return W.round_to_storage(rng.standard_normal(shape) / np.sqrt(fan_in), dtype).astype(np.float64)


def _to_host(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("n_H,n_G,d", [(4, 4, 128), (4, 2, 128), (6, 1, 96), (6, 4, 48)])
def test_pack_gqa_matches_oracle_and_runs(dtype, n_H, n_G, d):
    rng = np.random.default_rng(7 + n_H * 10 + n_G)
    d_H = d // n_H
    WQ, WO = _host(rng, (d, d), d, dtype), _host(rng, (d, d), d, dtype)
    WKg, WVg = _host(rng, (d, n_G * d_H), d, dtype), _host(rng, (d, n_G * d_H), d, dtype)
    ref_w = O.tucker_from_gqa(WQ, WKg, WVg, WO, n_H, n_G)
    dev = [H.to_device(a, dtype) for a in (WQ, WKg, WVg, WO)]
    packed = Bd.tucker_pack_gqa(*dev, n_H=n_H, n_G=n_G)
    for k, t in zip(KEYS, packed):             # copies, selectors and a transpose: exact
        assert np.array_equal(_to_host(t), ref_w[k]), k
    if n_G == n_H:
        again = Bd.tucker_pack_mha(*dev, n_H=n_H)
        for a, b in zip(packed, again):
            assert bool((a == b).all())
    # the packed weights, through the layer, against the independent GQA model
    N = 40
    X = _host(rng, (1, N, d), 1.0, dtype)
    Y = Bd.tucker_attn_fwd(H.to_device(X, dtype), *packed, n_H=n_H, causal=True, rope=False)
    assert Bd.last_device_error() == 0
    ref = O.gqa_reference(X[0], WQ, WKg, WVg, WO, n_H, n_G, causal=True)
    H.check(_to_host(Y)[0], ref, dtype, f"pack_gqa n_H={n_H} n_G={n_G} d={d}")
    # d = 128 has every rank a multiple of 32 and d a multiple of 64: the packed weights reach the tensor-core kernels
    assert Bd.last_path() == (2 if (dtype == "bf16" and d == 128) else 1)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shared", [False, True])
def test_pack_mla_matches_oracle_and_runs(dtype, shared):
    rng = np.random.default_rng(31 + int(shared))
    d, n_H, dcq, dck = 96, 6, 40, 24
    WDQ, WDKV = _host(rng, (d, dcq), d, dtype), _host(rng, (d, dck), d, dtype)
    WDV = WDKV if shared else _host(rng, (d, dck), d, dtype)
    WUQ, WUK, WUV = _host(rng, (dcq, d), dcq, dtype), _host(rng, (dck, d), dck, dtype), _host(rng, (dck, d), dck, dtype)
    WO = _host(rng, (d, d), d, dtype)
    ref_w = O.tucker_from_mla(WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H)
    dev = [H.to_device(a, dtype) for a in (WDQ, WUQ, WDKV, WUK, WDV, WUV, WO)]
    packed = Bd.tucker_pack_mla(*dev, n_H=n_H)
    tol = 2e-6 if dtype == "fp32" else 8e-3        # cores: fp32 sums of d_H products, then the storage rounding
    for k, t in zip(KEYS, packed):
        got = _to_host(t)
        if k in ("C", "Ct"):
            assert np.abs(got - ref_w[k]).max() <= tol * max(1.0, np.abs(ref_w[k]).max()), k
        else:
            assert np.array_equal(got, ref_w[k]), k
    N = 33
    X = _host(rng, (1, N, d), 1.0, dtype)
    Y = Bd.tucker_attn_fwd(H.to_device(X, dtype), *packed, n_H=n_H, causal=True, rope=False)
    assert Bd.last_device_error() == 0
    # (1) the layer itself, against the oracle on exactly the weights it was given (the packed, storage-rounded
    # tensors): the ordinary bounds of the layer apply
    pw = {k: _to_host(t) for k, t in zip(KEYS, packed)}
    ref_packed = O.tucker_attn_fwd(X[0], *[pw[k] for k in KEYS], causal=True, rope=False)
    H.check(_to_host(Y)[0], ref_packed, dtype, f"pack_mla layer shared={shared}")
    # (2) end to end against the independently coded MLA model on the unpacked weights: the packed cores carry
    # one storage rounding that this model does not have, which the oracle itself quantifies
    ref = O.mla_reference(X[0], WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H, causal=True)
    core_rounding = np.abs(ref_packed - ref).max()
    mx, mean = H.err_stats(_to_host(Y)[0], ref)
    tmax, tmean = H.tolerances(dtype)
    assert mx <= tmax + core_rounding and mean <= tmean + core_rounding, (mx, mean, core_rounding)


def _mla_case(rng, d, n_H, dcq, dck, shared, dtype="bf16"):
    WDQ, WDKV = _host(rng, (d, dcq), d, dtype), _host(rng, (d, dck), d, dtype)
    WDV = WDKV if shared else _host(rng, (d, dck), d, dtype)
    WUQ, WUK, WUV = _host(rng, (dcq, d), dcq, dtype), _host(rng, (dck, d), dck, dtype), _host(rng, (dck, d), dck, dtype)
    WO = _host(rng, (d, d), d, dtype)
    return WDQ, WUQ, WDKV, WUK, WDV, WUV, WO


@pytest.mark.parametrize("shared", [False, True])
def test_pack_mla_with_latent_rope_prefill_and_decode(shared):
    """MLA with RoPE in its key latent (Sec. 3.2.1; App. C.2 "MLA - coupled RoPE"): tucker_pack_mla output run
    with rope = 1 on the tensor-core kernels, prefill and one cached decode step, against the independent
    explicit-rotation-matrix evaluator of the fused form."""
    import torch
    rng = np.random.default_rng(47 + int(shared))
    d, n_H, dcq, dck, base, N = 256, 4, 64, 64, 10000.0, 150
    Ws = _mla_case(rng, d, n_H, dcq, dck, shared)
    packed = Bd.tucker_pack_mla(*[H.to_device(a, "bf16") for a in Ws], n_H=n_H)
    pw = {k: _to_host(t) for k, t in zip(KEYS, packed)}
    X = _host(rng, (1, N, d), 1.0, "bf16")
    Kc = torch.zeros(1, N + 8, dck, device="cuda", dtype=torch.bfloat16)
    Vc = torch.zeros(1, N + 8, dck, device="cuda", dtype=torch.bfloat16)
    Y = Bd.tucker_attn_fwd(H.to_device(X[:, :N - 1], "bf16"), *packed, n_H=n_H, causal=True, rope=True, rope_base=base,
                           Kcache=Kc, Vcache=Vc)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    # the layer on the weights it was given
    ref_packed = O.tucker_attn_fwd(X[0], *[pw[k] for k in KEYS], causal=True, rope=True, rope_base=base)
    H.check(_to_host(Y)[0], ref_packed[:N - 1], "bf16", f"pack_mla latent RoPE prefill shared={shared}")
    # the independent MLA evaluator with explicit rotation matrices
    ref = O.mla_latent_rope_reference(X[0], *Ws, n_H, causal=True, rope_base=base)
    core_rounding = np.abs(ref_packed - ref).max()
    tmax, tmean = H.tolerances("bf16")
    mx, mean = H.err_stats(_to_host(Y)[0], ref[:N - 1])
    assert mx <= tmax + core_rounding and mean <= tmean + core_rounding, (mx, mean, core_rounding)
    # one decode step for the last token over the cache the prefill wrote = last row of the full sequence
    lens = torch.tensor([N - 1], dtype=torch.int32, device="cuda")
    y = Bd.tucker_attn_decode(H.to_device(X[0, N - 1:N], "bf16"), *packed, Kc, Vc, lens, n_H=n_H, rope=True,
                              rope_base=base, append=True)
    assert Bd.last_device_error() == 0 and Bd.last_path() == 2
    H.check(_to_host(y)[0], ref_packed[N - 1], "bf16", f"pack_mla latent RoPE decode shared={shared}")
    mx, mean = H.err_stats(_to_host(y)[0], ref[N - 1])
    assert mx <= tmax + core_rounding and mean <= tmean + core_rounding, (mx, mean, core_rounding)


def test_pack_rejects_bad_sizes():
    import torch
    z = torch.zeros(8, 8, device="cuda")
    with pytest.raises(ValueError):
        Bd.tucker_pack_gqa(z, z, z, z, n_H=3, n_G=1)          # d not a multiple of n_H
    with pytest.raises(ValueError):
        Bd.tucker_pack_gqa(z, z, z, z, n_H=2, n_G=4)          # more groups than heads

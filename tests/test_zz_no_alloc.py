"""tucker_attn_decode_static: the decode entry point for callers that cannot allocate device
memory (their memory belongs to someone else's pool, or cudaMalloc's device-wide
synchronisation is off limits on their hot path).  It keeps its scratch in a static device
array inside the library instead of taking a workspace argument.

Checked here, through the C ABI: two calls in a row (different inputs, the first one larger,
so the second one meets the first one's leftovers in the shared scratch) each give bit for
bit the result of tucker_attn_decode with a freshly allocated workspace, on the tensor-core
path and on the generic path, and the second also agrees with the CPU oracle; a problem whose
scratch would not fit the array is refused up front.
This file sorts last so that a run stopping at the first failure has run everything else.
"""
import numpy as np
import pytest

from paper_2603_30033_b200 import binding as Bd
from paper_2603_30033_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _state(w, lens, Lmax, seed_shift):
    import torch
    w2 = H.with_(w, seed=w.seed + seed_shift)
    wt = {k: W.round_to_storage(v, w.dtype) for k, v in W.make_weights(w2).items()}
    x, Kc, Vc, cache_len = W.make_decode_state(w2, B=len(lens), L=max(lens), Lmax=Lmax, cache_len=lens)
    dev = lambda a: H.to_device(W.round_to_storage(a, w.dtype), w.dtype)
    return dev(x), H.weights_to_device(wt, w.dtype), dev(Kc), dev(Vc), torch.from_numpy(cache_len).cuda()


@pytest.mark.parametrize("dtype,shape,path", [
    ("bf16", dict(d_model=256, n_H=8, r=(4, 64, 64), t=(4, 64, 64)), 2),
    ("fp32", dict(d_model=64, n_H=4, r=(2, 16, 12), t=(2, 10, 20)), 1),
])
def test_static_scratch_decode_matches_workspace_decode_twice(dtype, shape, path):
    """Two calls in a row through tucker_attn_decode_static.  The first is the larger one (more sequences,
    longer caches), so the second meets leftovers in every region of the shared array that it uses and in
    regions beyond.  Both forms run the same deterministic kernels (no atomics), so the results must be
    bit-identical to tucker_attn_decode with a fresh workspace; the second call is also held to the oracle."""
    import torch
    from oracle import tucker_oracle as O
    w = H.custom_workload(kind="decode", dtype=dtype, rope=True, rope_base=500000.0, seed=41, **shape)
    Lmax = 2100
    tmax, tmean = H.tolerances(dtype)
    calls = [[0, 129, 650, 31, 2099, 1500, 777, 1, 128, 2048, 300, 64], [512, 3, 300, 699]]
    for call, lens in enumerate(calls):
        x, dw, Kd, Vd, ld = _state(w, lens, Lmax, seed_shift=call)
        K0, V0 = Kd.clone(), Vd.clone()
        K2, V2 = Kd.clone(), Vd.clone()
        ref = Bd.tucker_attn_decode(x, *dw, Kd, Vd, ld, n_H=w.n_H, rope=True, rope_base=w.rope_base, append=True)
        assert Bd.last_device_error() == 0
        out = torch.full_like(x, float("nan"))
        got = Bd.tucker_attn_decode_static(x, *dw, K2, V2, ld, out, n_H=w.n_H, rope=True, rope_base=w.rope_base,
                                           append=True)
        assert Bd.last_device_error() == 0 and Bd.last_path() == path
        assert got.data_ptr() == out.data_ptr()
        assert torch.isfinite(got).all()
        assert torch.equal(got, ref), f"call {call}: static-scratch result differs from the workspace result"
        assert torch.equal(K2, Kd) and torch.equal(V2, Vd)      # the appended cache rows agree as well
        if call == 1:
            host = lambda t: t.float().cpu().numpy().astype(np.float64)
            yo, _, _ = O.tucker_attn_decode(host(x), *[host(t) for t in dw], host(K0), host(V0), np.asarray(lens),
                                            rope=True, rope_base=w.rope_base)
            mx, mean = H.err_stats(host(got), yo)
            assert mx <= tmax and mean <= tmean, f"against the oracle: max-abs {mx:.3e}, mean-abs {mean:.3e}"


def test_static_scratch_reports_the_same_status_as_the_workspace_form():
    # an invalid descriptor is refused by the decode call's own validation, with its status
    import torch
    f = dict(dtype=torch.float32, device="cuda")
    z = lambda *s: torch.zeros(*s, **f)
    args = (z(2, 32), z(2, 8, 7), z(4, 2), z(32, 8), z(32, 7), z(2, 8, 8), z(4, 2), z(32, 8), z(32, 8), z(2, 4, 7), z(2, 4, 8),
            torch.zeros(2, dtype=torch.int32, device="cuda"))
    with pytest.raises(Bd.TuckerAttnError) as e1:                 # odd r3 with latent RoPE
        Bd.tucker_attn_decode(*args, n_H=4, rope=True)
    with pytest.raises(Bd.TuckerAttnError) as e2:
        Bd.tucker_attn_decode_static(*args, z(2, 32), n_H=4, rope=True)
    assert e1.value.status == e2.value.status == -1


def test_static_scratch_rejects_oversized_problem():
    import torch
    # 2048 sequences need far more than the 16 MiB array; nothing may be launched or written
    d, n_H, B, Lmax = 1024, 32, 2048, 8
    r = t = (8, 128, 128)
    desc = Bd.make_desc(B=B, N=1, d_model=d, n_H=n_H, r=r, t=t, causal=True, rope=True, dtype=Bd.TA_DTYPE_BF16)
    assert Bd.decode_workspace_bytes(desc, Lmax) > Bd.TA_STATIC_SCRATCH_BYTES
    bf = dict(dtype=torch.bfloat16, device="cuda")
    z = lambda *s: torch.zeros(*s, **bf)
    out = torch.full((B, d), 3.0, **bf)
    with pytest.raises(Bd.TuckerAttnError) as e:
        Bd.tucker_attn_decode_static(z(B, d), z(*r), z(n_H, r[0]), z(d, r[1]), z(d, r[2]), z(*t), z(n_H, t[0]),
                                     z(d, t[1]), z(d, t[2]), z(B, Lmax, r[2]), z(B, Lmax, t[2]),
                                     torch.zeros(B, dtype=torch.int32, device="cuda"), out, n_H=n_H, rope=True)
    assert e.value.status == -3 and "workspace too small" in str(e.value)
    assert (out == 3.0).all()

"""GPU parity of the HOSVD initialiser (App. C.1 "MHA to Tucker Attention"; spectra of Sec. 2.1) against the
oracle's numpy-SVD statement: weight tensors, factor subspaces (singular vectors are unique only up to sign and,
inside clusters, rotation: what is compared is the projector and the reassembled tensor), cores, spectra, the
truncation error bound, and the initialised weights run through the attention layer."""
import numpy as np
import pytest

from oracle import tucker_oracle as O
from paper_2603_30033_b200 import binding as Bd
from paper_2603_30033_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _dev32(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _host(t):
    return t.float().cpu().numpy().astype(np.float64)


def _mha(d, n_H, rank, noise, seed):
    w = W.make_lowrank_mha(d, n_H, rank, noise, seed)
    return {k: v.astype(np.float32).astype(np.float64) for k, v in w.items()}


@pytest.mark.parametrize("d,n_H", [(48, 4), (128, 4)])
def test_mha_weight_tensors_match_oracle(d, n_H):
    w = _mha(d, n_H, 6, 0.05, 301)
    Wg, Wtg = Bd.tucker_mha_weight_tensors(*[_dev32(w[k]) for k in ("WQ", "WK", "WV", "WO")], n_H=n_H)
    Wo, Wto = O.mha_weight_tensors(w["WQ"], w["WK"], w["WV"], w["WO"], n_H)
    assert np.abs(_host(Wg) - Wo).max() <= 2e-6 * max(1.0, np.abs(Wo).max())
    assert np.abs(_host(Wtg) - Wto).max() <= 2e-6 * max(1.0, np.abs(Wto).max())


def _projector_gap(Ug, Uo):
    """largest sine of the principal angles between the two column spaces"""
    return np.linalg.norm(Ug - Uo @ (Uo.T @ Ug), 2)


# (d, n_H, rank of the synthetic structure, noise, ranks asked for): 48 -> fp32 FMA Gram route, 128 / 256 -> tensor cores
@pytest.mark.parametrize("d,n_H,rank,noise,ranks", [
    (48, 4, 5, 0.02, (3, 5, 5)),
    (128, 4, 8, 0.02, (4, 8, 8)),
    (256, 8, 16, 0.01, (6, 16, 16)),
    (128, 3, 8, 0.02, (2, 32, 16)),          # ranks beyond the structure: inside the noise cluster only the error counts
])
def test_hosvd_matches_oracle(d, n_H, rank, noise, ranks):
    w = _mha(d, n_H, rank, noise, 311 + d)
    T, _ = O.mha_weight_tensors(w["WQ"], w["WK"], w["WV"], w["WO"], n_H)
    T = T.astype(np.float32).astype(np.float64)
    C, U1, U2, U3, spec = Bd.tucker_hosvd_init(_dev32(T), ranks)
    assert Bd.last_device_error() == 0
    Cg, Ug = _host(C), [_host(U1), _host(U2), _host(U3)]
    Co, Uo, sv = O.hosvd(T, ranks)
    tnorm = np.linalg.norm(T)
    for j in range(3):
        r = ranks[j]
        np.testing.assert_allclose(Ug[j].T @ Ug[j], np.eye(r), atol=2e-4)                  # orthonormal columns
        s_g, s_o = _host(spec[j]), sv[j]
        big = s_o > 2e-3 * s_o[0]
        assert np.abs(s_g[:len(s_o)][big] - s_o[big]).max() <= 2e-3 * s_o[0], j           # spectra (Sec. 2.1)
        assert np.all(np.diff(s_g) <= 1e-6 * s_o[0])                                       # descending
        gap = (s_o[r - 1] ** 2 - (s_o[r] ** 2 if r < len(s_o) else 0.0)) / s_o[0] ** 2
        if gap > 1e-2:                                                                      # a well separated subspace
            assert _projector_gap(Ug[j], Uo[j]) <= 2e-3 / gap ** 0.5, (j, gap)
    # the core is the projection of T onto the GPU's own factors
    core_ref = T
    for mode in (1, 2, 3):
        core_ref = O.mode_product(core_ref, Ug[mode - 1].T, mode)
    assert np.abs(Cg - core_ref).max() <= 2e-4 * max(1.0, np.abs(core_ref).max())
    # reassembled tensor: as good as the oracle's truncation, and inside the HOSVD error bound
    err_g = np.linalg.norm(T - O.assemble_dense(Cg, *Ug))
    err_o = np.linalg.norm(T - O.assemble_dense(Co, *Uo))
    bound = np.sqrt(sum(np.sum(s[r:] ** 2) for s, r in zip(sv, ranks)))
    assert err_g <= err_o * 1.01 + 2e-4 * tnorm, (err_g, err_o)
    assert err_g <= bound * 1.01 + 2e-4 * tnorm


def test_hosvd_initialised_layer_reproduces_mha_at_full_rank():
    # ranks (n_H, d, d): nothing is truncated, so the initialised Tucker layer must equal the MHA layer it came from
    d, n_H, N = 64, 4, 48
    w = _mha(d, n_H, 8, 0.3, 331)
    dev = [_dev32(w[k]) for k in ("WQ", "WK", "WV", "WO")]
    Wg, Wtg = Bd.tucker_mha_weight_tensors(*dev, n_H=n_H)
    C, U1, U2, U3, _ = Bd.tucker_hosvd_init(Wg, (n_H, d, d))
    Ct, Ut1, Ut2, Ut3, _ = Bd.tucker_hosvd_init(Wtg, (n_H, d, d))
    rng = np.random.default_rng(5)
    X = rng.standard_normal((1, N, d)).astype(np.float32)
    Y = Bd.tucker_attn_fwd(_dev32(X), C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, n_H=n_H, causal=True, rope=False)
    assert Bd.last_device_error() == 0
    ref = O.mha_reference(X[0].astype(np.float64), w["WQ"], w["WK"], w["WV"], w["WO"], n_H, causal=True)
    mx, mean = H.err_stats(_host(Y)[0], ref)
    assert mx <= 2e-3 * max(1.0, np.abs(ref).max()) and mean <= 2e-4, (mx, mean)
    # and the oracle's own HOSVD of the same weights agrees (pins the statement the GPU result is compared with)
    wo = O.mha_to_tucker(w["WQ"], w["WK"], w["WV"], w["WO"], n_H, (n_H, d, d), (n_H, d, d))
    ref2 = O.tucker_attn_fwd(X[0].astype(np.float64), *[wo[k] for k in H.WEIGHT_KEYS], causal=True)
    np.testing.assert_allclose(ref2, ref, atol=1e-9)


def test_hosvd_rejects_bad_sizes():
    import torch
    T = torch.zeros(4, 32, 32, device="cuda")
    with pytest.raises(Bd.TuckerAttnError):
        Bd.tucker_hosvd_init(T, (5, 8, 8))           # r1 > n_H
    with pytest.raises(ValueError):
        Bd.tucker_hosvd_init(torch.zeros(4, 32, 16, device="cuda"), (2, 8, 8))

"""Pins of the oracle functions behind the widened rows: MLA with RoPE in its key latent
(Sec. 3.2.1), the shared latent cache with latent RoPE (Sec. 3.1 + Definition 2) and the HOSVD
initialiser (App. C.1, Sec. 2.1).  CPU only."""
import numpy as np
import pytest

from oracle import tucker_oracle as O

KEYS = ("C", "U1", "U2", "U3", "Ct", "Ut1", "Ut2", "Ut3")


def fwd(X, w, **kw):
    return O.tucker_attn_fwd(X, *[w[k] for k in KEYS], **kw)


def _mla_weights(rng, d, cq, ck, shared):
    WDQ = rng.standard_normal((d, cq)) / np.sqrt(d)
    WUQ = rng.standard_normal((cq, d)) / np.sqrt(cq)
    WDKV = rng.standard_normal((d, ck)) / np.sqrt(d)
    WUK = rng.standard_normal((ck, d)) / np.sqrt(ck)
    WDV = WDKV if shared else rng.standard_normal((d, ck)) / np.sqrt(d)
    WUV = rng.standard_normal((ck, d)) / np.sqrt(ck)
    WO = rng.standard_normal((d, d)) / np.sqrt(d)
    return WDQ, WUQ, WDKV, WUK, WDV, WUV, WO


# --------------------------------------------------------------------------------------
# MLA with RoPE in the key latent
# --------------------------------------------------------------------------------------

def test_rope_matrix_is_a_rotation_with_the_relative_property():
    base, r = 10000.0, 8
    Rm, Rn = O.rope_matrix(11, r, base), O.rope_matrix(4, r, base)
    np.testing.assert_allclose(Rm @ Rm.T, np.eye(r), atol=1e-13)
    np.testing.assert_allclose(Rm @ Rn.T, O.rope_matrix(7, r, base), atol=1e-12)      # Eq. 10
    np.testing.assert_allclose(O.rope_matrix(0, r, base), np.eye(r), atol=0)
    # first pair turns by exactly pos radians: (1, 0) -> (cos, sin)
    np.testing.assert_allclose((np.eye(r)[0] @ O.rope_matrix(0.5, r, base))[:2], [np.cos(0.5), np.sin(0.5)], atol=1e-15)
    # and the vectorised routine applies the same matrix
    x = np.random.default_rng(0).standard_normal((3, r))
    for n, pos in enumerate((2, 9, 31)):
        np.testing.assert_allclose(O.rope_rotate(x[n:n + 1], np.array([pos]), base)[0], x[n] @ O.rope_matrix(pos, r, base),
                                   atol=1e-13)


@pytest.mark.parametrize("shared", [False, True])
@pytest.mark.parametrize("causal", [False, True])
def test_mla_latent_rope_equals_tucker_latent_rope_on_the_mla_embedding(shared, causal):
    rng = np.random.default_rng(61)
    d, n_H, N, cq, ck, base = 16, 4, 9, 6, 8, 10000.0
    Ws = _mla_weights(rng, d, cq, ck, shared)
    X = rng.standard_normal((N, d))
    w = O.tucker_from_mla(*Ws, n_H)
    ref = O.mla_latent_rope_reference(X, *Ws, n_H, causal=causal, rope_base=base, pos0=5)
    got = fwd(X, w, causal=causal, rope=True, rope_base=base, pos0=5)
    np.testing.assert_allclose(got, ref, atol=1e-11, rtol=0)
    # the rotation matters, and it is not MLA without RoPE
    assert np.abs(ref - O.mla_reference(X, *Ws, n_H, causal=causal)).max() > 1e-3


def test_mla_latent_rope_position_offset_invariance():
    rng = np.random.default_rng(62)
    d, n_H, N = 12, 3, 7
    Ws = _mla_weights(rng, d, 5, 6, True)
    X = rng.standard_normal((N, d))
    a = O.mla_latent_rope_reference(X, *Ws, n_H, causal=True, pos0=0)
    b = O.mla_latent_rope_reference(X, *Ws, n_H, causal=True, pos0=913)
    np.testing.assert_allclose(a, b, atol=1e-9, rtol=0)


def test_one_head_mla_without_up_projection_is_mha_with_standard_rope():
    # n_H = 1, dcK = d_H = d and WUK = I: the key latent IS the head dimension, so RoPE in the key latent
    # is textbook RoPE on one head (App. C.2 "MHA").  Pins mha_reference(rope=True) and gqa_reference(rope=True)
    # against the explicit-matrix evaluator.
    rng = np.random.default_rng(63)
    d, N, base = 8, 6, 10000.0
    WDQ = rng.standard_normal((d, d)) / np.sqrt(d)
    WUQ = rng.standard_normal((d, d)) / np.sqrt(d)
    WDKV = rng.standard_normal((d, d)) / np.sqrt(d)
    WDV = rng.standard_normal((d, d)) / np.sqrt(d)
    WUV = rng.standard_normal((d, d)) / np.sqrt(d)
    WO = rng.standard_normal((d, d)) / np.sqrt(d)
    X = rng.standard_normal((N, d))
    ref = O.mla_latent_rope_reference(X, WDQ, WUQ, WDKV, np.eye(d), WDV, WUV, WO, 1, causal=True, rope_base=base, pos0=2)
    mha = O.mha_reference(X, WDQ @ WUQ, WDKV, WDV @ WUV, WO, 1, causal=True, rope=True, rope_base=base, pos0=2)
    np.testing.assert_allclose(mha, ref, atol=1e-11, rtol=0)
    gqa = O.gqa_reference(X, WDQ @ WUQ, WDKV, WDV @ WUV, WO, 1, 1, causal=True, rope=True, rope_base=base, pos0=2)
    np.testing.assert_allclose(gqa, ref, atol=1e-11, rtol=0)


def test_mha_standard_rope_is_per_head():
    # several heads: mha_reference(rope=True) rotates every head's d_H coordinates separately;
    # checked against per-head explicit matrices (a third coding)
    rng = np.random.default_rng(64)
    d, n_H, N, base = 12, 3, 5, 100.0
    d_H = d // n_H
    WQ, WK, WV, WO = (rng.standard_normal((d, d)) / np.sqrt(d) for _ in range(4))
    X = rng.standard_normal((N, d))
    out = np.zeros((N, d))
    for i in range(n_H):
        sl = slice(i * d_H, (i + 1) * d_H)
        q = np.stack([X[m] @ WQ[:, sl] @ O.rope_matrix(m, d_H, base) for m in range(N)])
        k = np.stack([X[m] @ WK[:, sl] @ O.rope_matrix(m, d_H, base) for m in range(N)])
        s = q @ k.T / np.sqrt(d_H)
        p = np.exp(s) / np.exp(s).sum(1, keepdims=True)
        out += p @ (X @ WV[:, sl]) @ WO[sl]
    np.testing.assert_allclose(O.mha_reference(X, WQ, WK, WV, WO, n_H, rope=True, rope_base=base), out, atol=1e-11)


# --------------------------------------------------------------------------------------
# shared latent cache with latent RoPE
# --------------------------------------------------------------------------------------

def _shared_w(rng, d, n_H, r, t2):
    r1, r2, r3 = r
    w = dict(C=rng.standard_normal((r1, r2, r3)) * 0.7, U1=rng.standard_normal((n_H, r1)),
             U2=rng.standard_normal((d, r2)) / np.sqrt(d) * 2, U3=rng.standard_normal((d, r3)) / np.sqrt(d) * 2,
             Ct=rng.standard_normal((r1, t2, r3)) * 0.7, Ut1=rng.standard_normal((n_H, r1)),
             Ut2=rng.standard_normal((d, t2)) / np.sqrt(d))
    w["Ut3"] = w["U3"]
    return w


def test_shared_cache_rope_decode_equals_last_row_of_shared_projection_prefill():
    rng = np.random.default_rng(71)
    d, n_H, L, base = 12, 3, 9, 10000.0
    w = _shared_w(rng, d, n_H, (2, 6, 8), 5)
    X = rng.standard_normal((2, L + 1, d))
    Yfull, parts = fwd(X, w, causal=True, rope=True, rope_base=base, return_parts=True)
    lens = np.array([L, L - 4])
    Lc = np.zeros((2, L + 3, 8))
    for b in range(2):
        Lc[b, :L] = parts[b]["V"][:L]                  # un-rotated latent rows (V = X U3)
    Lc[1, L - 4:] = 1e30                                # slots beyond the length are never read
    xs = np.stack([X[0, L], X[1, L - 4]])
    y, ln = O.tucker_attn_decode_shared_rope(xs, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"], Lc, lens,
                                             rope_base=base)
    np.testing.assert_allclose(y[0], Yfull[0, L], atol=1e-11, rtol=0)
    np.testing.assert_allclose(y[1], Yfull[1, L - 4], atol=1e-11, rtol=0)
    np.testing.assert_allclose(ln[0], parts[0]["V"][L], atol=1e-12)


def test_shared_cache_rope_decode_equals_two_cache_decode_on_rotated_and_plain_copies():
    rng = np.random.default_rng(72)
    d, n_H, L, base = 10, 2, 7, 500000.0
    w = _shared_w(rng, d, n_H, (2, 4, 6), 3)
    Lc = rng.standard_normal((1, L + 1, 6))
    x = rng.standard_normal((1, d))
    lens = np.array([L])
    Kc = np.zeros_like(Lc)
    Kc[0, :L] = np.stack([Lc[0, n] @ O.rope_matrix(n, 6, base) for n in range(L)])
    y2, _, _ = O.tucker_attn_decode(x, *[w[k] for k in KEYS], Kc, Lc, lens, rope=True, rope_base=base)
    y1, _ = O.tucker_attn_decode_shared_rope(x, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"], Lc, lens,
                                             rope_base=base)
    np.testing.assert_allclose(y1, y2, atol=1e-12, rtol=0)


# --------------------------------------------------------------------------------------
# HOSVD
# --------------------------------------------------------------------------------------

def _assemble(core, Us):
    return O.assemble_dense(core, *Us)


def test_mode_unfold_matches_fibre_definition():
    rng = np.random.default_rng(80)
    T = rng.standard_normal((2, 3, 4))
    for mode in (1, 2, 3):
        M = O.mode_unfold(T, mode)
        assert M.shape == (T.shape[mode - 1], T.size // T.shape[mode - 1])
        # every column is a mode-`mode` fibre: fixing the other two indices
        fibres = {tuple(np.round(np.take(np.take(T, a, axis=[1, 0, 0][mode - 1]), b, axis=[1, 1, 0][mode - 1]), 12))
                  for a in range(T.shape[[1, 0, 0][mode - 1]]) for b in range(T.shape[[2, 2, 1][mode - 1]])}
        assert {tuple(np.round(M[:, j], 12)) for j in range(M.shape[1])} == fibres
    # Gram of the unfolding = contraction over the other two modes
    np.testing.assert_allclose(O.mode_unfold(T, 2) @ O.mode_unfold(T, 2).T, np.einsum("ajc,akc->jk", T, T), atol=1e-12)


def test_hosvd_recovers_an_exact_rank_tensor():
    rng = np.random.default_rng(81)
    core = rng.standard_normal((2, 3, 4))
    Us = [np.linalg.qr(rng.standard_normal((n, r)))[0] for n, r in ((5, 2), (7, 3), (6, 4))]
    T = _assemble(core, Us)
    c2, U2s, sv = O.hosvd(T, (2, 3, 4))
    np.testing.assert_allclose(_assemble(c2, U2s), T, atol=1e-12)
    for U, U0, s, r in zip(U2s, Us, sv, (2, 3, 4)):
        np.testing.assert_allclose(U.T @ U, np.eye(r), atol=1e-12)               # orthonormal
        np.testing.assert_allclose(U @ (U.T @ U0), U0, atol=1e-11)               # same column space
        assert np.all(s[r:] < 1e-12 * s[0])                                       # exact multilinear rank
    # all-orthogonality of the HOSVD core: slices of one mode are mutually orthogonal, norms = singular values
    for mode in (1, 2, 3):
        M = O.mode_unfold(c2, mode)
        G = M @ M.T
        np.testing.assert_allclose(G, np.diag(sv[mode - 1][:G.shape[0]] ** 2), atol=1e-10)


def test_hosvd_truncation_error_bound_and_spectra():
    rng = np.random.default_rng(82)
    T = rng.standard_normal((4, 9, 8)) * np.logspace(0, -2, 9)[None, :, None]
    ranks = (3, 5, 4)
    core, Us, sv = O.hosvd(T, ranks)
    err2 = np.sum((T - _assemble(core, Us)) ** 2)
    bound = sum(np.sum(s[r:] ** 2) for s, r in zip(sv, ranks))
    assert err2 <= bound * (1 + 1e-12)
    assert err2 >= max(np.sum(s[r:] ** 2) for s, r in zip(sv, ranks)) * (1 - 1e-12)   # no better than the best single-mode cut
    for mode in (1, 2, 3):
        s = np.sqrt(np.clip(np.linalg.eigvalsh(np.einsum("abc,abd->cd", *(np.moveaxis(T, mode - 1, 2),) * 2))[::-1], 0, None))
        np.testing.assert_allclose(O.mode_spectrum(T, mode), s / s[0], atol=1e-10)
        assert O.mode_spectrum(T, mode)[0] == 1.0


def test_mha_to_tucker_round_trip_at_full_rank_and_matches_selector_embedding():
    rng = np.random.default_rng(83)
    d, n_H, N = 8, 2, 6
    WQ, WK, WV, WO = (rng.standard_normal((d, d)) / np.sqrt(d) for _ in range(4))
    W, Wt = O.mha_weight_tensors(WQ, WK, WV, WO, n_H)
    # the weight tensors are the dense tensors of the selector-core embedding (Lemma 1)
    emb = O.tucker_from_mha(WQ, WK, WV, WO, n_H)
    np.testing.assert_allclose(W, O.assemble_dense(emb["C"], emb["U1"], emb["U2"], emb["U3"]), atol=1e-12)
    np.testing.assert_allclose(Wt, O.assemble_dense(emb["Ct"], emb["Ut1"], emb["Ut2"], emb["Ut3"]), atol=1e-12)
    w = O.mha_to_tucker(WQ, WK, WV, WO, n_H, (n_H, d, d), (n_H, d, d))
    X = rng.standard_normal((N, d))
    np.testing.assert_allclose(fwd(X, w, causal=True), O.mha_reference(X, WQ, WK, WV, WO, n_H, causal=True), atol=1e-10)
    # low-rank MHA weights (rank-3 query / key maps shared by the heads) are reproduced exactly at ranks (n_H, 3, 3)
    A, Bm = rng.standard_normal((d, 3)), rng.standard_normal((d, 3))
    WQl = A @ rng.standard_normal((3, d))
    WKl = Bm @ rng.standard_normal((3, d))
    w2 = O.mha_to_tucker(WQl, WKl, WV, WO, n_H, (n_H, 3, 3), (n_H, d, d))
    np.testing.assert_allclose(fwd(X, w2, causal=True), O.mha_reference(X, WQl, WKl, WV, WO, n_H, causal=True), atol=1e-9)

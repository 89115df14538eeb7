"""Pins for the CPU oracle: every check compares it with something other than itself --
the brute-force tensor definition, independently coded MHA / GQA / MQA / MLA, closed forms,
invariants the paper states, and the sizes the paper prints.  No GPU needed."""
import os

import numpy as np
import pytest

from oracle import tucker_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_tucker(rng, d, n_H, r, t):
    r1, r2, r3 = r
    t1, t2, t3 = t
    return dict(
        C=rng.standard_normal((r1, r2, r3)) * 0.7, U1=rng.standard_normal((n_H, r1)),
        U2=rng.standard_normal((d, r2)) / np.sqrt(d) * 2, U3=rng.standard_normal((d, r3)) / np.sqrt(d) * 2,
        Ct=rng.standard_normal((t1, t2, t3)) * 0.7, Ut1=rng.standard_normal((n_H, t1)),
        Ut2=rng.standard_normal((d, t2)) / np.sqrt(d), Ut3=rng.standard_normal((d, t3)) / np.sqrt(d))


def fwd(X, w, **kw):
    return O.tucker_attn_fwd(X, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"], w["Ut3"], **kw)


def brute(X, w, **kw):
    return O.tucker_attn_bruteforce(X, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"],
                                    w["Ut3"], **kw)


# --------------------------------------------------------------------------------------
# brute force from the dense tensors (Eqs. 2-6) vs the factored evaluation order
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [
    dict(N=7, d=12, n_H=3, r=(2, 5, 4), t=(3, 6, 2)),
    dict(N=16, d=32, n_H=4, r=(2, 16, 16), t=(2, 16, 16)),
    dict(N=5, d=8, n_H=2, r=(2, 8, 8), t=(1, 3, 7)),
])
def test_fast_equals_bruteforce(shape, causal):
    rng = np.random.default_rng(11)
    w = rand_tucker(rng, shape["d"], shape["n_H"], shape["r"], shape["t"])
    X = rng.standard_normal((2, shape["N"], shape["d"]))
    np.testing.assert_allclose(fwd(X, w, causal=causal), brute(X, w, causal=causal), rtol=0, atol=1e-11)


def test_bruteforce_on_tiny_config_shapes():
    # shapes of the tiny fp32 workload (N=64, d=128, n_H=4, ranks 2/16/16), causal
    rng = np.random.default_rng(5)
    w = rand_tucker(rng, 128, 4, (2, 16, 16), (2, 16, 16))
    X = rng.standard_normal((64, 128))
    np.testing.assert_allclose(fwd(X, w, causal=True), brute(X, w, causal=True), rtol=0, atol=1e-10)


def test_mode_product_matches_elementwise_definition():
    # (T x_2 M)[a, j, c] = sum_b T[a, b, c] M[j, b], checked entry by entry with python loops
    rng = np.random.default_rng(0)
    T = rng.standard_normal((2, 3, 4))
    for mode, J in ((1, 5), (2, 2), (3, 3)):
        M = rng.standard_normal((J, T.shape[mode - 1]))
        got = O.mode_product(T, M, mode)
        for idx in np.ndindex(*got.shape):
            s = 0.0
            for i in range(T.shape[mode - 1]):
                src = list(idx)
                src[mode - 1] = i
                s += T[tuple(src)] * M[idx[mode - 1], i]
            assert abs(got[idx] - s) < 1e-12


def test_post_softmax_mode_order_transpose_convention():
    # Wt stacks the TRANSPOSED per-head matrices: Wt[h, o, v] = (WV_h WO_h)[v, o].  A swapped
    # output/value mode in the oracle fails here (rectangular t2 != t3 makes the swap visible).
    rng = np.random.default_rng(3)
    d, n_H, N = 6, 2, 4
    w = rand_tucker(rng, d, n_H, (2, 3, 3), (2, 4, 5))
    X = rng.standard_normal((N, d))
    Wt = O.assemble_dense(w["Ct"], w["Ut1"], w["Ut2"], w["Ut3"])       # [h, out, val]
    W = O.assemble_dense(w["C"], w["U1"], w["U2"], w["U3"])
    out = np.zeros((N, d))
    for h in range(n_H):
        S = X @ W[h] @ X.T / np.sqrt(d / n_H)
        P = np.exp(S - S.max(1, keepdims=True))
        P /= P.sum(1, keepdims=True)
        out += P @ X @ Wt[h].T            # X Wtilde_h with Wtilde_h = Wt[h]^T  ([val, out])
    np.testing.assert_allclose(fwd(X, w), out, atol=1e-11, rtol=0)


# --------------------------------------------------------------------------------------
# special cases: MHA, GQA, MQA, MLA (Lemma 1, Theorems 1-3)
# --------------------------------------------------------------------------------------

def _mha_weights(rng, d):
    return [rng.standard_normal((d, d)) / np.sqrt(d) for _ in range(4)]


@pytest.mark.parametrize("causal", [False, True])
def test_mha_reduction(causal):
    rng = np.random.default_rng(21)
    d, n_H, N = 16, 4, 9
    WQ, WK, WV, WO = _mha_weights(rng, d)
    X = rng.standard_normal((N, d))
    w = O.tucker_from_mha(WQ, WK, WV, WO, n_H)
    assert w["C"].shape == (n_H, d, d)
    ref = O.mha_reference(X, WQ, WK, WV, WO, n_H, causal=causal)
    np.testing.assert_allclose(fwd(X, w, causal=causal), ref, atol=1e-11, rtol=0)
    np.testing.assert_allclose(brute(X, w, causal=causal), ref, atol=1e-11, rtol=0)


def test_mha_reference_matches_concat_form():
    # textbook MHA: concat(head_i) W^O, coded here a third way
    rng = np.random.default_rng(22)
    d, n_H, N = 12, 3, 6
    d_H = d // n_H
    WQ, WK, WV, WO = _mha_weights(rng, d)
    X = rng.standard_normal((N, d))
    heads = []
    for i in range(n_H):
        q, k, v = (X @ W[:, i * d_H:(i + 1) * d_H] for W in (WQ, WK, WV))
        s = q @ k.T / np.sqrt(d_H)
        p = np.exp(s) / np.exp(s).sum(1, keepdims=True)
        heads.append(p @ v)
    np.testing.assert_allclose(O.mha_reference(X, WQ, WK, WV, WO, n_H), np.concatenate(heads, 1) @ WO,
                               atol=1e-12, rtol=0)


@pytest.mark.parametrize("n_G", [1, 2])
def test_gqa_mqa_reduction(n_G):
    rng = np.random.default_rng(23)
    d, n_H, N = 16, 4, 8
    d_H = d // n_H
    WQ, _, _, WO = _mha_weights(rng, d)
    WKg = rng.standard_normal((d, n_G * d_H)) / np.sqrt(d)
    WVg = rng.standard_normal((d, n_G * d_H)) / np.sqrt(d)
    X = rng.standard_normal((N, d))
    w = O.tucker_from_gqa(WQ, WKg, WVg, WO, n_H, n_G)
    assert w["C"].shape == (n_H, d, n_G * d_H)           # ranks (n_H, d, n_G d_H)
    ref = O.gqa_reference(X, WQ, WKg, WVg, WO, n_H, n_G, causal=True)
    np.testing.assert_allclose(fwd(X, w, causal=True), ref, atol=1e-11, rtol=0)
    # GQA equals MHA with repeated KV heads
    WK = np.concatenate([WKg[:, O.gqa_group(h, n_H, n_G) * d_H:][:, :d_H] for h in range(n_H)], 1)
    WV = np.concatenate([WVg[:, O.gqa_group(h, n_H, n_G) * d_H:][:, :d_H] for h in range(n_H)], 1)
    np.testing.assert_allclose(ref, O.mha_reference(X, WQ, WK, WV, WO, n_H, causal=True), atol=1e-11, rtol=0)


@pytest.mark.parametrize("shared", [False, True])
def test_mla_reduction(shared):
    rng = np.random.default_rng(24)
    d, n_H, N, cq, ck = 16, 4, 7, 6, 5
    WDQ = rng.standard_normal((d, cq)) / np.sqrt(d)
    WUQ = rng.standard_normal((cq, d)) / np.sqrt(cq)
    WDKV = rng.standard_normal((d, ck)) / np.sqrt(d)
    WUK = rng.standard_normal((ck, d)) / np.sqrt(ck)
    WDV = WDKV if shared else rng.standard_normal((d, ck)) / np.sqrt(d)
    WUV = rng.standard_normal((ck, d)) / np.sqrt(ck)
    WO = rng.standard_normal((d, d)) / np.sqrt(d)
    X = rng.standard_normal((N, d))
    w = O.tucker_from_mla(WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H)
    assert w["C"].shape == (n_H, cq, ck) and w["Ct"].shape == (n_H, d, ck)
    ref = O.mla_reference(X, WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H, causal=True)
    np.testing.assert_allclose(fwd(X, w, causal=True), ref, atol=1e-11, rtol=0)
    # MLA is MHA with the factored weights multiplied out
    ref2 = O.mha_reference(X, WDQ @ WUQ, WDKV @ WUK, WDV @ WUV, WO, n_H, causal=True)
    np.testing.assert_allclose(ref, ref2, atol=1e-11, rtol=0)


# --------------------------------------------------------------------------------------
# RoPE
# --------------------------------------------------------------------------------------

def test_rope_matches_explicit_rotation_matrix():
    # build R(l, r) as an explicit block-diagonal matrix and right-multiply
    r, base = 8, 10000.0
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, r))
    pos = np.array([0, 1, 2, 17, 300])
    got = O.rope_rotate(x, pos, base)
    for n, l in enumerate(pos):
        R = np.zeros((r, r))
        for i in range(r // 2):
            a = l * base ** (-2.0 * i / r)
            R[2 * i, 2 * i], R[2 * i, 2 * i + 1] = np.cos(a), np.sin(a)
            R[2 * i + 1, 2 * i], R[2 * i + 1, 2 * i + 1] = -np.sin(a), np.cos(a)
        np.testing.assert_allclose(got[n], x[n] @ R, atol=1e-12, rtol=0)
        # relative property R(m) R(n)^T = R(m - n), orthogonality, identity at 0
        np.testing.assert_allclose(R @ R.T, np.eye(r), atol=1e-12)
    np.testing.assert_allclose(got[0], x[0], atol=0)
    np.testing.assert_allclose(np.linalg.norm(got, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)


def test_rope_relative_property_on_scores():
    r, base = 6, 500000.0
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, r)), rng.standard_normal((1, r))
    s1 = O.rope_rotate(q, [9], base) @ O.rope_rotate(k, [4], base).T
    s2 = O.rope_rotate(q, [1005], base) @ O.rope_rotate(k, [1000], base).T
    s3 = O.rope_rotate(q, [5], base) @ k.T
    np.testing.assert_allclose(s1, s2, atol=1e-9)
    np.testing.assert_allclose(s1, s3, atol=1e-12)


def test_latent_rope_equals_mqa_with_standard_rope():
    # With r3 = d_H, r2 = d and the selector core C[h, (h,l), l] = 1, latent RoPE in r3 is
    # standard RoPE in the head dimension of MQA (App. C.2).
    rng = np.random.default_rng(31)
    d, n_H, N, base = 16, 4, 10, 10000.0
    d_H = d // n_H
    WQ, _, _, WO = _mha_weights(rng, d)
    WKg = rng.standard_normal((d, d_H)) / np.sqrt(d)
    WVg = rng.standard_normal((d, d_H)) / np.sqrt(d)
    X = rng.standard_normal((N, d))
    w = O.tucker_from_gqa(WQ, WKg, WVg, WO, n_H, 1)
    ref = O.gqa_reference(X, WQ, WKg, WVg, WO, n_H, 1, causal=True, rope=True, rope_base=base, pos0=3)
    got = fwd(X, w, causal=True, rope=True, rope_base=base, pos0=3)
    np.testing.assert_allclose(got, ref, atol=1e-11, rtol=0)
    # and RoPE changes the result (the test is not vacuous)
    assert np.abs(got - fwd(X, w, causal=True)).max() > 1e-3


def test_position_offset_invariance():
    rng = np.random.default_rng(32)
    w = rand_tucker(rng, 12, 3, (2, 6, 8), (2, 5, 4))
    X = rng.standard_normal((2, 9, 12))
    a = fwd(X, w, causal=True, rope=True, rope_base=10000.0, pos0=0)
    b = fwd(X, w, causal=True, rope=True, rope_base=10000.0, pos0=777)
    np.testing.assert_allclose(a, b, atol=1e-9, rtol=0)
    assert np.abs(a - fwd(X, w, causal=True)).max() > 1e-4


# --------------------------------------------------------------------------------------
# softmax, equivariance, causality, closed forms
# --------------------------------------------------------------------------------------

def test_softmax_rows_sum_to_one_and_mask():
    rng = np.random.default_rng(41)
    w = rand_tucker(rng, 12, 3, (2, 6, 6), (2, 5, 4))
    X = rng.standard_normal((8, 12))
    _, parts = fwd(X, w, causal=True, return_parts=True)
    P = parts[0]["P"]                                   # [n_H, N, N]
    np.testing.assert_allclose(P.sum(-1), 1.0, atol=1e-13)
    assert np.all(P[:, np.triu_indices(8, 1)[0], np.triu_indices(8, 1)[1]] == 0.0)
    assert np.all(P[:, 0, 0] == 1.0)                    # first token sees only itself


def test_all_ones_values_closed_form():
    # If every latent value row equals the same vector v, every O_h row is v, so
    # Y rows = (sum_h Gt_h v) Ut2^T -- a closed form that does not involve the softmax.
    rng = np.random.default_rng(42)
    d, n_H = 10, 2
    w = rand_tucker(rng, d, n_H, (2, 4, 4), (2, 3, 5))
    X = rng.standard_normal((6, d))
    v = rng.standard_normal(5)
    w["Ut3"] = np.linalg.pinv(X) @ np.tile(v, (6, 1))   # X Ut3 = rows of v (X has full row rank)
    np.testing.assert_allclose(X @ w["Ut3"], np.tile(v, (6, 1)), atol=1e-10)
    Gt = np.einsum("ha,abc->hbc", w["Ut1"], w["Ct"])
    row = sum(Gt[h] @ v for h in range(n_H)) @ w["Ut2"].T
    np.testing.assert_allclose(fwd(X, w, causal=True), np.tile(row, (6, 1)), atol=1e-9)


def test_single_token_closed_form():
    # N = 1: softmax is 1, Y = x Ut3 (sum_h Gt_h)^T Ut2^T
    rng = np.random.default_rng(43)
    w = rand_tucker(rng, 8, 2, (2, 3, 4), (2, 5, 3))
    x = rng.standard_normal((1, 8))
    Gt = np.einsum("ha,abc->hbc", w["Ut1"], w["Ct"]).sum(0)
    np.testing.assert_allclose(fwd(x, w, causal=True, rope=True), x @ w["Ut3"] @ Gt.T @ w["Ut2"].T, atol=1e-12)


def test_permutation_equivariance_without_mask():
    rng = np.random.default_rng(44)
    w = rand_tucker(rng, 12, 3, (2, 6, 6), (3, 5, 4))
    X = rng.standard_normal((9, 12))
    perm = rng.permutation(9)
    np.testing.assert_allclose(fwd(X[perm], w), fwd(X, w)[perm], atol=1e-12, rtol=0)


def test_causal_prefix_independence():
    rng = np.random.default_rng(45)
    w = rand_tucker(rng, 12, 3, (2, 6, 6), (3, 5, 4))
    X = rng.standard_normal((9, 12))
    X2 = X.copy()
    X2[5:] = rng.standard_normal((4, 12))
    a, b = fwd(X, w, causal=True, rope=True), fwd(X2, w, causal=True, rope=True)
    np.testing.assert_allclose(a[:5], b[:5], atol=1e-13, rtol=0)
    assert np.abs(a[5:] - b[5:]).max() > 1e-3
    np.testing.assert_allclose(fwd(X, w, causal=True, rope=True, rows=[2, 7]), a[[2, 7]], atol=1e-13)


def test_scale_is_inverse_sqrt_head_dim():
    # scale = 1/sqrt(d_model/n_H) regardless of the latent ranks: doubling it by hand must
    # equal multiplying the pre-softmax core by 2
    rng = np.random.default_rng(46)
    d, n_H = 12, 3
    w = rand_tucker(rng, d, n_H, (2, 6, 6), (3, 5, 4))
    X = rng.standard_normal((7, d))
    w2 = dict(w, C=2 * w["C"])
    np.testing.assert_allclose(fwd(X, w, scale=2 / np.sqrt(d / n_H)), fwd(X, w2), atol=1e-12)


def test_orthonormal_projection_statistics():
    # orthonormal factors and X ~ N(0,1) give latent entries ~ N(0,1) (closed form)
    from paper_2603_30033_b200 import workloads as W
    wl = W.get_workload("c2")
    wt = W.make_weights(wl)
    for k in ("U2", "U3", "Ut2", "Ut3", "U1", "Ut1"):
        np.testing.assert_allclose(wt[k].T @ wt[k], np.eye(wt[k].shape[1]), atol=1e-10)
    X = W.make_X(wl, B=1, N=512)[0].astype(np.float64)
    lat = X @ wt["U3"]
    assert abs(lat.mean()) < 0.02 and abs(lat.std() - 1.0) < 0.02
    assert abs(wt["C"].std() - (64 * 64) ** -0.25) < 0.01


# --------------------------------------------------------------------------------------
# decode
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("rope", [False, True])
def test_decode_equals_last_row_of_prefill(rope):
    rng = np.random.default_rng(51)
    d, n_H, L = 12, 3, 9
    w = rand_tucker(rng, d, n_H, (2, 6, 8), (2, 5, 4))
    X = rng.standard_normal((2, L + 1, d))
    Yfull, parts = fwd(X, w, causal=True, rope=rope, rope_base=10000.0, return_parts=True)
    Lmax = L + 3
    Kc = np.zeros((2, Lmax, 8))
    Vc = np.zeros((2, Lmax, 4))
    lens = np.array([L, L - 4])
    for b in range(2):
        Kc[b, :L] = parts[b]["K"][:L]                   # prefill K is stored rotated
        Vc[b, :L] = parts[b]["V"][:L]
    xs = np.stack([X[0, L], X[1, L - 4]])
    y, kn, vn = O.tucker_attn_decode(xs, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"],
                                     w["Ut3"], Kc, Vc, lens, rope=rope, rope_base=10000.0)
    np.testing.assert_allclose(y[0], Yfull[0, L], atol=1e-11, rtol=0)
    np.testing.assert_allclose(y[1], Yfull[1, L - 4], atol=1e-11, rtol=0)
    np.testing.assert_allclose(kn[0], parts[0]["K"][L], atol=1e-12)
    np.testing.assert_allclose(vn[1], parts[1]["V"][L - 4], atol=1e-12)


def test_decode_empty_cache_attends_to_itself():
    rng = np.random.default_rng(52)
    w = rand_tucker(rng, 8, 2, (2, 3, 4), (2, 5, 3))
    x = rng.standard_normal((1, 8))
    y, _, _ = O.tucker_attn_decode(x, w["C"], w["U1"], w["U2"], w["U3"], w["Ct"], w["Ut1"], w["Ut2"], w["Ut3"],
                                   np.zeros((1, 4, 4)), np.zeros((1, 4, 3)), np.array([0]), rope=True)
    Gt = np.einsum("ha,abc->hbc", w["Ut1"], w["Ct"]).sum(0)
    np.testing.assert_allclose(y, x @ w["Ut3"] @ Gt.T @ w["Ut2"].T, atol=1e-12)


# --------------------------------------------------------------------------------------
# printed sizes
# --------------------------------------------------------------------------------------

def _golden():
    out = {}
    with open(os.path.join(GOLDEN, "paper_sizes.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v, _, tol, _ = [s.strip() for s in line.split("|")]
            out[k] = (float(v), float(tol))
    return out


def test_printed_sizes():
    g = _golden()
    MB = 1e6
    layers, d, nH, N = 12, 768, 12, 1024
    got = {
        "gpt2_tucker_8_128_128_params_MB": O.tucker_param_count(d, nH, 8, 128) * layers * 2 / MB,
        "gpt2_tucker_8_128_64_params_MB": O.tucker_param_count_general(d, nH, (8, 128, 64), (8, 128, 64)) * layers * 2 / MB,
        "gpt2_tucker_8_64_64_params_MB": O.tucker_param_count(d, nH, 8, 64) * layers * 2 / MB,
        "gpt2_tucker_r128_cache_MB": O.tucker_kv_cache_elems(N, 128) * layers * 2 / MB,
        "gpt2_tucker_r64_cache_MB": O.tucker_kv_cache_elems(N, 64) * layers * 2 / MB,
        "gpt2_mha_params_MB": O.mha_param_count(d) * layers * 2 / MB,
        "gpt2_mha_cache_MB": O.gqa_kv_cache_elems(N, d, nH, nH) * layers * 2 / MB,
        "gpt2_gqa2_params_MB": O.gqa_param_count(d, nH, 2) * layers * 2 / MB,
        "gpt2_gqa2_cache_MB": O.gqa_kv_cache_elems(N, d, nH, 2) * layers * 2 / MB,
        "gpt2_gqa4_params_MB": O.gqa_param_count(d, nH, 4) * layers * 2 / MB,
    }
    layers, d, nH, N = 16, 2048, 32, 4096
    got.update({
        "llama_tucker_32_128_128_params_M": O.tucker_param_count(d, nH, 32, 128) * layers / MB,
        "llama_tucker_32_128_64_params_M": O.tucker_param_count_general(d, nH, (32, 128, 64), (32, 128, 64)) * layers / MB,
        "llama_tucker_32_64_64_params_M": O.tucker_param_count(d, nH, 32, 64) * layers / MB,
        "llama_tucker_r128_cache_M": O.tucker_kv_cache_elems(N, 128) * layers / MB,
        "llama_tucker_r64_cache_M": O.tucker_kv_cache_elems(N, 64) * layers / MB,
        "llama_mha_params_M": O.mha_param_count(d) * layers / MB,
        "llama_gqa8_cache_M": O.gqa_kv_cache_elems(N, d, nH, 8) * layers / MB,
    })
    # Shakespeare ablation table: shared and separated K,V; parameters in 10^6 bytes, caches in 2^20 bytes
    layers, d, nH, N, MiB = 12, 768, 12, 256, float(1 << 20)
    for r1, r in ((8, 128), (8, 64), (6, 64), (4, 32)):
        got[f"shake_tucker_shared_{r1}_{r}_{r}_params_MB"] = O.tucker_param_count(d, nH, r1, r, shared_kv=True) * layers * 2 / MB
    for r1, r in ((8, 128), (6, 32)):
        got[f"shake_tucker_sep_{r1}_{r}_{r}_params_MB"] = O.tucker_param_count(d, nH, r1, r) * layers * 2 / MB
    for r in (128, 64, 32):
        got[f"shake_tucker_shared_r{r}_cache_MiB"] = O.tucker_kv_cache_elems(N, r, shared_kv=True) * layers * 2 / MiB
    for r in (128, 64):
        got[f"shake_tucker_sep_r{r}_cache_MiB"] = O.tucker_kv_cache_elems(N, r) * layers * 2 / MiB
    got["shake_mha_cache_MiB"] = O.gqa_kv_cache_elems(N, d, nH, nH) * layers * 2 / MiB
    got["shake_gqa1_cache_MiB"] = O.gqa_kv_cache_elems(N, d, nH, 1) * layers * 2 / MiB
    assert set(got) == set(g)
    for k, (val, tol) in g.items():
        assert abs(got[k] - val) <= tol, (k, got[k], val)
    # the general count reduces to the table's formula when all ranks are tied
    assert O.tucker_param_count_general(768, 12, (8, 64, 64), (8, 64, 64)) == O.tucker_param_count(768, 12, 8, 64)

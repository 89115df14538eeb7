"""CPU oracle for Tucker Attention (TEST INFRASTRUCTURE, not a product path).

A plain, slow, fp64 numpy statement of what one Tucker-factorised attention layer computes,
written from the paper's definitions.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this file; the CUDA library never does, and this file imports
nothing from the CUDA package.

Notation (paper, "Notation" paragraph and Table "Summary of notation"):
  X  [N, d_model] one embedded sequence (a leading batch axis B = independent sequences)
  n_H heads, d_H = d_model / n_H
  pre-softmax tensor   W  = C  x_1 U1  x_2 U2  x_3 U3     (Definition 1, Eq. "tucker-rep")
  post-softmax tensor  Wt = Ct x_1 Ut1 x_2 Ut2 x_3 Ut3    (mode 2 = output, mode 3 = value,
                                                          because the transposed per-head
                                                          matrices are stacked, Eq. 3)
Two independent evaluators of the same function are given:
  * tucker_attn_fwd        -- the evaluation order of Sec. 3 ("KV Caching", "Latent RoPE",
                              "Flash Attention / Implementation"): latent projections, head-mode
                              core contraction, per-head queries, (latent RoPE), softmax, PV,
                              output-side factors.
  * tucker_attn_bruteforce -- Eq. (6) "eq_full_rank_MHA" evaluated on the dense n_H x d x d
                              tensors reassembled from the cores and factors with mode products.
plus independent textbook MHA / GQA / MLA evaluators and the constructions that embed them
into Tucker form (Lemma 1, Theorems 1-3), used to pin the evaluators against each other.

Pins (see tests/test_oracle_pins.py): brute force == fast path; MHA / GQA / MQA / MLA
reductions; MQA with standard RoPE in d_H == Tucker with latent RoPE when r3 = d_H;
position-offset invariance; softmax rows sum to one; permutation equivariance; causality;
decode == last row of prefill; printed parameter / cache sizes of the paper's tables
(separated and shared K,V); MLA with RoPE in its key latent (Sec. 3.2.1), written with
explicit rotation matrices, == the Tucker evaluator with latent RoPE on the MLA embedding and
== single-head MHA with standard RoPE when there is one head and no up-projection; shared
latent cache with latent RoPE == the two-cache decode on (rotated, un-rotated) copies; HOSVD:
exact recovery of an exact-rank tensor, orthonormal factors, the truncation error bound,
full-rank round trip of MHA weights, spectra == numpy's singular values of the unfoldings.
Parity unpinned: the paper prints no numeric forward-pass example, so absolute outputs are
pinned only through these identities.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------------
# small tensor helpers (Kolda & Bader conventions, as the paper's Notation paragraph states)
# ----------------------------------------------------------------------------------------

def mode_product(T: np.ndarray, M: np.ndarray, mode: int) -> np.ndarray:
    """n-mode product T x_mode M for a 3-way tensor (mode in {1,2,3}); M is [J, I_mode].
    (T x_n M)[..., j, ...] = sum_i T[..., i, ...] * M[j, i]."""
    ax = mode - 1
    out = np.tensordot(M, T, axes=([1], [ax]))          # new axis first
    return np.moveaxis(out, 0, ax)


def softmax_rows(S: np.ndarray) -> np.ndarray:
    """Row-wise softmax over the last axis; -inf entries get probability zero."""
    m = np.max(S, axis=-1, keepdims=True)
    e = np.exp(S - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def causal_mask(q_pos: np.ndarray, k_pos: np.ndarray) -> np.ndarray:
    """True where the key is NOT visible: key position > query position (the diagonal is
    visible; decoder-only reading of "the last row of the attention matrix", Sec. 3.1)."""
    return k_pos[None, :] > q_pos[:, None]


# ----------------------------------------------------------------------------------------
# RoPE (Sec. 3.2; rotation matrix R(l, r) of Su et al., interleaved pairs)
# ----------------------------------------------------------------------------------------

def rope_rotate(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Right-multiply each row vector x[..., n, :] by R(pos[n], r), r = x.shape[-1] (even).
    R is block diagonal with 2x2 blocks acting on coordinate pairs (2i, 2i+1) with angle
    pos * theta_i, theta_i = base**(-2i/r):
        x'[2i]   = x[2i] cos - x[2i+1] sin
        x'[2i+1] = x[2i] sin + x[2i+1] cos
    so that R(m) R(n)^T = R(m - n) (Eq. "eq_ROPE_condition")."""
    r = x.shape[-1]
    if r % 2:
        raise ValueError("RoPE needs an even rotated dimension")
    i = np.arange(r // 2, dtype=F64)
    theta = np.asarray(base, dtype=F64) ** (-2.0 * i / r)
    ang = np.asarray(pos, dtype=F64)[:, None] * theta[None, :]     # [n, r/2]
    c, s = np.cos(ang), np.sin(ang)
    xe, xo = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x, dtype=F64)
    out[..., 0::2] = xe * c - xo * s
    out[..., 1::2] = xe * s + xo * c
    return out


def rope_matrix(pos: float, r: int, base: float) -> np.ndarray:
    """The dense r x r rotation R(pos, r) itself (row-vector convention x' = x R): 2 x 2 blocks
    [[cos, sin], [-sin, cos]] on coordinate pairs (2i, 2i+1), angle pos * base**(-2i/r).
    Written entry by entry so that it shares nothing with rope_rotate."""
    R = np.zeros((r, r), F64)
    for i in range(r // 2):
        a = float(pos) * float(base) ** (-2.0 * i / r)
        R[2 * i, 2 * i], R[2 * i, 2 * i + 1] = np.cos(a), np.sin(a)
        R[2 * i + 1, 2 * i], R[2 * i + 1, 2 * i + 1] = -np.sin(a), np.cos(a)
    return R


# ----------------------------------------------------------------------------------------
# Evaluator 1: the paper's evaluation order (Sec. 3.1-3.3)
# ----------------------------------------------------------------------------------------

def head_cores(C: np.ndarray, U1: np.ndarray) -> np.ndarray:
    """C x_1 U1: G[h] = sum_a U1[h, a] C[a, :, :]  ("per-head queries", Sec. 3.3)."""
    return mode_product(np.asarray(C, F64), np.asarray(U1, F64), 1)


def tucker_attn_fwd(X, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, *, causal=False, rope=False,
                    rope_base=10000.0, pos0=0, scale=None, rows=None, return_parts=False):
    """Forward of one Tucker attention layer.  X is [N, d] or [B, N, d]; returns Y of the
    same leading shape, [.., N, d] (or [.., len(rows), d] when `rows`, a list of query
    indices, restricts the query rows that are evaluated -- keys/values always span all N).

    Steps, in the paper's order:
      K = X U3, V = X Ut3 (the latent KV cache, Sec. 3.1); Qt = X U2
      Qhat = C x_1 U1 x_2 (X U2)            -> per head h: Qhat_h = Qt G_h     (Def. 2)
      latent RoPE: Qhat_{h,m} R(m, r3), K_n R(n, r3)                            (Eq. 12 / App. C.2)
      S_h = Qhat_h K^T / sqrt(d_H); causal mask; row softmax                    (Eq. 4)
      O_h = P_h V;  Y = sum_h O_h Gt_h^T Ut2^T   (Eqs. 5-6 with Wt = Ct x_j Ut_j: the value
      mode of Gt_h contracts with V, its output mode with Ut2)
    """
    X = np.asarray(X, F64)
    single = X.ndim == 2
    if single:
        X = X[None]
    B, N, d = X.shape
    U1, U2, U3 = (np.asarray(a, F64) for a in (U1, U2, U3))
    Ut1, Ut2, Ut3 = (np.asarray(a, F64) for a in (Ut1, Ut2, Ut3))
    n_H = U1.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d / n_H)
    G = head_cores(C, U1)                       # [n_H, r2, r3]
    Gt = head_cores(Ct, Ut1)                    # [n_H, t2(out), t3(val)]
    q_idx = np.arange(N) if rows is None else np.asarray(rows, dtype=np.int64)
    k_pos = pos0 + np.arange(N)
    q_pos = pos0 + q_idx
    Y = np.empty((B, len(q_idx), d), F64)
    parts = []
    for b in range(B):
        Qt = X[b] @ U2                          # [N, r2]
        K = X[b] @ U3                           # [N, r3]
        V = X[b] @ Ut3                          # [N, t3]
        if rope:
            K = rope_rotate(K, k_pos, rope_base)
        Z = np.zeros((len(q_idx), Ut2.shape[1]), F64)
        P_all = []
        for h in range(n_H):
            Qh = Qt[q_idx] @ G[h]               # [nq, r3]
            if rope:
                Qh = rope_rotate(Qh, q_pos, rope_base)
            S = (Qh @ K.T) * scale
            if causal:
                S = np.where(causal_mask(q_pos, k_pos), -np.inf, S)
            P = softmax_rows(S)
            O = P @ V                           # [nq, t3]
            Z += O @ Gt[h].T                    # [nq, t2]
            if return_parts:
                P_all.append(P)
        Y[b] = Z @ Ut2.T
        if return_parts:
            parts.append({"Qt": Qt, "K": K, "V": V, "P": np.stack(P_all), "Z": Z})
    if single:
        Y = Y[0]
    return (Y, parts) if return_parts else Y


def tucker_attn_decode(x, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, Kc, Vc, cache_len, *, rope=False,
                       rope_base=10000.0, scale=None):
    """One cached decode step (Eq. "eq_kv_caching", read with the pre-softmax core C and the
    output-side factors applied afterwards).  x [B, d]; Kc [B, Lmax, r3] holds rotated latent
    keys K_n R(n) in slots n < cache_len[b]; Vc [B, Lmax, t3].  The new token sits at position
    L = cache_len[b]; it attends to the L cached entries and to itself.
    Returns (y [B, d], k_new [B, r3] (rotated), v_new [B, t3])."""
    x = np.asarray(x, F64)
    B, d = x.shape
    U1, U2, U3 = (np.asarray(a, F64) for a in (U1, U2, U3))
    Ut1, Ut2, Ut3 = (np.asarray(a, F64) for a in (Ut1, Ut2, Ut3))
    n_H = U1.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d / n_H)
    G = head_cores(C, U1)
    Gt = head_cores(Ct, Ut1)
    y = np.empty((B, d), F64)
    k_new = np.empty((B, U3.shape[1]), F64)
    v_new = np.empty((B, Ut3.shape[1]), F64)
    for b in range(B):
        L = int(cache_len[b])
        pos = np.array([L])
        qt = x[b:b + 1] @ U2                     # [1, r2]
        k = x[b:b + 1] @ U3                      # [1, r3]
        v = x[b:b + 1] @ Ut3                     # [1, t3]
        if rope:
            k = rope_rotate(k, pos, rope_base)
        K = np.concatenate([np.asarray(Kc[b, :L], F64), k], axis=0)     # [L+1, r3]
        V = np.concatenate([np.asarray(Vc[b, :L], F64), v], axis=0)     # [L+1, t3]
        z = np.zeros((1, Ut2.shape[1]), F64)
        for h in range(n_H):
            qh = qt @ G[h]
            if rope:
                qh = rope_rotate(qh, pos, rope_base)
            p = softmax_rows((qh @ K.T) * scale)
            z += (p @ V) @ Gt[h].T
        y[b] = (z @ Ut2.T)[0]
        k_new[b], v_new[b] = k[0], v[0]
    return y, k_new, v_new


# ----------------------------------------------------------------------------------------
# Evaluator 2: brute force from the dense tensors (Eqs. 2-6), no RoPE
# ----------------------------------------------------------------------------------------

def assemble_dense(C, U1, U2, U3) -> np.ndarray:
    """C x_1 U1 x_2 U2 x_3 U3 -> dense [n_H, d, d] tensor (Eq. "tucker-rep")."""
    T = np.asarray(C, F64)
    for mode, U in ((1, U1), (2, U2), (3, U3)):
        T = mode_product(T, np.asarray(U, F64), mode)
    return T


def full_rank_mha(X, W, Wt, *, causal=False, scale=None) -> np.ndarray:
    """Eq. (6): Out[j,k] = sum_{i,l} H1[i,j,l] H2[i,k,l] with
    H1 = softmax((W x_2 X x_3 X)/sqrt(d_H)) and H2 = Wt x_3 X, for one sequence X [N, d]."""
    X = np.asarray(X, F64)
    N, d = X.shape
    n_H = W.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d / n_H)
    A = mode_product(mode_product(W, X, 2), X, 3) * scale       # [n_H, N, N]
    if causal:
        pos = np.arange(N)
        A = np.where(causal_mask(pos, pos)[None], -np.inf, A)
    H1 = softmax_rows(A)
    H2 = mode_product(Wt, X, 3)                                 # [n_H, d, N]
    out = np.zeros((N, d), F64)
    for i in range(n_H):
        for l in range(N):
            out += np.outer(H1[i, :, l], H2[i, :, l])
    return out


def tucker_attn_bruteforce(X, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, *, causal=False, scale=None):
    X = np.asarray(X, F64)
    W = assemble_dense(C, U1, U2, U3)
    Wt = assemble_dense(Ct, Ut1, Ut2, Ut3)
    if X.ndim == 2:
        return full_rank_mha(X, W, Wt, causal=causal, scale=scale)
    return np.stack([full_rank_mha(x, W, Wt, causal=causal, scale=scale) for x in X])


# ----------------------------------------------------------------------------------------
# Independent textbook attention variants (Eq. 1 and Sec. 2.2), one sequence X [N, d]
# ----------------------------------------------------------------------------------------

def _attend(Q, K, V, d_H, causal, q_pos=None, k_pos=None):
    S = (Q @ K.T) / np.sqrt(d_H)
    if causal:
        qp = np.arange(Q.shape[0]) if q_pos is None else q_pos
        kp = np.arange(K.shape[0]) if k_pos is None else k_pos
        S = np.where(causal_mask(qp, kp), -np.inf, S)
    return softmax_rows(S) @ V


def mha_reference(X, WQ, WK, WV, WO, n_H, *, causal=False, rope=False, rope_base=10000.0, pos0=0):
    """sum_i softmax(X WQ_i (X WK_i)^T / sqrt(d_H)) X WV_i WO_i with column-split heads
    (Eq. 1); optional standard RoPE in the head dimension (App. C.2, "MHA")."""
    X = np.asarray(X, F64)
    N, d = X.shape
    d_H = d // n_H
    pos = pos0 + np.arange(N)
    out = np.zeros((N, d), F64)
    for i in range(n_H):
        sl = slice(i * d_H, (i + 1) * d_H)
        Q, K, V = X @ WQ[:, sl], X @ WK[:, sl], X @ WV[:, sl]
        if rope:
            Q, K = rope_rotate(Q, pos, rope_base), rope_rotate(K, pos, rope_base)
        out += _attend(Q, K, V, d_H, causal) @ WO[sl, :]
    return out


def gqa_group(h: int, n_H: int, n_G: int) -> int:
    """Head -> KV group map used throughout: contiguous groups."""
    return (h * n_G) // n_H


def gqa_reference(X, WQ, WKg, WVg, WO, n_H, n_G, *, causal=False, rope=False,
                  rope_base=10000.0, pos0=0):
    """GQA: n_H query heads, n_G key/value heads WKg, WVg [d, n_G*d_H]; n_G = 1 is MQA."""
    X = np.asarray(X, F64)
    N, d = X.shape
    d_H = d // n_H
    pos = pos0 + np.arange(N)
    out = np.zeros((N, d), F64)
    for i in range(n_H):
        g = gqa_group(i, n_H, n_G)
        sl, gl = slice(i * d_H, (i + 1) * d_H), slice(g * d_H, (g + 1) * d_H)
        Q, K, V = X @ WQ[:, sl], X @ WKg[:, gl], X @ WVg[:, gl]
        if rope:
            Q, K = rope_rotate(Q, pos, rope_base), rope_rotate(K, pos, rope_base)
        out += _attend(Q, K, V, d_H, causal) @ WO[sl, :]
    return out


def mla_reference(X, WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H, *, causal=False):
    """MLA without RoPE (Sec. 2.2.2): Q_i = X WDQ WUQ_i, K_i = X WDKV WUK_i,
    V_i = X WDV WUV_i (WDV is WDKV for the shared-KV variant), full-rank WO.
    WUQ [dcQ, d], WUK [dcK, d], WUV [dcK, d] are column-split into heads."""
    X = np.asarray(X, F64)
    N, d = X.shape
    d_H = d // n_H
    cq, ckv, cv = X @ WDQ, X @ WDKV, X @ WDV
    out = np.zeros((N, d), F64)
    for i in range(n_H):
        sl = slice(i * d_H, (i + 1) * d_H)
        out += _attend(cq @ WUQ[:, sl], ckv @ WUK[:, sl], cv @ WUV[:, sl], d_H, causal) @ WO[sl, :]
    return out


# ----------------------------------------------------------------------------------------
# Embeddings of MHA / GQA / MLA into Tucker form (Lemma 1, Theorems 1-3)
# ----------------------------------------------------------------------------------------

def tucker_from_mha(WQ, WK, WV, WO, n_H) -> dict:
    """Ranks (n_H, d, d) for both tensors.  U1 = I; U2 = WQ, U3 = WK (head-major columns, so
    the column permutation of Theorem 1 is the identity); selector core of Lemma 1:
    C[i, n, m] = 1 iff n = m lies in head block i.  Post-softmax: Ut3 = WV, Ut2 = WO^T."""
    d = WQ.shape[0]
    d_H = d // n_H
    C = np.zeros((n_H, d, d), F64)
    for i in range(n_H):
        for l in range(d_H):
            C[i, i * d_H + l, i * d_H + l] = 1.0
    eye = np.eye(n_H)
    return dict(C=C, U1=eye, U2=np.asarray(WQ, F64), U3=np.asarray(WK, F64),
                Ct=C.copy(), Ut1=eye.copy(), Ut2=np.asarray(WO, F64).T.copy(),
                Ut3=np.asarray(WV, F64))


def tucker_from_gqa(WQ, WKg, WVg, WO, n_H, n_G) -> dict:
    """Ranks (n_H, d, n_G*d_H) (Theorem 2): the key/value factor holds the n_G shared heads,
    the core routes head i's block to its group's block."""
    d = WQ.shape[0]
    d_H = d // n_H
    C = np.zeros((n_H, d, n_G * d_H), F64)
    for i in range(n_H):
        g = gqa_group(i, n_H, n_G)
        for l in range(d_H):
            C[i, i * d_H + l, g * d_H + l] = 1.0
    eye = np.eye(n_H)
    return dict(C=C, U1=eye, U2=np.asarray(WQ, F64), U3=np.asarray(WKg, F64),
                Ct=C.copy(), Ut1=eye.copy(), Ut2=np.asarray(WO, F64).T.copy(),
                Ut3=np.asarray(WVg, F64))


def tucker_from_mla(WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H) -> dict:
    """Ranks (n_H, dcQ, dcK) and (n_H, d, dcK) (Theorem 3): the up-projections are absorbed
    into the cores: C[i] = WUQ_i WUK_i^T,  Ct[i, o, c] = (WUV_i WO_i)[c, o],  Ut2 = I."""
    d = WDQ.shape[0]
    d_H = d // n_H
    C = np.stack([WUQ[:, i * d_H:(i + 1) * d_H] @ WUK[:, i * d_H:(i + 1) * d_H].T
                  for i in range(n_H)])
    Ct = np.stack([(WUV[:, i * d_H:(i + 1) * d_H] @ WO[i * d_H:(i + 1) * d_H, :]).T
                   for i in range(n_H)])
    eye = np.eye(n_H)
    return dict(C=C, U1=eye, U2=np.asarray(WDQ, F64), U3=np.asarray(WDKV, F64),
                Ct=Ct, Ut1=eye.copy(), Ut2=np.eye(d), Ut3=np.asarray(WDV, F64))


# ----------------------------------------------------------------------------------------
# Size formulas (Table "Comparison of the memory footprint ...")
# ----------------------------------------------------------------------------------------

def tucker_param_count(d, n_H, r1, r, shared_kv=False) -> int:
    """Tucker (separated KV): 2 (n_H r1 + 2 r d + r1 r^2); (shared KV): 2 n_H r1 + 3 r d + 2 r1 r^2."""
    if shared_kv:
        return 2 * n_H * r1 + 3 * r * d + 2 * r1 * r * r
    return 2 * (n_H * r1 + 2 * r * d + r1 * r * r)


def tucker_param_count_general(d, n_H, r, t) -> int:
    """Element count of (C, U1, U2, U3) and (Ct, Ut1, Ut2, Ut3) for arbitrary ranks."""
    r1, r2, r3 = r
    t1, t2, t3 = t
    return (r1 * r2 * r3 + n_H * r1 + d * (r2 + r3)) + (t1 * t2 * t3 + n_H * t1 + d * (t2 + t3))


def tucker_kv_cache_elems(N, r, shared_kv=False) -> int:
    return N * r if shared_kv else 2 * N * r


def mha_param_count(d) -> int:
    return 4 * d * d


def gqa_param_count(d, n_H, n_G) -> int:
    return 2 * d * d + 2 * n_G * (d // n_H) * d


def gqa_kv_cache_elems(N, d, n_H, n_G) -> int:
    return 2 * N * n_G * (d // n_H)


# ----------------------------------------------------------------------------------------
# Shared latent cache with latent RoPE (Sec. 3.1, last paragraph, together with Definition 2)
# ----------------------------------------------------------------------------------------

def tucker_attn_decode_shared_rope(x, C, U1, U2, U3, Ct, Ut1, Ut2, Lc, cache_len, *,
                                   rope_base=10000.0, scale=None):
    """Cached decode step with ONE latent cache L^KV = X U3 (Sec. 3.1: keys and values replaced by
    the shared down-projection, cache size N r3) and latent RoPE (Definition 2).  The paper does
    not say what the single cache holds when the keys are rotated; reading taken here: the cache
    holds the UN-rotated latent rows, the value side uses them as they are, and the key of slot n
    is the cached row times R(n, r3), formed when it is used.  Lc [B, Lmax, r3]; the new token at
    position L = cache_len[b] attends to slots 0..L-1 and to itself.
    Returns (y [B, d], l_new [B, r3] un-rotated latent row of the new token)."""
    x = np.asarray(x, F64)
    B, d = x.shape
    U1, U2, U3 = (np.asarray(a, F64) for a in (U1, U2, U3))
    Ut1, Ut2 = np.asarray(Ut1, F64), np.asarray(Ut2, F64)
    n_H = U1.shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(d / n_H)
    G = head_cores(C, U1)
    Gt = head_cores(Ct, Ut1)
    y = np.empty((B, d), F64)
    l_new = np.empty((B, U3.shape[1]), F64)
    for b in range(B):
        L = int(cache_len[b])
        lat = np.concatenate([np.asarray(Lc[b, :L], F64), x[b:b + 1] @ U3], axis=0)   # [L+1, r3] = V
        K = rope_rotate(lat, np.arange(L + 1), rope_base)
        qt = x[b:b + 1] @ U2
        z = np.zeros((1, Ut2.shape[1]), F64)
        for h in range(n_H):
            qh = rope_rotate(qt @ G[h], np.array([L]), rope_base)
            p = softmax_rows((qh @ K.T) * scale)
            z += (p @ lat) @ Gt[h].T
        y[b] = (z @ Ut2.T)[0]
        l_new[b] = lat[L]
    return y, l_new


# ----------------------------------------------------------------------------------------
# MLA with RoPE in its key latent (Sec. 3.2.1 "Simplified RoPE for MLA"; App. C.2 "MLA - coupled RoPE")
# ----------------------------------------------------------------------------------------

def mla_latent_rope_reference(X, WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, n_H, *, causal=False,
                              rope_base=10000.0, pos0=0):
    """One sequence X [N, d].  Per head i the query-side matrices are fused into
    WQ_i^MLA = WDQ WUQ_i WUK_i^T  [d, dcK]  (the paper prints W^UV_i for the last factor; the
    key up-projection transposed is what makes the product land in the key latent), and
        score_i[m, n] = X_m WQ_i^MLA R(m, dcK) R(n, dcK)^T WDKV^T X_n^T / sqrt(d_H);
    values and output as in MLA without RoPE: V_i = X WDV WUV_i, out = sum_i P_i V_i WO_i.
    Rotations are applied as explicit dense matrices, position by position."""
    X = np.asarray(X, F64)
    N, d = X.shape
    d_H = d // n_H
    dck = WDKV.shape[1]
    Rm = [rope_matrix(pos0 + m, dck, rope_base) for m in range(N)]
    Krot = np.stack([(X[n] @ WDKV) @ Rm[n] for n in range(N)])              # [N, dcK]
    cv = X @ WDV
    out = np.zeros((N, d), F64)
    for i in range(n_H):
        sl = slice(i * d_H, (i + 1) * d_H)
        WQmla = WDQ @ WUQ[:, sl] @ WUK[:, sl].T                             # [d, dcK]
        Qrot = np.stack([(X[m] @ WQmla) @ Rm[m] for m in range(N)])
        S = (Qrot @ Krot.T) / np.sqrt(d_H)
        if causal:
            pos = np.arange(N)
            S = np.where(causal_mask(pos, pos), -np.inf, S)
        out += softmax_rows(S) @ (cv @ WUV[:, sl]) @ WO[sl, :]
    return out


# ----------------------------------------------------------------------------------------
# HOSVD initialiser (App. C.1 "MHA to Tucker Attention"; Sec. 2.1 "Informed Compression Across All Modes")
# ----------------------------------------------------------------------------------------

def mode_unfold(T: np.ndarray, mode: int) -> np.ndarray:
    """Mat_mode(T): the mode-`mode` fibres of a 3-way tensor as columns, [I_mode, prod of the others]."""
    ax = mode - 1
    return np.moveaxis(np.asarray(T, F64), ax, 0).reshape(T.shape[ax], -1)


def mode_spectrum(T: np.ndarray, mode: int) -> np.ndarray:
    """Singular values of Mat_mode(T) divided by the largest (the normalised per-mode spectrum
    that Sec. 2.1 plots to choose the ranks)."""
    s = np.linalg.svd(mode_unfold(T, mode), compute_uv=False)
    return s / s[0]


def hosvd(T: np.ndarray, ranks) -> tuple:
    """Truncated higher-order SVD: factor j = the ranks[j] leading left singular vectors of
    Mat_j(T); core = T x_1 U1^T x_2 U2^T x_3 U3^T.  Returns (core, [U1, U2, U3], [s1, s2, s3])
    with s_j all singular values of Mat_j(T).  T is approximated by core x_1 U1 x_2 U2 x_3 U3 with
    ||T - approx||^2 <= sum_j sum_{k >= ranks[j]} s_j[k]^2."""
    T = np.asarray(T, F64)
    Us, svals = [], []
    for mode in (1, 2, 3):
        U, s, _ = np.linalg.svd(mode_unfold(T, mode), full_matrices=False)
        Us.append(U[:, :ranks[mode - 1]])
        svals.append(s)
    core = T
    for mode in (1, 2, 3):
        core = mode_product(core, Us[mode - 1].T, mode)
    return core, Us, svals


def mha_weight_tensors(WQ, WK, WV, WO, n_H) -> tuple:
    """The two n_H x d x d tensors of Eqs. 2-3: W[i] = WQ_i WK_i^T and the transposed stack
    Wt[i] = (WV_i WO_i)^T (mode 2 = output, mode 3 = value)."""
    d = WQ.shape[0]
    d_H = d // n_H
    W = np.stack([WQ[:, i * d_H:(i + 1) * d_H] @ WK[:, i * d_H:(i + 1) * d_H].T for i in range(n_H)])
    Wt = np.stack([(WV[:, i * d_H:(i + 1) * d_H] @ WO[i * d_H:(i + 1) * d_H, :]).T for i in range(n_H)])
    return W.astype(F64), Wt.astype(F64)


def mha_to_tucker(WQ, WK, WV, WO, n_H, r, t) -> dict:
    """MHA weights -> Tucker-attention weights by HOSVD of the two weight tensors (App. C.1)."""
    W, Wt = mha_weight_tensors(np.asarray(WQ, F64), np.asarray(WK, F64), np.asarray(WV, F64), np.asarray(WO, F64), n_H)
    C, (U1, U2, U3), sv = hosvd(W, r)
    Ct, (Ut1, Ut2, Ut3), svt = hosvd(Wt, t)
    return dict(C=C, U1=U1, U2=U2, U3=U3, Ct=Ct, Ut1=Ut1, Ut2=Ut2, Ut3=Ut3, spectra=sv, spectra_t=svt)

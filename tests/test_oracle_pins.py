"""Pins for the fp64 oracle: each test ties it to something the paper or plain mathematics fixes,
never to itself.  All run on CPU in well under a minute."""
import json
import os

import numpy as np
import pytest

import oracle
from tests import paper_forms as pfm

HERE = os.path.dirname(os.path.abspath(__file__))
TOL = 1e-12


def rnd(seed):
    return np.random.default_rng(seed)


def unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def make(seed, L, r, d_k, d_v, B=1, H=1, beta_hi=1.0, s0=True):
    g = rnd(seed)
    q = g.standard_normal((B, H, L, d_k)).astype(np.float32)
    k = unit(g.standard_normal((B, H, L, r, d_k))).astype(np.float32)
    v = g.standard_normal((B, H, L, r, d_v)).astype(np.float32)
    beta = (beta_hi * g.uniform(0.05, 0.95, (B, H, L, r))).astype(np.float32)
    S0 = g.standard_normal((B, H, d_k, d_v)) if s0 else None
    return q, k, v, beta, S0


def f64(*xs):
    return [None if x is None else np.asarray(x, dtype=np.float64) for x in xs]


# --- worked examples (tests/golden/worked_examples.json: hand arithmetic on the recurrence) -----

def test_hand_worked_examples():
    with open(os.path.join(HERE, "golden", "worked_examples.json")) as f:
        data = json.load(f)
    assert len(data["examples"]) >= 2
    for ex in data["examples"]:
        q = np.array(ex["q"], dtype=np.float32)[None, None]
        k = np.array(ex["k"], dtype=np.float32)[None, None]
        v = np.array(ex["v"], dtype=np.float32)[None, None]
        beta = np.array(ex["beta"], dtype=np.float32)[None, None]
        S0 = None if ex["S0"] is None else np.array(ex["S0"], dtype=np.float64)[None, None]
        O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
        # every input is a binary fraction: the fp64 result is exact
        np.testing.assert_allclose(O[0, 0], np.array(ex["O"]), rtol=0, atol=1e-15, err_msg=ex["name"])
        np.testing.assert_allclose(Sf[0, 0], np.array(ex["S_final"]), rtol=0, atol=1e-15, err_msg=ex["name"])


# --- P1: with no delta term the recurrence is causal linear attention (Section 1.2) -------------

def test_linear_attention_special_case():
    # keys orthonormal across the whole sequence and S0 = 0  =>  S_{t-1} k_{t,j} = 0 for every t,j,
    # so O = (Q K^T . Mincl) diag(beta) V with the inclusive causal mask over rows m = t*r + j.
    L, r, d_k, d_v = 6, 2, 16, 5
    g = rnd(1)
    Qm, _ = np.linalg.qr(g.standard_normal((d_k, d_k)))
    k = Qm[: L * r].reshape(1, 1, L, r, d_k)
    # fp32 storage makes the keys orthonormal only to 1e-7: keep the comparison at that level
    k32 = k.astype(np.float32)
    q = g.standard_normal((1, 1, L, d_k)).astype(np.float32)
    v = g.standard_normal((1, 1, L, r, d_v)).astype(np.float32)
    beta = g.uniform(0.1, 1.9, (1, 1, L, r)).astype(np.float32)
    O, Sf = oracle.deltanet_fwd(q, k32, v, beta, None)
    K = k32.reshape(L * r, d_k).astype(np.float64)
    V = v.reshape(L * r, d_v).astype(np.float64)
    b = beta.reshape(L * r).astype(np.float64)
    tok = np.arange(L * r) // r
    mask = tok[None, :] <= np.arange(L)[:, None]
    O_lin = ((q[0, 0].astype(np.float64) @ K.T) * mask) @ (b[:, None] * V)
    np.testing.assert_allclose(O[0, 0], O_lin, rtol=0, atol=5e-6)
    np.testing.assert_allclose(Sf[0, 0], ((b[:, None] * V).T @ K).T, rtol=0, atol=5e-6)


def test_linear_attention_exact_with_axis_keys():
    # same statement with keys = distinct coordinate vectors: orthonormal exactly, so it is exact.
    L, r, d_k, d_v = 5, 3, 15, 4
    g = rnd(2)
    perm = g.permutation(d_k)
    k = np.zeros((1, 1, L, r, d_k), dtype=np.float32)
    for m in range(L * r):
        k[0, 0, m // r, m % r, perm[m]] = 1.0
    q = g.standard_normal((1, 1, L, d_k)).astype(np.float32)
    v = g.standard_normal((1, 1, L, r, d_v)).astype(np.float32)
    beta = g.uniform(0.1, 1.9, (1, 1, L, r)).astype(np.float32)
    O, _ = oracle.deltanet_fwd(q, k, v, beta, None)
    K, V, b = f64(k.reshape(L * r, d_k), v.reshape(L * r, d_v), beta.reshape(L * r))
    tok = np.arange(L * r) // r
    mask = tok[None, :] <= np.arange(L)[:, None]
    O_lin = ((q[0, 0].astype(np.float64) @ K.T) * mask) @ (b[:, None] * V)
    np.testing.assert_allclose(O[0, 0], O_lin, rtol=0, atol=TOL)


# --- P2: beta = 0 leaves the state alone ---------------------------------------------------------

def test_beta_zero_keeps_state():
    q, k, v, beta, S0 = make(3, L=9, r=2, d_k=6, d_v=4, B=2, H=2)
    beta[:] = 0
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    np.testing.assert_allclose(Sf, S0, rtol=0, atol=0)
    # o_t = S0 q_t with S = S0^T (d_v x d_k)
    np.testing.assert_allclose(O, np.einsum("bhij,bhti->bhtj", S0, q.astype(np.float64)), rtol=0, atol=TOL)


# --- P3: beta = 1, unit key: the update is a projection; S_t k_t = v_t ---------------------------

def test_projection_property():
    L, d_k, d_v = 7, 8, 5
    q, k, v, beta, S0 = make(4, L=L, r=1, d_k=d_k, d_v=d_v)
    beta[:] = 1.0
    S = S0.copy()
    for t in range(L):      # one token per call, state threaded through S_final -> S0
        sl = slice(t, t + 1)
        _, S_new = oracle.deltanet_fwd(q[:, :, sl], k[:, :, sl], v[:, :, sl], beta[:, :, sl], S)
        kt = k[0, 0, t, 0].astype(np.float64)
        kt_n2 = kt @ kt                     # fp32-stored unit key: norm^2 = 1 + O(1e-7)
        Sk_new = S_new[0, 0].T @ kt
        Sk_old = S[0, 0].T @ kt
        # general identity  S_t k = S_{t-1} k (1 - beta |k|^2) + beta v |k|^2
        np.testing.assert_allclose(Sk_new, Sk_old * (1 - kt_n2) + v[0, 0, t, 0] * kt_n2, rtol=0, atol=TOL)
        np.testing.assert_allclose(Sk_new, v[0, 0, t, 0], rtol=0, atol=5e-6)   # projection: S_t k_t = v_t
        # directions orthogonal to k are untouched
        w = rnd(100 + t).standard_normal(d_k)
        w -= (w @ kt) / kt_n2 * kt
        np.testing.assert_allclose(S_new[0, 0].T @ w, S[0, 0].T @ w, rtol=0, atol=1e-11)
        S = S_new


def test_partial_beta_interpolates():
    # S_t k_t = (1 - beta) S_{t-1} k_t + beta v_t for a unit key (exact axis key)
    d_k, d_v = 5, 3
    g = rnd(5)
    S0 = g.standard_normal((1, 1, d_k, d_v))
    k = np.zeros((1, 1, 1, 1, d_k), dtype=np.float32)
    k[..., 2] = 1
    v = g.standard_normal((1, 1, 1, 1, d_v)).astype(np.float32)
    beta = np.full((1, 1, 1, 1), 0.25, dtype=np.float32)
    q = g.standard_normal((1, 1, 1, d_k)).astype(np.float32)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    np.testing.assert_allclose(Sf[0, 0, 2], 0.75 * S0[0, 0, 2] + 0.25 * v[0, 0, 0, 0], rtol=0, atol=TOL)
    np.testing.assert_allclose(np.delete(Sf[0, 0], 2, axis=0), np.delete(S0[0, 0], 2, axis=0), rtol=0, atol=0)


# --- P4: beta = 2, unit key, v = 0: a Householder reflection -------------------------------------

def test_reflection_property():
    d_k, d_v = 6, 4
    g = rnd(6)
    S0 = g.standard_normal((1, 1, d_k, d_v))
    # a unit key that is exact in fp32: four entries of 0.5
    k = np.zeros((1, 1, 2, 1, d_k), dtype=np.float32)
    k[0, 0, :, 0, 0] = 0.5
    k[0, 0, :, 0, 1] = 0.5
    k[0, 0, :, 0, 2] = 0.5
    k[0, 0, :, 0, 3] = 0.5             # norm exactly 1
    v = np.zeros((1, 1, 2, 1, d_v), dtype=np.float32)
    beta = np.full((1, 1, 2, 1), 2.0, dtype=np.float32)
    q = g.standard_normal((1, 1, 2, d_k)).astype(np.float32)
    _, S1 = oracle.deltanet_fwd(q[:, :, :1], k[:, :, :1], v[:, :, :1], beta[:, :, :1], S0)
    # rows of S (d_v x d_k) keep their norm under an orthogonal A_t
    np.testing.assert_allclose(np.linalg.norm(S1[0, 0], axis=0), np.linalg.norm(S0[0, 0], axis=0), rtol=1e-13)
    assert np.abs(S1 - S0).max() > 0.1
    # reflecting twice is the identity
    _, S2 = oracle.deltanet_fwd(q, k, v, beta, S0)
    np.testing.assert_allclose(S2, S0, rtol=0, atol=1e-14)


# --- P5: closed form -- all keys e_1: an exponential moving average in one column ---------------

def test_ema_closed_form():
    L, d_k, d_v = 11, 4, 3
    g = rnd(7)
    S0 = g.standard_normal((1, 1, d_k, d_v))
    k = np.zeros((1, 1, L, 1, d_k), dtype=np.float32)
    k[..., 1] = 1.0
    v = g.standard_normal((1, 1, L, 1, d_v)).astype(np.float32)
    beta = g.uniform(0, 1, (1, 1, L, 1)).astype(np.float32)
    q = g.standard_normal((1, 1, L, d_k)).astype(np.float32)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    s = S0[0, 0, 1].copy()
    S = S0[0, 0].copy()
    for t in range(L):
        b = float(beta[0, 0, t, 0])
        s = (1 - b) * s + b * v[0, 0, t, 0].astype(np.float64)
        S[1] = s
        np.testing.assert_allclose(O[0, 0, t], S.T @ q[0, 0, t].astype(np.float64), rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf[0, 0, 1], s, rtol=0, atol=TOL)
    np.testing.assert_allclose(np.delete(Sf[0, 0], 1, axis=0), np.delete(S0[0, 0], 1, axis=0), rtol=0, atol=0)


# --- P6: brute force with explicit d x d products ------------------------------------------------

@pytest.mark.parametrize("r", [1, 2, 3])
def test_brute_force_products(r):
    L, d_k, d_v = 5, 4, 3
    q, k, v, beta, S0 = make(8 + r, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=2.0)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    kk, vv, bb, qq = f64(k[0, 0], v[0, 0], beta[0, 0], q[0, 0])
    mats = [pfm.token_matrices(kk[t], vv[t], bb[t]) for t in range(L)]
    S_start = S0[0, 0].T
    for T in range(1, L + 1):
        # S_T = S0 prod_{t<T} A_t + sum_t X_t prod_{t<s<T} A_s
        prod_all = np.eye(d_k)
        for t in range(T):
            prod_all = prod_all @ mats[t][0]
        S_T = S_start @ prod_all
        for t in range(T):
            tail = np.eye(d_k)
            for s in range(t + 1, T):
                tail = tail @ mats[s][0]
            S_T = S_T + mats[t][1] @ tail
        np.testing.assert_allclose(O[0, 0, T - 1], S_T @ qq[T - 1], rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf[0, 0], S_T.T, rtol=0, atol=TOL)


# --- P7: flows compose (Proposition 2.1); splitting a call changes nothing -----------------------

def test_flow_composition_and_split_invariance():
    L, r, d_k, d_v = 24, 2, 6, 5
    q, k, v, beta, S0 = make(12, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.5)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    kk, vv, bb = f64(k[0, 0], v[0, 0], beta[0, 0])
    for chunk in (4, 7, 24):
        S = S0[0, 0].T.copy()
        for c0 in range(0, L, chunk):
            P, Xi = pfm.interval_flow(kk[c0:c0 + chunk], vv[c0:c0 + chunk], bb[c0:c0 + chunk])
            S = S @ P + Xi
        np.testing.assert_allclose(Sf[0, 0], S.T, rtol=0, atol=TOL)
    # two calls, state threaded through
    L1 = 10
    O1, S_mid = oracle.deltanet_fwd(q[:, :, :L1], k[:, :, :L1], v[:, :, :L1], beta[:, :, :L1], S0)
    O2, S_end = oracle.deltanet_fwd(q[:, :, L1:], k[:, :, L1:], v[:, :, L1:], beta[:, :, L1:], S_mid)
    np.testing.assert_allclose(np.concatenate([O1, O2], axis=2), O, rtol=0, atol=TOL)
    np.testing.assert_allclose(S_end, Sf, rtol=0, atol=TOL)


# --- P8: Theorem 3.2 (library triangular solve), the block inverse, Theorem 3.3 -------------------

@pytest.mark.parametrize("C,r,d_k,d_v", [(7, 1, 5, 4), (6, 3, 5, 4), (8, 2, 4, 6)])
def test_theorem_3_2_matches_recurrence(C, r, d_k, d_v):
    q, k, v, beta, S0 = make(20 + r, L=C, r=r, d_k=d_k, d_v=d_v, beta_hi=2.0)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    kk, vv, bb = f64(k[0, 0], v[0, 0], beta[0, 0])
    S1 = pfm.thm32_chunk_state(kk, vv, bb, S0[0, 0].T)
    np.testing.assert_allclose(Sf[0, 0], S1.T, rtol=0, atol=TOL)
    # using W S0 instead of W S0^T (possible only when d_k = d_v) must NOT agree: guards the transpose
    if d_k == d_v:
        pytest.skip("square case handled in test_state_transpose_matters")


def test_state_transpose_matters():
    C, r, d = 5, 2, 4
    q, k, v, beta, S0 = make(31, L=C, r=r, d_k=d, d_v=d, beta_hi=1.0)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    kk, vv, bb = f64(k[0, 0], v[0, 0], beta[0, 0])
    A, At, Bm = pfm.drivers(kk, vv, bb)
    W, U, _ = pfm.thm32_WU(A, At, Bm)
    S = S0[0, 0].T
    right = S + (U + W @ S.T).T @ Bm.reshape(C * r, d)
    wrong = S + (U + W @ S).T @ Bm.reshape(C * r, d)
    np.testing.assert_allclose(Sf[0, 0], right.T, rtol=0, atol=TOL)
    assert np.abs(Sf[0, 0] - wrong.T).max() > 1e-3


def test_block_triangular_inverse_and_thm_3_3():
    C, r, d = 6, 3, 5
    g = rnd(40)
    kk = unit(g.standard_normal((C, r, d)))
    vv = g.standard_normal((C, r, d))
    bb = g.uniform(0.1, 1.9, (C, r))
    A, At, Bm = pfm.drivers(kk, vv, bb)
    W, U, Cmat = pfm.thm32_WU(A, At, Bm)
    D = pfm.block_triangular_inverse(Cmat, C, r)
    np.testing.assert_allclose(D @ Cmat, np.eye(C * r), rtol=0, atol=1e-13)
    # diagonal R x R blocks of C are the identity (proof of Theorem 3.2)
    for t in range(C):
        np.testing.assert_allclose(Cmat[t * r:(t + 1) * r, t * r:(t + 1) * r], np.eye(r), rtol=0, atol=0)
    np.testing.assert_allclose(D @ A.reshape(C * r, d), W, rtol=0, atol=1e-13)
    W33 = pfm.thm33_W(A, Bm).reshape(C * r, d)
    np.testing.assert_allclose(W33, W, rtol=0, atol=1e-12)


# --- chunk-form forward (the formulas the kernels implement) against the recurrence --------------

@pytest.mark.parametrize("L,r,d_k,d_v,chunk", [(37, 1, 8, 6, 8), (29, 3, 6, 8, 5), (64, 2, 8, 8, 16)])
def test_chunk_form_outputs_match_recurrence(L, r, d_k, d_v, chunk):
    q, k, v, beta, S0 = make(50 + r, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=2.0)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    qq, kk, vv, bb = f64(q[0, 0], k[0, 0], v[0, 0], beta[0, 0])
    O2, Sf2, _ = pfm.chunked_forward(qq, kk, vv, bb, S0[0, 0], chunk)
    np.testing.assert_allclose(O[0, 0], O2, rtol=0, atol=1e-11)
    np.testing.assert_allclose(Sf[0, 0], Sf2, rtol=0, atol=1e-11)


# --- P9: the r factors of a token commute (sum form); zero-beta factors drop out ------------------

def test_factor_permutation_invariance_and_rank_reduction():
    L, r, d_k, d_v = 9, 3, 6, 5
    q, k, v, beta, S0 = make(60, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.5)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    perm = [2, 0, 1]
    O2, Sf2 = oracle.deltanet_fwd(q, k[:, :, :, perm], v[:, :, :, perm], beta[:, :, :, perm], S0)
    np.testing.assert_allclose(O2, O, rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf2, Sf, rtol=0, atol=TOL)
    beta0 = beta.copy()
    beta0[..., 1:] = 0
    O3, Sf3 = oracle.deltanet_fwd(q, k, v, beta0, S0)
    O4, Sf4 = oracle.deltanet_fwd(q, k[:, :, :, :1], v[:, :, :, :1], beta[:, :, :, :1], S0)
    np.testing.assert_allclose(O3, O4, rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf3, Sf4, rtol=0, atol=TOL)


def test_sum_form_differs_from_sequential_factors():
    # r = 2 in one token must NOT equal two rank-1 tokens in sequence (that is the product form)
    d_k, d_v = 4, 3
    q, k, v, beta, S0 = make(61, L=1, r=2, d_k=d_k, d_v=d_v)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    k2 = k.reshape(1, 1, 2, 1, d_k)
    v2 = v.reshape(1, 1, 2, 1, d_v)
    b2 = beta.reshape(1, 1, 2, 1)
    q2 = np.repeat(q, 2, axis=2)
    _, Sf_prod = oracle.deltanet_fwd(q2, k2, v2, b2, S0)
    assert np.abs(Sf - Sf_prod).max() > 1e-3


# --- P10: linearity in (V, S0) and in q ------------------------------------------------------------

def test_linearity():
    q, k, v, beta, S0 = make(70, L=8, r=2, d_k=5, d_v=4, B=1, H=2)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    a = 4.0                                   # power of two: scaling fp32 inputs is exact
    O2, Sf2 = oracle.deltanet_fwd(q, k, a * v, beta, a * S0)
    np.testing.assert_allclose(O2, a * O, rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf2, a * Sf, rtol=0, atol=TOL)
    O3, Sf3 = oracle.deltanet_fwd(2.0 * q, k, v, beta, S0)
    np.testing.assert_allclose(O3, 2.0 * O, rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf3, Sf, rtol=0, atol=0)


# --- layout: batch/head independence and the [d_k, d_v] state layout ------------------------------

def test_batch_head_independence_and_threads():
    q, k, v, beta, S0 = make(80, L=6, r=2, d_k=4, d_v=3, B=2, H=3)
    O, Sf, used = oracle.deltanet_fwd(q, k, v, beta, S0, num_threads=3, return_threads=True)
    assert 1 <= used <= 3
    for b in range(2):
        for h in range(3):
            Ob, Sb = oracle.deltanet_fwd(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], v[b:b + 1, h:h + 1],
                                         beta[b:b + 1, h:h + 1], S0[b:b + 1, h:h + 1], num_threads=1)
            np.testing.assert_allclose(O[b, h], Ob[0, 0], rtol=0, atol=0)
            np.testing.assert_allclose(Sf[b, h], Sb[0, 0], rtol=0, atol=0)


def test_empty_sequence_returns_S0():
    q, k, v, beta, S0 = make(81, L=0, r=2, d_k=4, d_v=3)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0)
    assert O.shape == (1, 1, 0, 3)
    np.testing.assert_allclose(Sf, S0, rtol=0, atol=0)


# --- product form: the r factors of a token act one after another -------------------------------------
# (rank-1 delta rule of Section 1.3, r times per token; the chunk form is the general block-triangular case
# of Theorem 3.2 with the mask strict in the flattened row index)

def test_product_form_is_rank1_deltanet_on_the_interleaved_sequence():
    # the sum-form oracle with r = 1 (pinned by everything above) on the L*r factors, read out every r-th step
    L, r, d_k, d_v = 7, 3, 6, 5
    q, k, v, beta, S0 = make(80, L=L, r=r, d_k=d_k, d_v=d_v, B=1, H=2, beta_hi=1.8)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0, mode="product")
    k1 = k.reshape(1, 2, L * r, 1, d_k)
    v1 = v.reshape(1, 2, L * r, 1, d_v)
    b1 = beta.reshape(1, 2, L * r, 1)
    q1 = np.repeat(q, r, axis=2)
    O1, Sf1 = oracle.deltanet_fwd(q1, k1, v1, b1, S0)
    np.testing.assert_allclose(O, O1[:, :, r - 1::r], rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf, Sf1, rtol=0, atol=TOL)


def test_product_form_brute_force_matrices():
    # explicit d_k x d_k transition matrices, multiplied out in numpy
    L, r, d_k, d_v = 5, 2, 4, 3
    q, k, v, beta, S0 = make(81, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.9)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0, mode="product")
    qd, kd, vd, bd, s0 = f64(q[0, 0], k[0, 0], v[0, 0], beta[0, 0], S0[0, 0])
    S = s0.T.copy()
    for t in range(L):
        for j in range(r):
            kk, vv, b = kd[t, j], vd[t, j], bd[t, j]
            S = S @ (np.eye(d_k) - b * np.outer(kk, kk)) + b * np.outer(vv, kk)
        np.testing.assert_allclose(O[0, 0, t], S @ qd[t], rtol=0, atol=TOL)
    np.testing.assert_allclose(Sf[0, 0], S.T, rtol=0, atol=TOL)


def test_product_equals_sum_when_a_tokens_keys_are_orthogonal():
    # (I - b1 k1 k1^T)(I - b2 k2 k2^T) = I - b1 k1 k1^T - b2 k2 k2^T  and  v1 k1^T (I - b2 k2 k2^T) = v1 k1^T
    L, r, d_k, d_v = 6, 3, 8, 4
    q, k, v, beta, S0 = make(82, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.5)
    g = rnd(83)
    for t in range(L):
        Qm, _ = np.linalg.qr(g.standard_normal((d_k, d_k)))
        k[0, 0, t] = Qm[:r].astype(np.float32)
    # float32 rounding leaves the keys orthogonal only to ~1e-7: compare at that level
    O_s, Sf_s = oracle.deltanet_fwd(q, k, v, beta, S0)
    O_p, Sf_p = oracle.deltanet_fwd(q, k, v, beta, S0, mode="product")
    np.testing.assert_allclose(O_p, O_s, rtol=0, atol=5e-6)
    np.testing.assert_allclose(Sf_p, Sf_s, rtol=0, atol=5e-6)


def test_product_form_depends_on_factor_order_and_r1_is_the_sum_form():
    L, r, d_k, d_v = 6, 2, 5, 4
    q, k, v, beta, S0 = make(84, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.5)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0, mode="product")
    _, Sf_swapped = oracle.deltanet_fwd(q, k[:, :, :, ::-1], v[:, :, :, ::-1], beta[:, :, :, ::-1], S0, mode="product")
    assert np.abs(Sf - Sf_swapped).max() > 1e-3
    _, Sf_sum = oracle.deltanet_fwd(q, k, v, beta, S0)
    assert np.abs(Sf - Sf_sum).max() > 1e-3
    O1, S1 = oracle.deltanet_fwd(q, k[:, :, :, :1], v[:, :, :, :1], beta[:, :, :, :1], S0)
    O2, S2 = oracle.deltanet_fwd(q, k[:, :, :, :1], v[:, :, :, :1], beta[:, :, :, :1], S0, mode="product")
    np.testing.assert_array_equal(O1, O2)
    np.testing.assert_array_equal(S1, S2)


def test_product_form_is_contractive_for_beta_in_0_2():
    # unit keys, v = 0: every factor I - b k k^T has norm <= 1 for b in [0, 2], and is orthogonal for b = 2
    L, r, d_k, d_v = 40, 3, 6, 5
    q, k, v, beta, S0 = make(85, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=2.0)
    k = unit(k)
    v = np.zeros_like(v)
    norms = [np.linalg.norm(f64(S0[0, 0])[0])]
    for t in range(1, L + 1):
        _, Sf = oracle.deltanet_fwd(q[:, :, :t], k[:, :, :t], v[:, :, :t], beta[:, :, :t], S0, mode="product")
        norms.append(np.linalg.norm(Sf[0, 0]))
    assert all(b <= a * (1 + 1e-6) for a, b in zip(norms, norms[1:]))
    beta2 = np.full_like(beta, 2.0)
    _, Sf2 = oracle.deltanet_fwd(q, k, v, beta2, S0, mode="product")
    np.testing.assert_allclose(np.linalg.norm(Sf2[0, 0]), norms[0], rtol=1e-5)


@pytest.mark.parametrize("L,r,d_k,d_v,chunk", [(37, 2, 6, 5, 8), (50, 3, 8, 8, 16), (16, 4, 4, 6, 16)])
def test_chunk_form_with_flattened_mask_matches_product_recurrence(L, r, d_k, d_v, chunk):
    q, k, v, beta, S0 = make(86, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.7)
    O, Sf = oracle.deltanet_fwd(q, k, v, beta, S0, mode="product")
    qd, kd, vd, bd, s0 = f64(q[0, 0], k[0, 0], v[0, 0], beta[0, 0], S0[0, 0])
    O_c, Sf_c, _ = pfm.chunked_forward(qd, kd, vd, bd, s0, chunk, product=True)
    np.testing.assert_allclose(O_c, O[0, 0], rtol=0, atol=1e-11)
    np.testing.assert_allclose(Sf_c, Sf[0, 0], rtol=0, atol=1e-11)


# --- exact step of a rank-1 factor ("An alternative representation of the flow as product of exponentials") -----

def test_exact_step_is_the_matrix_exponential():
    # one token, v = 0: S_1 = S_0 exp(-beta k k^T), with the exponential from a library routine
    import scipy.linalg
    d_k, d_v = 6, 4
    q, k, v, beta, S0 = make(90, L=1, r=1, d_k=d_k, d_v=d_v, beta_hi=3.0)
    k = (k * 1.7).astype(np.float32)              # not unit norm: |k|^2 must enter the formula
    v = np.zeros_like(v)
    _, Sf = oracle.deltanet_fwd(q, k, v, beta, S0, exact=True)
    kd, bd, s0 = f64(k[0, 0, 0, 0], beta[0, 0, 0, 0], S0[0, 0])
    want = s0.T @ scipy.linalg.expm(-bd * np.outer(kd, kd))
    np.testing.assert_allclose(Sf[0, 0], want.T, rtol=0, atol=TOL)


@pytest.mark.parametrize("mode,r", [("sum", 1), ("product", 3)])
def test_exact_step_is_the_limit_of_many_small_euler_steps(mode, r):
    # a token split into N sub-steps of size beta / N (same k, v) is the Euler scheme on a finer grid: it converges,
    # with error O(1/N), to the exact step -- for the input term as well as for the transition
    L, d_k, d_v = 4, 5, 4
    q, k, v, beta, S0 = make(91, L=L, r=r, d_k=d_k, d_v=d_v, beta_hi=1.5)
    k = (k * 1.3).astype(np.float32)
    O_x, Sf_x = oracle.deltanet_fwd(q, k, v, beta, S0, mode=mode, exact=True)
    errs = []
    for N in (200, 400):
        # flatten to rank-1 factors, repeat each N times with beta / N: sub-steps act one after another
        kf = np.repeat(k.reshape(1, 1, L * r, 1, d_k), N, axis=2)
        vf = np.repeat(v.reshape(1, 1, L * r, 1, d_v), N, axis=2)
        bf = np.repeat(beta.reshape(1, 1, L * r, 1).astype(np.float64) / N, N, axis=2).astype(np.float32)
        qf = np.repeat(q, r * N, axis=2)
        O_e, Sf_e = oracle.deltanet_fwd(qf, kf, vf, bf, S0)
        errs.append(max(np.abs(O_e[:, :, r * N - 1::r * N] - O_x).max(), np.abs(Sf_e - Sf_x).max()))
    assert errs[1] < 2e-2 and errs[1] < 0.6 * errs[0], errs      # first order in 1/N


def test_exact_step_small_beta_limit_and_rank_restriction():
    q, k, v, beta, S0 = make(92, L=6, r=1, d_k=5, d_v=4, beta_hi=1e-4)
    O_e, Sf_e = oracle.deltanet_fwd(q, k, v, beta, S0)
    O_x, Sf_x = oracle.deltanet_fwd(q, k, v, beta, S0, exact=True)
    np.testing.assert_allclose(O_x, O_e, rtol=0, atol=1e-7)       # beta' = beta (1 - beta |k|^2 / 2 + ...)
    q, k, v, beta, S0 = make(93, L=3, r=2, d_k=5, d_v=4)
    with pytest.raises(RuntimeError):
        oracle.deltanet_fwd(q, k, v, beta, S0, exact=True)        # sum form with r > 1: not rank 1
    k0 = np.zeros_like(k[:, :, :, :1])
    O_z, Sf_z = oracle.deltanet_fwd(q, k0, v[:, :, :, :1], beta[:, :, :, :1], S0, exact=True)
    np.testing.assert_allclose(Sf_z, S0, rtol=0, atol=0)          # k = 0: nothing changes, no division by zero

"""Independent fp64 numpy evaluations of the paper's closed forms, used only by the tests.

These are second opinions for the token-by-token oracle: they reach the same numbers through the
compact W/U chunk form (Theorem 3.2), the block-triangular inverse (Proposition "Triangular Tensor
Inversion"), the two-index wavefront system (Theorem 3.3) and flow composition (Proposition 2.1).
They call neither the oracle nor the CUDA path.
"""
from __future__ import annotations

import numpy as np
import scipy.linalg


def drivers(k, v, beta):
    """Rank-R drivers of Eq. (discretization) for one chunk, stacked as in Theorem 3.2.

    k [C,r,d_k], v [C,r,d_v], beta [C,r]  ->  A [C,r,d_k], At [C,r,d_v], Bm [C,r,d_k] with
    A_t = K_t diag(beta_t), A~_t = -V_t diag(beta_t), B_t = -K_t (the R=1 Remark, column-wise)."""
    A = beta[..., None] * k
    At = -beta[..., None] * v
    Bm = -k
    return A, At, Bm


def time_strict_mask(C, r):
    """M[(t,i),(s,j)] = 1(s < t), flattened to (C*r) x (C*r) with row index t*r+i."""
    tok = np.arange(C * r) // r
    return (tok[None, :] < tok[:, None]).astype(np.float64)


def thm32_WU(A, At, Bm):
    """W = (Id - M.(A B^T))^{-1} A and U likewise with A~ (Theorem 3.2), via a library solve."""
    C, r, d_k = A.shape
    n = C * r
    Af, Atf, Bf = A.reshape(n, d_k), At.reshape(n, -1), Bm.reshape(n, d_k)
    Cmat = np.eye(n) - time_strict_mask(C, r) * (Af @ Bf.T)
    W = scipy.linalg.solve_triangular(Cmat, Af, lower=True)
    U = scipy.linalg.solve_triangular(Cmat, Atf, lower=True)
    return W, U, Cmat


def thm32_chunk_state(k, v, beta, S):
    """S_1 = S_0 + (U + W S_0^T)^T B for one chunk (Theorem 3.2).  S is d_v x d_k."""
    A, At, Bm = drivers(k, v, beta)
    W, U, _ = thm32_WU(A, At, Bm)
    n = W.shape[0]
    # In the paper S is d x d and acts as S A B^T; with S in R^{d_v x d_k}: (U + W S^T) is n x d_v.
    return S + (U + W @ S.T).T @ Bm.reshape(n, -1)


def block_triangular_inverse(Cmat, T, R):
    """D with D C = Id from the Proposition's recursion on R x R blocks (sequential form)."""
    D = np.zeros_like(Cmat)
    blk = lambda M, t, s: M[t * R:(t + 1) * R, s * R:(s + 1) * R]
    for t in range(T):
        Dtt = np.linalg.inv(blk(Cmat, t, t))
        D[t * R:(t + 1) * R, t * R:(t + 1) * R] = Dtt
        for s in range(t):
            acc = np.zeros((R, R))
            for rr in range(s, t):
                acc += blk(Cmat, t, rr) @ blk(D, rr, s)
            D[t * R:(t + 1) * R, s * R:(s + 1) * R] = -Dtt @ acc
    return D


def thm33_W(A, Bm):
    """Diagonal of the two-index system of Theorem 3.3, evaluated literally.

    The paper's per-step objects are d x R matrices: A_{t_k} = A[k].T, B_{t_k} = Bm[k].T.
    Returns W stacked [C, r, d] like Theorem 3.2 (row (k,i) = column i of W_{t_k})."""
    C, r, d = A.shape
    At = [A[t].T for t in range(C)]
    Bt = [Bm[t].T for t in range(C)]
    W2 = {}
    for kk in range(C):
        W2[(0, kk)] = At[kk].copy()
    for k1 in range(1, C):          # column index k+1
        kk = k1 - 1
        for m in range(kk):         # m < k
            W2[(m + 1, k1)] = (W2[(m, k1)] + W2[(m + 1, kk)] - W2[(m, kk)]
                               + W2[(m, m)] @ Bt[m].T @ (At[k1] - At[kk]))
        W2[(k1, k1)] = W2[(kk, k1)] + W2[(kk, kk)] @ Bt[kk].T @ At[k1]
    return np.stack([W2[(t, t)].T for t in range(C)], axis=0)


def token_matrices(k_t, v_t, beta_t):
    """(A_t, X_t) with S_t = S_{t-1} A_t + X_t:  A_t = I - K diag(beta) K^T, X_t = V diag(beta) K^T."""
    d_k = k_t.shape[-1]
    A_t = np.eye(d_k) - (k_t.T * beta_t) @ k_t
    X_t = (v_t.T * beta_t) @ k_t
    return A_t, X_t


def interval_flow(k, v, beta):
    """Flow of an interval (Proposition 2.1, discrete): (P, Xi) with S_end = S_start P + Xi."""
    d_k, d_v = k.shape[-1], v.shape[-1]
    P, Xi = np.eye(d_k), np.zeros((d_v, d_k))
    for t in range(k.shape[0]):
        A_t, X_t = token_matrices(k[t], v[t], beta[t])
        P, Xi = P @ A_t, Xi @ A_t + X_t
    return P, Xi


def chunked_forward(q, k, v, beta, S0, chunk, product=False):
    """The chunk-form forward pass for one sequence in fp64 (what the kernels compute, step by step).
    ``product``: the strict mask is taken in the flattened row index m' < m instead of the time index
    (the general block-triangular case: the factors of a token act one after another).

    q [L,d_k], k [L,r,d_k], v [L,r,d_v], beta [L,r], S0 [d_k,d_v] or None.
    Per chunk (rows m = t*r + j, n = C*r):
        Lm = I + Mstrict . (diag(b) K K^T),  T' = Lm^{-1} diag(b),  W = T' K,  Uh = T' V,
        U' = Uh - W S^T,  P = (Q K^T) . Mincl,  O = Q S^T + P U',  S <- S + U'^T K.
    Returns O [L,d_v], S_final [d_k,d_v] and the per-chunk intermediates."""
    L, r, d_k = k.shape
    d_v = v.shape[-1]
    S = np.zeros((d_v, d_k)) if S0 is None else np.asarray(S0, dtype=np.float64).T.copy()
    O = np.zeros((L, d_v))
    inter = []
    for c0 in range(0, L, chunk):
        c1 = min(L, c0 + chunk)
        C = c1 - c0
        n = C * r
        K = k[c0:c1].reshape(n, d_k)
        V = v[c0:c1].reshape(n, d_v)
        b = beta[c0:c1].reshape(n)
        Q = q[c0:c1]
        tok = np.arange(n) // r
        rows = np.arange(n)
        strict = (rows[None, :] < rows[:, None]) if product else (tok[None, :] < tok[:, None])
        Lm = np.eye(n) + strict * (b[:, None] * (K @ K.T))
        Tp = scipy.linalg.solve_triangular(Lm, np.diag(b), lower=True)
        W = Tp @ K
        Uh = Tp @ V
        Up = Uh - W @ S.T
        P = (Q @ K.T) * (tok[None, :] <= np.arange(C)[:, None])
        O[c0:c1] = Q @ S.T + P @ Up
        inter.append(dict(S_in=S.copy(), T=Tp, W=W, Uh=Uh, Up=Up, P=P))
        S = S + Up.T @ K
    return O, S.T.copy(), inter

"""fp64 CPU oracle for the MonarchAttention forward pass (arXiv 2505.18698).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
it exists so that tests, the smoke check and the benchmark's CPU-baseline leg
have a slow, plain statement of the method to compare the CUDA path with.  It
shares no code with the CUDA path.

What it computes, per (batch, head), for N = m*b, in float64:

    L^(0)[j,k,l] = delta_kl                                    (Sec. 3, init)
    for t = 1..T:   R-update first, then L-update             (App. C.2)
        aR[k,j,:] = sum_l L[j,k,l] Qb[j,l,:]                   (Eq. 9)
        cR[k,j]   = sum_l L[j,k,l]                             (Eq. 9)
        Z_R[k,j,i] = <aR[k,j,:], Kb[k,i,:]> / cR[k,j] (+ mask) (Eq. 7, App. C.3)
        R[k,j,:]  = softmax_i Z_R[k,j,:]                       (Eq. 7)
        aL[j,k,:] = sum_i R[k,j,i] Kb[k,i,:]                   (Eq. 10)
        cL[j,k]   = sum_i R[k,j,i] log R[k,j,i]                (Eq. 10)
        Z_L[j,k,l] = <aL[j,k,:], Qb[j,l,:]> - cL[j,k]          (Eq. 8)
        L[j,:,l]  = softmax_k Z_L[j,:,l]                       (Eq. 8)
    y[j,k,:]  = sum_i R[k,j,i] Vb[k,i,:]                       (Eq. 4)
    O[b*l+j,:] = sum_k L[j,k,l] y[j,k,:]                       (Eq. 4)

with Qb[j,l,:] = scale * Q[b*l + j], Kb[k,i,:] = K[b*k + i], Vb likewise
(0-based; Sec. 3 below Eq. 10; the softmax scale is absorbed into Q as the
footnote to Eq. 3 says, so it multiplies both score tensors and never cL).

Readings taken where the paper is silent:
  * 0*log 0 = 0 in cL (R log R is evaluated as R*(Z - logsumexp Z) and set to 0
    where R == 0).
  * T >= 1 is required (R^(0) is never defined).
  * cR == 0 cannot happen in exact arithmetic; in fp64 it would need logit gaps
    beyond ~745.  Such a row gets Z_R = 0 and the event is counted.
  * Padding (App. C.3): with n_valid < N, key columns b*k+i >= n_valid get
    omega = -inf added to Z_R (post-padding).

Pins (tests/test_oracle_pins.py): the dense Monarch matrix of Eq. 5 and
M = P^T B; the printed permutation example of App. B; row-stochasticity;
closed forms for Q = 0, constant V, block-constant K; exact reduction to
textbook softmax attention for b = N and b = 1; monotone ascent of the dense
objective and its softmax upper bound; a finite-difference KKT check of each
half-step against the dense objective; separable objective = dense objective.
Numerical output values for a real workload: parity unpinned (the paper prints
none that can be reproduced without its models and datasets).
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "block_views", "r_update", "l_update", "monarch_multiply",
    "monarch_attention_head", "monarch_attention", "monarch_attention_state_form_head",
    "transpose_permutation", "block_rank_one", "dense_monarch",
    "objective_dense", "objective_factored",
]


# --------------------------------------------------------------------------- views
def block_views(Q, K, V, b, scale):
    """Qb[j,l,:] = scale*Q[b*l+j], Kb[k,i,:] = K[b*k+i], Vb[k,i,:] = V[b*k+i]
    (text below Eq. 10; Eq. 4)."""
    N, d = Q.shape
    assert N % b == 0
    m = N // b
    Qb = (scale * Q).reshape(m, b, d).transpose(1, 0, 2)   # [j, l, v]
    Kb = K.reshape(m, b, d)                                # [k, i, v]
    Vb = V.reshape(m, b, V.shape[1])                       # [k, i, v]
    return Qb, Kb, Vb


def _key_mask(m, b, n_valid):
    """omega[k,i] of App. C.3 (post-padding): 0 for b*k+i < n_valid, -inf after."""
    col = b * np.arange(m)[:, None] + np.arange(b)[None, :]
    return np.where(col < n_valid, 0.0, -np.inf)


# --------------------------------------------------------------------------- updates
def r_update(L, Qb, Kb, omega=None, stats=None):
    """Eq. 7 with Eq. 9.  Returns R[k,j,i] and log R[k,j,i]."""
    aR = np.einsum("jkl,jlv->kjv", L, Qb)                  # alpha_R
    cR = np.einsum("jkl->kj", L)                           # c_R
    betaR = np.einsum("kjv,kiv->kji", aR, Kb)              # beta_R
    zero = cR == 0.0
    if stats is not None:
        stats["min_cR"] = min(stats.get("min_cR", np.inf), float(cR.min()))
        stats["cR_zero_rows"] = stats.get("cR_zero_rows", 0) + int(zero.sum())
    ZR = np.where(zero[:, :, None], 0.0, betaR / np.where(zero, 1.0, cR)[:, :, None])
    if omega is not None:
        ZR = ZR + omega[:, None, :]
    zmax = ZR.max(axis=2, keepdims=True)
    lse = zmax + np.log(np.exp(ZR - zmax).sum(axis=2, keepdims=True))
    logR = ZR - lse
    R = np.exp(logR)
    return R, logR


def l_update(R, logR, Qb, Kb):
    """Eq. 8 with Eq. 10.  Returns L[j,k,l]."""
    aL = np.einsum("kji,kiv->jkv", R, Kb)                  # alpha_L
    RlogR = np.where(R > 0.0, R * np.where(R > 0.0, logR, 0.0), 0.0)   # 0 log 0 = 0
    cL = np.einsum("kji->jk", RlogR)                       # c_L
    betaL = np.einsum("jkv,jlv->jkl", aL, Qb)              # beta_L
    ZL = betaL - cL[:, :, None]
    ZL = ZL - ZL.max(axis=1, keepdims=True)
    E = np.exp(ZL)
    return E / E.sum(axis=1, keepdims=True)                # softmax over k


def monarch_multiply(L, R, Vb):
    """Eq. 4: O[b*l+j,:] = sum_k L[j,k,l] * (sum_i R[k,j,i] Vb[k,i,:])."""
    b, m, _ = L.shape
    y = np.einsum("kji,kiv->jkv", R, Vb)
    z = np.einsum("jkl,jkv->ljv", L, y)                    # row b*l+j
    return z.reshape(m * b, Vb.shape[2])


# --------------------------------------------------------------------------- one head
def monarch_attention_head(Q, K, V, b, T, scale=None, n_valid=None,
                           return_factors=False, stats=None, trace=None):
    """One head.  Q, K: (N, d); V: (N, dv); returns O (N, dv) in float64.

    `trace`, if a list, receives (name, L.copy(), R.copy()) after every
    half-step (used by the ascent pin)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N, d = Q.shape
    if T < 1:
        raise ValueError("T must be >= 1")
    if b < 1 or N % b != 0:
        raise ValueError("N must be a multiple of b")
    m = N // b
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    Qb, Kb, Vb = block_views(Q, K, V, b, scale)
    omega = None if n_valid is None or n_valid >= N else _key_mask(m, b, n_valid)

    L = np.broadcast_to(np.eye(m), (b, m, m)).copy()       # L^(0)[j,k,l] = delta_kl
    R = logR = None
    for _ in range(T):
        R, logR = r_update(L, Qb, Kb, omega, stats)
        if trace is not None:
            trace.append(("R", L.copy(), R.copy()))
        L = l_update(R, logR, Qb, Kb)
        if trace is not None:
            trace.append(("L", L.copy(), R.copy()))
    O = monarch_multiply(L, R, Vb)
    if return_factors:
        return O, L, R
    return O


def monarch_attention(Q, K, V, b, T, scale=None, n_valid=None):
    """Batched: Q, K, V of shape (..., N, d); heads are independent (Sec. 2)."""
    Q = np.asarray(Q)
    lead = Q.shape[:-2]
    N, d = Q.shape[-2:]
    dv = np.asarray(V).shape[-1]
    Qf = np.asarray(Q).reshape(-1, N, d)
    Kf = np.asarray(K).reshape(-1, N, d)
    Vf = np.asarray(V).reshape(-1, N, dv)
    out = np.empty((Qf.shape[0], N, dv), dtype=np.float64)
    for h in range(Qf.shape[0]):
        out[h] = monarch_attention_head(Qf[h], Kf[h], Vf[h], b, T, scale, n_valid)
    return out.reshape(*lead, N, dv)


# --------------------------------------------------------------------------- state form
def monarch_attention_state_form_head(Q, K, V, b, T, scale=None):
    """The same recursion carried by the states (alpha, c) only, L and R living
    just inside one half-step (Sec. 3 'Implementation', Fig. 4).  A second
    statement of the algorithm used as a cross-check of the first."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N, d = Q.shape
    m = N // b
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    Qb, Kb, Vb = block_views(Q, K, V, b, scale)

    # L^(0) = identity  =>  alpha_R^(1)[k,j,:] = Qb[j,k,:],  c_R^(1) = 1
    aR = Qb.transpose(1, 0, 2).copy()
    cR = np.ones((m, b))
    out = None
    for t in range(1, T + 1):
        # alpha_R, c_R -> alpha_L, c_L (and y on the last step)
        ZR = np.einsum("kjv,kiv->kji", aR, Kb) / cR[:, :, None]
        ZR = ZR - ZR.max(axis=2, keepdims=True)
        R = np.exp(ZR)
        R = R / R.sum(axis=2, keepdims=True)
        with np.errstate(divide="ignore", invalid="ignore"):
            cL = np.where(R > 0, R * np.log(R), 0.0).sum(axis=2).T      # [j,k]
        aL = np.einsum("kji,kiv->jkv", R, Kb)
        ZL = np.einsum("jkv,jlv->jkl", aL, Qb) - cL[:, :, None]
        ZL = ZL - ZL.max(axis=1, keepdims=True)
        Lf = np.exp(ZL)
        Lf = Lf / Lf.sum(axis=1, keepdims=True)
        if t < T:
            aR = np.einsum("jkl,jlv->kjv", Lf, Qb)
            cR = Lf.sum(axis=2).T
        else:
            y = np.einsum("kji,kiv->jkv", R, Vb)
            out = np.einsum("jkl,jkv->ljv", Lf, y).reshape(N, Vb.shape[2])
    return out


# --------------------------------------------------------------------------- dense forms
def transpose_permutation(m, b):
    """P of Sec. 2: row i is e_{sigma(i)}, sigma(i) = b*(i mod m) + floor(i/m)."""
    N = m * b
    P = np.zeros((N, N))
    for i in range(N):
        P[i, b * (i % m) + i // m] = 1.0
    return P


def block_rank_one(L, R):
    """B of Sec. 2: a b-by-m grid of m-by-b blocks B_jk = L[j,k,:] R[k,j,:]^T."""
    b, m, _ = L.shape
    B = np.zeros((b * m, m * b))
    for j in range(b):
        for k in range(m):
            B[j * m:(j + 1) * m, k * b:(k + 1) * b] = np.outer(L[j, k, :], R[k, j, :])
    return B


def dense_monarch(L, R):
    """Eq. 5: M[b*l+j, b*k+i] = L[j,k,l] * R[k,j,i]."""
    b, m, _ = L.shape
    M = np.zeros((m * b, m * b))
    for l in range(m):
        for j in range(b):
            for k in range(m):
                M[b * l + j, b * k:b * (k + 1)] = L[j, k, l] * R[k, j, :]
    return M


def _neg_xlogx_sum(A):
    A = np.asarray(A, dtype=np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        return -np.where(A > 0, A * np.log(A), 0.0).sum()


def objective_dense(M, Q, K, scale):
    """Eq. 6: f(M; Q, K) = <M, scale*Q K^T> + H(M) on the dense matrix."""
    S = scale * (np.asarray(Q, np.float64) @ np.asarray(K, np.float64).T)
    return float((M * S).sum() + _neg_xlogx_sum(M))


def final_row_lse(R, Q, K, b, scale):
    """Row-wise log-sum-exp of the logits of the L update that follows R (Eq. 8 with Eq. 10):
    lse[b*l + j] = log sum_k exp(Z_L[j,k,l]).  Because that update is the exact maximiser over L
    (L = softmax_k Z_L, so Z_L - log L is constant in k) and every R[k,j,:] sums to one, the
    objective of Eq. 6 at (L, R) is the plain sum of these N numbers; the pin is
    test_objective_equals_sum_of_final_row_lse."""
    Q = np.asarray(Q, np.float64)
    K = np.asarray(K, np.float64)
    Qb, Kb, _ = block_views(Q, K, K, b, scale)
    m = Q.shape[0] // b
    logR = np.where(R > 0.0, np.log(np.where(R > 0.0, R, 1.0)), 0.0)
    aL = np.einsum("kji,kiv->jkv", R, Kb)
    cL = np.einsum("kji->jk", np.where(R > 0.0, R * logR, 0.0))
    ZL = np.einsum("jkv,jlv->jkl", aL, Qb) - cL[:, :, None]
    zmax = ZL.max(axis=1)
    lse = zmax + np.log(np.exp(ZL - zmax[:, None, :]).sum(axis=1))          # [j, l]
    return lse.T.reshape(m * b)                                            # row b*l + j


def objective_factored(L, R, Q, K, scale):
    """Sec. 3 'Softmax Objective': sum over (j,k) of
    <Qb_j^T L_jk, Kb_k^T R_kj> + (1^T R_kj) H(L_jk) + (1^T L_jk) H(R_kj)."""
    b, m, _ = L.shape
    Qb, Kb, _ = block_views(np.asarray(Q, np.float64), np.asarray(K, np.float64),
                            np.asarray(K, np.float64), b, scale)
    total = 0.0
    for j in range(b):
        for k in range(m):
            Ljk = L[j, k, :]
            Rkj = R[k, j, :]
            total += float((Qb[j].T @ Ljk) @ (Kb[k].T @ Rkj))
            total += Rkj.sum() * _neg_xlogx_sum(Ljk) + Ljk.sum() * _neg_xlogx_sum(Rkj)
    return total

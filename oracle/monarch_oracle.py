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
  * Batched sequences of different lengths (App. C.3 names the case, gives no
    formula): a block lying wholly in the padding has no admissible R row
    (softmax of all -inf).  Reading: such a block is absent from the
    sequence's problem -- R = 0 there, Z_L = -inf for it as a key block (so
    the rows of M still sum to one over valid keys), and as a query block it
    is left out of the sums over l of Eq. 9.  Pin: the valid rows equal those
    of the same sequence run alone at its own padded length.

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
# Every contraction below is written per block, as a plain 2-D matrix product over the block's own
# index pair: "for each key block k" or "for each in-block position j", exactly the batching the
# equations state.  Nothing is fused or reordered beyond that.
def _softmax_rows(Z, axis):
    """softmax and log-softmax along `axis`, max-subtracted; an all -inf slice gives zeros."""
    zmax = Z.max(axis=axis, keepdims=True)
    dead = ~np.isfinite(zmax)                       # slice with no admissible entry
    shifted = Z - np.where(dead, 0.0, zmax)
    lse = np.log(np.exp(shifted).sum(axis=axis, keepdims=True), where=~dead,
                 out=np.zeros_like(zmax)) + np.where(dead, 0.0, zmax)
    logS = np.where(dead, -np.inf, Z - lse)
    return np.exp(logS), logS


def r_update(L, Qb, Kb, omega=None, stats=None, m_live=None):
    """Eq. 7 with Eq. 9.  Returns R[k,j,i] and log R[k,j,i].

    `m_live` (batched sequences of different lengths, App. C.3): blocks from m_live on lie wholly in
    the padding; every key of such a block is masked, so it has no admissible R row.  Reading: those
    blocks are absent from the sequence's problem, as key blocks (R = 0) and as query blocks (no
    term in the sums over l of Eq. 9); their rows of Q, K are never touched."""
    b, m, _ = L.shape
    d = Qb.shape[2]
    live = m if m_live is None else m_live
    alpha_R = np.zeros((m, b, d))
    c_R = np.zeros((m, b))
    for j in range(b):                              # Eq. 9, position j: [k,l] x [l,v]
        alpha_R[:live, j, :] = L[j][:live, :live] @ Qb[j][:live]
        c_R[:live, j] = L[j][:live, :live].sum(axis=1)
    R = np.zeros((m, b, b))
    logR = np.full((m, b, b), -np.inf)
    for k in range(live):                           # Eq. 7, key block k: [j,v] x [v,i]
        beta_R = alpha_R[k] @ Kb[k].T
        zero = c_R[k] == 0.0
        if stats is not None:
            stats["min_cR"] = min(stats.get("min_cR", np.inf), float(c_R[k].min()))
            stats["cR_zero_rows"] = stats.get("cR_zero_rows", 0) + int(zero.sum())
        Z_R = np.where(zero[:, None], 0.0, beta_R / np.where(zero, 1.0, c_R[k])[:, None])
        if omega is not None:
            Z_R = Z_R + omega[k][None, :]
        R[k], logR[k] = _softmax_rows(Z_R, axis=1)
    return R, logR


def l_update(R, logR, Qb, Kb, m_live=None):
    """Eq. 8 with Eq. 10.  Returns L[j,k,l].

    `m_live`: see r_update.  An absent key block has Z_L = -inf, i.e. L[j,k,:] = 0, so that the
    rows of M still sum to one over the valid keys; an absent query block has L[j,:,l] = 0."""
    m, b, _ = R.shape
    d = Kb.shape[2]
    live = m if m_live is None else m_live
    alpha_L = np.zeros((b, m, d))
    c_L = np.zeros((b, m))
    for k in range(live):                           # Eq. 10, key block k: [j,i] x [i,v]
        alpha_L[:, k, :] = R[k] @ Kb[k]
        RlogR = np.where(R[k] > 0.0, R[k] * np.where(R[k] > 0.0, logR[k], 0.0), 0.0)   # 0 log 0 = 0
        c_L[:, k] = RlogR.sum(axis=1)
    L = np.zeros((b, m, m))
    for j in range(b):                              # Eq. 8, position j: [k,v] x [v,l]
        Z_L = alpha_L[j][:live] @ Qb[j][:live].T - c_L[j][:live, None]
        L[j][:live, :live], _ = _softmax_rows(Z_L, axis=0)        # over k for every l
    return L


def monarch_multiply(L, R, Vb, m_live=None):
    """Eq. 4: O[b*l+j,:] = sum_k L[j,k,l] * (sum_i R[k,j,i] Vb[k,i,:]).  Rows of absent blocks
    (`m_live`, see r_update) are zero."""
    b, m, _ = L.shape
    dv = Vb.shape[2]
    live = m if m_live is None else m_live
    y = np.zeros((b, m, dv))
    for k in range(live):                           # first factor, key block k: [j,i] x [i,v]
        y[:, k, :] = R[k] @ Vb[k]
    O = np.zeros((m, b, dv))                        # [l, j, v] = row b*l + j
    for j in range(b):                              # second factor, position j: [l,k] x [k,v]
        O[:live, j, :] = L[j][:live, :live].T @ y[j][:live]
    return O.reshape(m * b, dv)


# --------------------------------------------------------------------------- one head
def monarch_attention_head(Q, K, V, b, T, scale=None, n_valid=None,
                           return_factors=False, stats=None, trace=None):
    """One head.  Q, K: (N, d); V: (N, dv); returns O (N, dv) in float64.

    n_valid (App. C.3, post-padding): keys b*k+i >= n_valid are masked.  With less than one block
    of padding this is the appendix's case.  With more (a sequence of a padded batch), the blocks
    that lie wholly in the padding are absent from the sequence's problem: see r_update / l_update;
    rows of O from ceil(n_valid/b)*b on are zero.

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
    omega = None
    m_live = m
    if n_valid is not None and n_valid < N:
        if n_valid < 1:
            raise ValueError("n_valid must be >= 1")
        omega = _key_mask(m, b, n_valid)
        m_live = -(-n_valid // b)

    L = np.zeros((b, m, m))
    L[:, np.arange(m_live), np.arange(m_live)] = 1.0       # L^(0)[j,k,l] = delta_kl
    R = logR = None
    for _ in range(T):
        R, logR = r_update(L, Qb, Kb, omega, stats, m_live)
        if trace is not None:
            trace.append(("R", L.copy(), R.copy()))
        L = l_update(R, logR, Qb, Kb, m_live)
        if trace is not None:
            trace.append(("L", L.copy(), R.copy()))
    O = monarch_multiply(L, R, Vb, m_live)
    if return_factors:
        return O, L, R
    return O


def monarch_attention(Q, K, V, b, T, scale=None, n_valid=None):
    """Batched: Q, K, V of shape (..., N, d); heads are independent (Sec. 2).  n_valid: None, one
    length for all, or an array of lengths with the shape of the leading axes (or of the first of
    them: one length per batch entry)."""
    Q = np.asarray(Q)
    lead = Q.shape[:-2]
    N, d = Q.shape[-2:]
    dv = np.asarray(V).shape[-1]
    Qf = np.asarray(Q).reshape(-1, N, d)
    Kf = np.asarray(K).reshape(-1, N, d)
    Vf = np.asarray(V).reshape(-1, N, dv)
    if n_valid is None or np.ndim(n_valid) == 0:
        nv = [n_valid] * Qf.shape[0]
    else:
        nva = np.asarray(n_valid)
        if nva.shape != lead:                       # one length per batch entry
            nva = np.broadcast_to(nva.reshape(nva.shape + (1,) * (len(lead) - nva.ndim)), lead)
        nv = [int(x) for x in nva.reshape(-1)]
    out = np.empty((Qf.shape[0], N, dv), dtype=np.float64)
    for h in range(Qf.shape[0]):
        out[h] = monarch_attention_head(Qf[h], Kf[h], Vf[h], b, T, scale, nv[h])
    return out.reshape(*lead, N, dv)


# --------------------------------------------------------------------------- state form
def monarch_attention_state_form_head(Q, K, V, b, T, scale=None):
    """The same recursion carried by the states (alpha, c) only (Sec. 3 'Implementation'): the
    factors live only inside one half-step, a key block at a time (R) or a position at a time (L).
    A second statement of the algorithm, used as a cross-check of the first: its only state between
    half-steps is alpha_R, c_R (k-major) or alpha_L, c_L, y (j-major)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    N, d = Q.shape
    m = N // b
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    Qs = scale * Q
    dv = V.shape[1]
    # L^(0) = identity  =>  alpha_R^(1)[k,j,:] = Qs[b*k + j],  c_R^(1) = 1
    alpha_R = Qs.reshape(m, b, d).copy()
    c_R = np.ones((m, b))
    O = np.empty((N, dv))
    for t in range(1, T + 1):
        alpha_L = np.empty((b, m, d))
        c_L = np.empty((b, m))
        y = np.empty((b, m, dv))
        for k in range(m):                          # R half-step of key block k
            Kk = K[b * k:b * (k + 1)]
            Z = (alpha_R[k] @ Kk.T) / c_R[k][:, None]
            Z = Z - Z.max(axis=1, keepdims=True)
            E = np.exp(Z)
            s = E.sum(axis=1, keepdims=True)
            Rk = E / s
            with np.errstate(divide="ignore", invalid="ignore"):
                c_L[:, k] = np.where(Rk > 0, Rk * (Z - np.log(s)), 0.0).sum(axis=1)
            alpha_L[:, k, :] = Rk @ Kk
            if t == T:
                y[:, k, :] = Rk @ V[b * k:b * (k + 1)]
        for j in range(b):                          # L half-step of position j
            Qj = Qs[j::b]                           # rows b*l + j, l = 0..m-1
            Z = alpha_L[j] @ Qj.T - c_L[j][:, None]          # [k, l]
            Z = Z - Z.max(axis=0, keepdims=True)
            E = np.exp(Z)
            Lj = E / E.sum(axis=0, keepdims=True)
            if t < T:
                alpha_R[:, j, :] = Lj @ Qj
                c_R[:, j] = Lj.sum(axis=1)
            else:
                O[j::b] = Lj.T @ y[j]
    return O


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
    (L = softmax_k Z_L, so Z_L - log L is constant in k) and every R[k,j,:] sums to one, row
    b*l + j of M contributes exactly lse[b*l + j] to the objective of Eq. 6, and the objective is
    the plain sum of these N numbers; pins: test_objective_equals_sum_of_final_row_lse (sum) and
    test_final_row_lse_is_each_rows_own_term_of_the_objective (row by row)."""
    Q = np.asarray(Q, np.float64)
    K = np.asarray(K, np.float64)
    Qb, Kb, _ = block_views(Q, K, K, b, scale)
    m = Q.shape[0] // b
    lse = np.empty((m, b))                                                  # [l, j] = row b*l + j
    for j in range(b):
        alpha_L = np.stack([R[k, j] @ Kb[k] for k in range(m)])            # [k, v]
        with np.errstate(divide="ignore", invalid="ignore"):
            c_L = np.array([np.where(R[k, j] > 0, R[k, j] * np.log(R[k, j]), 0.0).sum()
                            for k in range(m)])
        Z_L = alpha_L @ Qb[j].T - c_L[:, None]                              # [k, l]
        zmax = Z_L.max(axis=0)
        lse[:, j] = zmax + np.log(np.exp(Z_L - zmax[None, :]).sum(axis=0))
    return lse.reshape(m * b)


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

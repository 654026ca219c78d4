"""Pins of the fp64 oracle to things other than itself: what the paper prints, closed
forms, textbook special cases, the dense objective, and finite differences."""
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import monarch_oracle as mo
from paper_2505_18698_b200.workloads import macs_per_head

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_qkv(N, d, seed, spread=1.0):
    rng = np.random.default_rng(seed)
    return (spread * rng.standard_normal((N, d)), spread * rng.standard_normal((N, d)),
            rng.standard_normal((N, d)))


def dense_softmax_attention(Q, K, V, scale):
    return softmax(scale * Q @ K.T, axis=1) @ V


SHAPES = [(6, 3), (6, 2), (12, 4), (12, 3), (16, 4), (24, 6), (24, 2), (24, 12)]


# ---------------------------------------------------------------- what the paper prints
def test_permutation_example_appendix_b():
    P_printed = np.loadtxt(os.path.join(GOLDEN, "permutation_appendix_b.txt"))
    P = mo.transpose_permutation(m=2, b=3)
    assert np.array_equal(P, P_printed)
    assert np.array_equal(P @ np.arange(1, 7), np.array([1, 4, 2, 5, 3, 6]))
    # footnote of Sec. 2: reshape to (m, b), transpose, flatten
    for m, b in [(2, 3), (3, 2), (4, 5), (5, 5)]:
        x = np.arange(m * b, dtype=float)
        assert np.array_equal(mo.transpose_permutation(m, b) @ x, x.reshape(m, b).T.reshape(-1))


def test_operation_counts_match_printed_tables():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "flop_tables.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for tab, N, d, b, T, units, soft, mon in rows:
        N, d, b, T, units = int(N), int(d), int(b), int(T), int(units)
        got = units * macs_per_head(N, d, b, T) / 1e9
        dense = units * 2 * N * N * d / 1e9
        assert abs(got - float(mon)) <= 0.006 * float(mon), (tab, N, got, mon)
        assert abs(dense - float(soft)) <= 0.006 * float(soft), (tab, N, dense, soft)
    # Tab. 1, "First Half" row: 14 of 28 layers replaced -> 5.95
    full = 896 * 2 * 256 * 256 * 72 / 1e9
    mon = 896 * macs_per_head(256, 72, 16, 3) / 1e9
    assert abs(0.5 * full + 0.5 * mon - 5.95) < 0.01


# ---------------------------------------------------------------- dense Monarch matrix
@pytest.mark.parametrize("N,b", SHAPES)
@pytest.mark.parametrize("T", [1, 2, 3])
def test_factored_apply_equals_dense_monarch(N, b, T):
    Q, K, V = rand_qkv(N, 5, seed=N * 10 + b + T)
    O, L, R = mo.monarch_attention_head(Q, K, V, b, T, return_factors=True)
    M = mo.dense_monarch(L, R)                           # Eq. 5
    assert np.allclose(M @ V, O, rtol=0, atol=1e-13)
    m = N // b
    P = mo.transpose_permutation(m, b)
    assert np.allclose(P.T @ mo.block_rank_one(L, R), M, rtol=0, atol=1e-15)   # M = P^T B
    # simplex constraints of Sec. 3 and their consequence
    assert (L >= 0).all() and (R >= 0).all()
    assert np.allclose(L.sum(axis=1), 1.0, atol=1e-13)   # over k for each (j, l)
    assert np.allclose(R.sum(axis=2), 1.0, atol=1e-13)   # over i for each (k, j)
    assert (M >= 0).all() and np.allclose(M.sum(axis=1), 1.0, atol=1e-13)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("N,b", SHAPES)
def test_constant_v_gives_constant_output(N, b):
    Q, K, _ = rand_qkv(N, 4, seed=3)
    c = np.array([1.5, -2.0, 0.25])
    O = mo.monarch_attention_head(Q, K, np.tile(c, (N, 1)), b, T=2)
    assert np.allclose(O, np.tile(c, (N, 1)), atol=1e-13)


@pytest.mark.parametrize("N,b", SHAPES)
@pytest.mark.parametrize("which", ["Q", "K"])
def test_zero_q_or_k_gives_uniform_average(N, b, which):
    Q, K, V = rand_qkv(N, 4, seed=5)
    if which == "Q":
        Q = np.zeros_like(Q)
    else:
        K = np.zeros_like(K)
    O, L, R = mo.monarch_attention_head(Q, K, V, b, T=2, return_factors=True)
    m = N // b
    assert np.allclose(R, 1.0 / b, atol=1e-15) and np.allclose(L, 1.0 / m, atol=1e-15)
    assert np.allclose(O, np.tile(V.mean(axis=0), (N, 1)), atol=1e-13)


@pytest.mark.parametrize("T", [1, 2, 4])
@pytest.mark.parametrize("N", [6, 16, 24])
def test_single_block_is_textbook_softmax_attention(N, T):
    """b = N (m = 1): L == 1, alpha_R = Q, c_R = 1, R = softmax(QK^T) exactly."""
    Q, K, V = rand_qkv(N, 7, seed=N + T, spread=2.0)
    scale = 0.37
    O = mo.monarch_attention_head(Q, K, V, b=N, T=T, scale=scale)
    assert np.allclose(O, dense_softmax_attention(Q, K, V, scale), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("T", [1, 2, 4])
@pytest.mark.parametrize("N", [6, 16, 24])
def test_unit_blocks_are_textbook_softmax_attention(N, T):
    """b = 1 (m = N): R == 1, c_L = 0, alpha_L = K, L = softmax_k(QK^T) exactly."""
    Q, K, V = rand_qkv(N, 7, seed=2 * N + T, spread=2.0)
    scale = 0.41
    O = mo.monarch_attention_head(Q, K, V, b=1, T=T, scale=scale)
    assert np.allclose(O, dense_softmax_attention(Q, K, V, scale), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("N,b", [(12, 4), (16, 4), (24, 6), (24, 3)])
def test_block_constant_keys_give_exact_softmax_attention(N, b):
    """If all keys inside each block coincide, softmax(QK^T) is itself Monarch
    (each b-by-b block is rank one) and one step recovers it exactly."""
    rng = np.random.default_rng(11)
    m = N // b
    Q = rng.standard_normal((N, 5))
    K = np.repeat(rng.standard_normal((m, 5)), b, axis=0)
    V = rng.standard_normal((N, 5))
    for T in (1, 2):
        O = mo.monarch_attention_head(Q, K, V, b, T, scale=0.5)
        assert np.allclose(O, dense_softmax_attention(Q, K, V, 0.5), rtol=1e-12, atol=1e-13)


def test_default_scale_is_inverse_sqrt_d():
    Q, K, V = rand_qkv(16, 9, seed=1)
    assert np.array_equal(mo.monarch_attention_head(Q, K, V, 4, 2),
                          mo.monarch_attention_head(Q, K, V, 4, 2, scale=1.0 / 3.0))


# ---------------------------------------------------------------- objective: ascent, bound, KKT
@pytest.mark.parametrize("N,b", [(12, 4), (16, 4), (24, 6), (24, 2), (12, 1), (12, 12)])
def test_monotone_ascent_and_softmax_upper_bound(N, b):
    Q, K, V = rand_qkv(N, 5, seed=N + b, spread=1.5)
    scale = 0.6
    trace = []
    mo.monarch_attention_head(Q, K, V, b, T=3, scale=scale, trace=trace)
    f = [mo.objective_dense(mo.dense_monarch(L, R), Q, K, scale) for _, L, R in trace]
    assert all(f[i + 1] >= f[i] - 1e-10 for i in range(len(f) - 1)), f
    bound = logsumexp(scale * Q @ K.T, axis=1).sum()       # f at the unconstrained maximiser
    assert all(x <= bound + 1e-10 for x in f)
    if b in (1, N):
        assert abs(f[-1] - bound) < 1e-9
    # the separable evaluation of Sec. 3 equals the dense one
    for _, L, R in trace:
        assert abs(mo.objective_factored(L, R, Q, K, scale)
                   - mo.objective_dense(mo.dense_monarch(L, R), Q, K, scale)) < 1e-9


def _fd_grad(fun, X, eps=1e-6):
    G = np.zeros_like(X)
    it = np.nditer(X, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        Xp = X.copy(); Xp[idx] += eps
        Xm = X.copy(); Xm[idx] -= eps
        G[idx] = (fun(Xp) - fun(Xm)) / (2 * eps)
    return G


@pytest.mark.parametrize("N,b", [(6, 3), (6, 2), (8, 2), (8, 4)])
def test_half_steps_satisfy_kkt_of_dense_objective(N, b):
    """Each update must be the maximiser of the dense objective over its simplex
    slices: the gradient (by finite differences of Eq. 6 on the dense M of Eq. 5,
    which never uses the update formulas) is constant along every slice."""
    Q, K, V = rand_qkv(N, 3, seed=7 * N + b)
    scale = 0.8
    trace = []
    mo.monarch_attention_head(Q, K, V, b, T=2, scale=scale, trace=trace)
    for name, L, R in trace:
        if name == "R":      # R maximises f(L fixed, .) over rows R[k,j,:]
            G = _fd_grad(lambda X: mo.objective_dense(mo.dense_monarch(L, X), Q, K, scale), R)
            spread = G.max(axis=2) - G.min(axis=2)
        else:                # L maximises f(., R fixed) over slices L[j,:,l]
            G = _fd_grad(lambda X: mo.objective_dense(mo.dense_monarch(X, R), Q, K, scale), L)
            spread = G.max(axis=1) - G.min(axis=1)
        assert spread.max() < 1e-6, (name, spread.max())


@pytest.mark.parametrize("N,b", [(12, 4), (12, 3)])
def test_random_feasible_perturbations_never_improve(N, b):
    rng = np.random.default_rng(2)
    Q, K, V = rand_qkv(N, 4, seed=9)
    scale = 0.5
    trace = []
    mo.monarch_attention_head(Q, K, V, b, T=2, scale=scale, trace=trace)
    for name, L, R in trace:
        f0 = mo.objective_dense(mo.dense_monarch(L, R), Q, K, scale)
        for _ in range(20):
            if name == "R":
                D = rng.dirichlet(np.ones(R.shape[2]), size=R.shape[:2])
                X = 0.9 * R + 0.1 * D
                f1 = mo.objective_dense(mo.dense_monarch(L, X), Q, K, scale)
            else:
                D = rng.dirichlet(np.ones(L.shape[1]), size=(L.shape[0], L.shape[2])).transpose(0, 2, 1)
                X = 0.9 * L + 0.1 * D
                f1 = mo.objective_dense(mo.dense_monarch(X, R), Q, K, scale)
            assert f1 <= f0 + 1e-10


# ---------------------------------------------------------------- invariances, two statements
@pytest.mark.parametrize("N,b", SHAPES)
def test_key_shift_and_in_block_permutation_invariance(N, b):
    rng = np.random.default_rng(4)
    Q, K, V = rand_qkv(N, 5, seed=13)
    O = mo.monarch_attention_head(Q, K, V, b, T=2)
    # in exact arithmetic K -> K + 1 c^T adds a per-row constant to both score tensors
    O2 = mo.monarch_attention_head(Q, K + rng.standard_normal(5), V, b, T=2)
    assert np.allclose(O, O2, atol=1e-11)
    m = N // b
    perm = np.concatenate([b * k + rng.permutation(b) for k in range(m)])
    O3 = mo.monarch_attention_head(Q, K[perm], V[perm], b, T=2)
    assert np.allclose(O, O3, atol=1e-12)


@pytest.mark.parametrize("N,b", SHAPES)
@pytest.mark.parametrize("T", [1, 2, 3])
def test_state_form_agrees_with_factor_form(N, b, T):
    Q, K, V = rand_qkv(N, 6, seed=17 + T, spread=1.5)
    A = mo.monarch_attention_head(Q, K, V, b, T)
    B = mo.monarch_attention_state_form_head(Q, K, V, b, T)
    assert np.allclose(A, B, rtol=1e-12, atol=1e-13)


def test_batch_and_head_permutation_equivariance():
    rng = np.random.default_rng(8)
    Q, K, V = (rng.standard_normal((2, 3, 16, 4)) for _ in range(3))
    O = mo.monarch_attention(Q, K, V, b=4, T=2)
    pb, ph = [1, 0], [2, 0, 1]
    O2 = mo.monarch_attention(Q[pb][:, ph], K[pb][:, ph], V[pb][:, ph], b=4, T=2)
    assert np.array_equal(O[pb][:, ph], O2)


# ---------------------------------------------------------------- padding (App. C.3)
@pytest.mark.parametrize("N,b,n_valid", [(12, 4, 10), (16, 4, 13), (15, 5, 11)])
def test_padding_mask_zeroes_padded_columns(N, b, n_valid):
    Q, K, V = rand_qkv(N, 4, seed=21)
    O, L, R = mo.monarch_attention_head(Q, K, V, b, T=2, n_valid=n_valid, return_factors=True)
    M = mo.dense_monarch(L, R)
    assert np.all(M[:, n_valid:] == 0.0)
    assert np.allclose(M.sum(axis=1), 1.0, atol=1e-13)
    assert np.isfinite(O).all()
    # garbage in the padded rows of K, V cannot change valid outputs
    K2, V2 = K.copy(), V.copy()
    K2[n_valid:] = 1e3
    V2[n_valid:] = -1e3
    O2 = mo.monarch_attention_head(Q, K2, V2, b, T=2, n_valid=n_valid)
    assert np.allclose(O, O2, atol=1e-12)


def test_single_block_with_padding_is_masked_softmax_attention():
    Q, K, V = rand_qkv(10, 4, seed=23)
    O = mo.monarch_attention_head(Q, K, V, b=10, T=1, scale=0.5, n_valid=7)
    assert np.allclose(O, dense_softmax_attention(Q, K[:7], V[:7], 0.5), atol=1e-13)


def test_argument_errors():
    Q, K, V = rand_qkv(12, 4, seed=0)
    with pytest.raises(ValueError):
        mo.monarch_attention_head(Q, K, V, b=4, T=0)
    with pytest.raises(ValueError):
        mo.monarch_attention_head(Q, K, V, b=5, T=1)


@pytest.mark.parametrize("N,b,T", [(12, 4, 1), (16, 4, 2), (24, 6, 3), (20, 2, 2), (18, 9, 2)])
def test_objective_equals_sum_of_final_row_lse(N, b, T):
    """After the final L update the objective of Eq. 6 at the returned (L, R) is the sum over rows
    of the log-sum-exp of that update's logits (the quantity the GPU path can emit for free)."""
    rng = np.random.default_rng(N * 31 + b + T)
    Q, K, V = (rng.standard_normal((N, 5)) * 1.3 for _ in range(3))
    scale = 0.37
    _, L, R = mo.monarch_attention_head(Q, K, V, b, T, scale=scale, return_factors=True)
    f_dense = mo.objective_dense(mo.dense_monarch(L, R), Q, K, scale)
    lse = mo.final_row_lse(R, Q, K, b, scale)
    assert lse.shape == (N,)
    assert abs(lse.sum() - f_dense) < 1e-9 * max(1.0, abs(f_dense))


@pytest.mark.parametrize("N,b,T", [(12, 4, 1), (12, 3, 2), (20, 2, 2), (18, 9, 2), (24, 6, 3)])
def test_final_row_lse_is_each_rows_own_term_of_the_objective(N, b, T):
    """Row r of the dense Monarch matrix contributes sum_c M[r,c] S[r,c] - sum_c M[r,c] log M[r,c]
    to Eq. 6.  Because the final L is the exact maximiser, that term equals the log-sum-exp of row
    r's L logits.  This pins the ROW ORDER of final_row_lse (row b*l + j), with m != b: a
    transposed order passes the sum test above but not this one."""
    rng = np.random.default_rng(N * 17 + b + T)
    Q, K, V = (rng.standard_normal((N, 5)) * 1.3 for _ in range(3))
    scale = 0.41
    _, L, R = mo.monarch_attention_head(Q, K, V, b, T, scale=scale, return_factors=True)
    M = mo.dense_monarch(L, R)
    S = scale * Q @ K.T
    with np.errstate(divide="ignore", invalid="ignore"):
        ent = -np.where(M > 0, M * np.log(M), 0.0).sum(axis=1)
    per_row = (M * S).sum(axis=1) + ent
    lse = mo.final_row_lse(R, Q, K, b, scale)
    assert np.allclose(lse, per_row, rtol=0, atol=1e-10)
    if N // b != b:      # the transposed order must be told apart
        m = N // b
        assert not np.allclose(lse.reshape(m, b).T.reshape(-1), per_row, atol=1e-6)


# ---------------------------------------------------------------- sequences of different lengths
@pytest.mark.parametrize("N,b,n_valid", [(24, 4, 9), (24, 4, 12), (24, 6, 5), (20, 5, 11), (32, 4, 3)])
@pytest.mark.parametrize("T", [1, 2, 3])
def test_sequence_inside_a_longer_padding_equals_the_sequence_alone(N, b, n_valid, T):
    """App. C.3 names batches padded to a maximum length.  Reading: blocks that lie wholly in the
    padding are absent from the sequence's problem, so the valid rows must equal those of the same
    sequence run alone at its own padded length ceil(n_valid/b)*b with the appendix's mask."""
    rng = np.random.default_rng(N + 7 * n_valid + T)
    Q, K, V = (rng.standard_normal((N, 4)) * 1.2 for _ in range(3))
    own = -(-n_valid // b) * b
    alone = mo.monarch_attention_head(Q[:own], K[:own], V[:own], b, T, scale=0.5,
                                      n_valid=n_valid if n_valid < own else None)
    padded, L, R = mo.monarch_attention_head(Q, K, V, b, T, scale=0.5, n_valid=n_valid,
                                             return_factors=True)
    assert np.allclose(padded[:n_valid], alone[:n_valid], rtol=0, atol=1e-13)
    assert np.all(padded[own:] == 0.0)
    # what is unique about M: no mass on padded keys, unit mass on valid keys for the sequence's rows
    M = mo.dense_monarch(L, R)
    assert np.all(M[:, n_valid:] == 0.0)
    assert np.allclose(M[:own].sum(axis=1), 1.0, atol=1e-13)
    # garbage (even non-finite values) in the rows past the sequence's own padded length is never read
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    K2[own:] = np.nan
    V2[own:] = np.inf
    Q2[own:] = -np.inf
    again = mo.monarch_attention_head(Q2, K2, V2, b, T, scale=0.5, n_valid=n_valid)
    assert np.array_equal(again[:own], padded[:own])


def test_batched_lengths_one_per_batch_entry():
    rng = np.random.default_rng(5)
    Q, K, V = (rng.standard_normal((3, 2, 24, 4)) for _ in range(3))
    lens = np.array([24, 10, 5])
    O = mo.monarch_attention(Q, K, V, b=4, T=2, n_valid=lens)
    for e in range(3):
        for h in range(2):
            ref = mo.monarch_attention_head(Q[e, h], K[e, h], V[e, h], 4, 2, n_valid=int(lens[e]))
            assert np.array_equal(O[e, h], ref)

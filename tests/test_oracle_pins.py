"""Pins for the fp64 CPU oracle: closed forms, invariants, library routines and
brute force that do not go through the oracle's own formulas."""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import torch

from oracle import gdn_oracle as orc
from paper_2606_06034_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _chunks(C, n=4, seed=0, adversarial="none", d=128):
    inp = gen.make_inputs(1, 2, 2, C * max(1, n // 2), C, d, d, seed=seed,
                          dtype=torch.float32, adversarial_heads=adversarial)
    sl = gen.chunk_slices(inp, range(inp.n_chunks))
    K = np.stack([s[0] for s in sl])
    V = np.stack([s[1] for s in sl])
    b = np.stack([s[2] for s in sl])
    g = np.stack([s[3] for s in sl])
    return K, V, b, g


def _rand_strict_lower(k, rng, scale=1.0):
    return np.tril(rng.uniform(-scale, scale, size=(k, k)), -1)


# -- A-build -------------------------------------------------------------------
def test_build_A_reduces_to_gram_when_ungated():
    rng = np.random.default_rng(0)
    K = rng.normal(size=(8, 5))
    A = orc.build_A(K, np.ones(8), np.zeros(8))
    assert np.allclose(A, np.tril(K @ K.T, -1), atol=0, rtol=1e-15)
    assert np.all(np.triu(A) == 0)


def test_build_A_row_scaling_and_decay_direction():
    # one non-zero pair: row 2 looks back at row 0 with decay exp(g2 - g0) and beta of the ROW
    K = np.zeros((3, 2))
    K[0] = [1.0, 0.0]
    K[2] = [2.0, 0.0]
    beta = np.array([0.3, 0.5, 0.7])
    g = np.array([-0.1, -0.4, -1.1])
    A = orc.build_A(K, beta, g)
    expect = 0.7 * math.exp(-1.1 - (-0.1)) * 2.0
    assert A[2, 0] == pytest.approx(expect, rel=1e-15)
    assert np.count_nonzero(A) == 1


def test_chunk_quantities_reproduce_gated_delta_rule_recurrence():
    """U, W against the token-by-token gated delta rule they stand for.

    S_t = a_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T, a_t = exp(graw_t).
    From S_0 = 0 the state after the chunk is sum_i exp(g_C - g_i) U_i k_i^T.
    Without gates and from a state S_0 it is S_0 + sum_i (U_i - W_i S_0^T)_i k_i^T.
    """
    rng = np.random.default_rng(3)
    C, dk, dv = 16, 6, 5
    K = rng.normal(size=(C, dk))
    K /= np.linalg.norm(K, axis=1, keepdims=True)
    V = rng.normal(size=(C, dv))
    beta = 1 / (1 + np.exp(-rng.normal(size=C)))
    graw = -np.log1p(np.exp(rng.normal(size=C)))
    g = np.cumsum(graw)

    def recurrence(S0, graw_):
        S = S0.copy()
        for t in range(C):
            S = math.exp(graw_[t]) * S
            S = S - beta[t] * np.outer(S @ K[t], K[t]) + beta[t] * np.outer(V[t], K[t])
        return S

    # gated, zero initial state
    W, U, T = orc.chunk_prepare(K, V, beta, g, exact=True)
    S_end = recurrence(np.zeros((dv, dk)), graw)
    S_chunk = sum(math.exp(g[-1] - g[i]) * np.outer(U[i], K[i]) for i in range(C))
    assert np.allclose(S_end, S_chunk, atol=1e-13)

    # ungated, non-zero initial state: needs W
    W0, U0, _ = orc.chunk_prepare(K, V, beta, np.zeros(C), exact=True)
    S0 = rng.normal(size=(dv, dk))
    S_end = recurrence(S0, np.zeros(C))
    Unew = U0 - W0 @ S0.T
    S_chunk = S0 + sum(np.outer(Unew[i], K[i]) for i in range(C))
    assert np.allclose(S_end, S_chunk, atol=1e-12)

    # gated AND a non-zero initial state: needs the gated W = T diag(beta exp(g)) K
    Wg, Ug, _ = orc.chunk_prepare(K, V, beta, g, exact=True, w_gated=True)
    assert np.array_equal(Ug, U)
    S_end = recurrence(S0, graw)
    Unew = Ug - Wg @ S0.T
    S_chunk = math.exp(g[-1]) * S0 + sum(math.exp(g[-1] - g[i]) * np.outer(Unew[i], K[i]) for i in range(C))
    assert np.allclose(S_end, S_chunk, atol=1e-12)
    # and the ungated W would be wrong here
    Unew_bad = U - W @ S0.T
    S_bad = math.exp(g[-1]) * S0 + sum(math.exp(g[-1] - g[i]) * np.outer(Unew_bad[i], K[i]) for i in range(C))
    assert not np.allclose(S_end, S_bad, atol=1e-6)


def test_chunkwise_state_passing_and_output_equal_the_token_recurrence():
    """chunk_state_output (W, U given per chunk) against the token-by-token gated delta rule over several chunks,
    from a non-zero initial state, with grouped scaling; also that an ungated W or a global (not chunk-local)
    cumulative gate would be wrong, so the conventions are pinned and not just the code path."""
    rng = np.random.default_rng(11)
    C, n_chunks, dk, dv = 8, 4, 5, 6
    T = C * n_chunks
    K = rng.normal(size=(T, dk))
    K /= np.linalg.norm(K, axis=1, keepdims=True)
    Q = rng.normal(size=(T, dk))
    V = rng.normal(size=(T, dv))
    beta = 1 / (1 + np.exp(-rng.normal(size=T)))
    graw = -np.log1p(np.exp(rng.normal(size=T)))
    S0 = rng.normal(size=(dv, dk))
    O_ref, S_ref = orc.gated_delta_rule(Q, K, V, beta, graw, scale=0.7, S0=S0)
    g_local = np.cumsum(graw.reshape(n_chunks, C), axis=1).reshape(T)
    W = np.zeros((T, dk)); U = np.zeros((T, dv)); Wplain = np.zeros((T, dk))
    for c in range(n_chunks):
        sl = slice(c * C, (c + 1) * C)
        W[sl], U[sl], _ = orc.chunk_prepare(K[sl], V[sl], beta[sl], g_local[sl], exact=True, w_gated=True)
        Wplain[sl], _, _ = orc.chunk_prepare(K[sl], V[sl], beta[sl], g_local[sl], exact=True)
    O, S = orc.chunk_state_output(Q, K, W, U, g_local, C, scale=0.7, S0=S0)
    assert np.allclose(O, O_ref, atol=1e-12) and np.allclose(S, S_ref, atol=1e-12)
    # zero initial state as the default
    O0_ref, S0_ref = orc.gated_delta_rule(Q, K, V, beta, graw)
    O0, S0_end = orc.chunk_state_output(Q, K, W, U, g_local, C)
    assert np.allclose(O0, O0_ref, atol=1e-12) and np.allclose(S0_end, S0_ref, atol=1e-12)
    # conventions: the ungated W, or a cumulative gate that does not restart per chunk, give something else
    O_bad, _ = orc.chunk_state_output(Q, K, Wplain, U, g_local, C, scale=0.7, S0=S0)
    assert not np.allclose(O_bad, O_ref, atol=1e-6)
    O_bad2, _ = orc.chunk_state_output(Q, K, W, U, np.cumsum(graw), C, scale=0.7, S0=S0)
    assert not np.allclose(O_bad2, O_ref, atol=1e-6)


def test_chunkwise_output_with_a_gate_that_closes_fast_is_finite_and_equals_the_token_recurrence():
    """A gate that closes by 30 nats per token: g_i - g_j reaches +1890 above the diagonal of a 64-token chunk, where
    the sum over j <= i has no term. The chunk-wise evaluation must not touch those entries (exp would overflow and
    0 * inf would poison the output) and still equal the token-by-token rule, where each token forgets the state."""
    rng = np.random.default_rng(12)
    C, n_chunks, dk, dv = 64, 2, 4, 3
    T = C * n_chunks
    K = rng.normal(size=(T, dk))
    K /= np.linalg.norm(K, axis=1, keepdims=True)
    Q = rng.normal(size=(T, dk))
    V = rng.normal(size=(T, dv))
    beta = np.full(T, 0.5)
    graw = np.full(T, -30.0)
    S0 = rng.normal(size=(dv, dk))
    O_ref, S_ref = orc.gated_delta_rule(Q, K, V, beta, graw, scale=1.0, S0=S0)
    g_local = np.cumsum(graw.reshape(n_chunks, C), axis=1).reshape(T)
    W = np.zeros((T, dk)); U = np.zeros((T, dv))
    for c in range(n_chunks):
        sl = slice(c * C, (c + 1) * C)
        W[sl], U[sl], _ = orc.chunk_prepare(K[sl], V[sl], beta[sl], g_local[sl], exact=True, w_gated=True)
    with np.errstate(over="raise", invalid="raise"):
        O, S = orc.chunk_state_output(Q, K, W, U, g_local, C, scale=1.0, S0=S0)
    assert np.isfinite(O).all() and np.isfinite(S).all()
    assert np.allclose(O, O_ref, atol=1e-12) and np.allclose(S, S_ref, atol=1e-12)
    # every token sees (almost) only its own write: o_i = beta_i <k_i, q_i> v_i up to e^-30
    own = 0.5 * np.einsum("td,td->t", K, Q)[:, None] * V
    assert np.allclose(O, own, atol=1e-10)


def test_key_normalisation_leaves_a_zero_key_zero():
    """Normalised keys: every non-zero row has unit norm and the result equals the plain call on rows normalised by
    hand; a zero key stays zero, so its token neither reads nor writes (row and column of A vanish, its row of T is
    the unit row and W_i = 0), and nothing is NaN."""
    rng = np.random.default_rng(21)
    C, d = 16, 8
    K = rng.normal(size=(C, d)) * rng.uniform(0.2, 5.0, size=(C, 1))
    K[5] = 0.0
    V = rng.normal(size=(C, d))
    beta = rng.uniform(0.2, 0.9, size=C)
    g = np.cumsum(-rng.uniform(0.01, 0.3, size=C))
    Kn = K.copy()
    nz = np.arange(C) != 5
    Kn[nz] /= np.linalg.norm(K[nz], axis=1, keepdims=True)
    assert np.allclose(np.linalg.norm(orc.l2_normalise_rows(K)[nz], axis=1), 1.0) and not orc.l2_normalise_rows(K)[5].any()
    with np.errstate(invalid="raise", divide="raise"):
        W, U, T = orc.chunk_prepare(K, V, beta, g, exact=True, k_l2norm=True)
    W0, U0, T0 = orc.chunk_prepare(Kn, V, beta, g, exact=True)
    assert np.isfinite(W).all() and np.allclose(W, W0, atol=1e-14) and np.allclose(U, U0, atol=1e-14) and np.allclose(T, T0, atol=1e-14)
    assert not T[5, :5].any() and not T[6:, 5].any() and not W[5].any() and np.allclose(U[5], beta[5] * V[5])


def test_variable_length_sequences_equal_the_token_recurrence_per_sequence():
    """Packed sequences of ragged lengths: the chunk quantities of `chunk_prepare_varlen` (chunks counted from each
    sequence's first token, the last one short) carried through the chunk-wise state passing reproduce the
    token-by-token gated delta rule run on every sequence by itself; the padding tokens of a short chunk leave the
    state alone. Also pinned: the chunk table, and that the rows of real tokens do not depend on what a padded
    chunk holds beyond its length."""
    rng = np.random.default_rng(21)
    C, dk, dv = 8, 5, 6
    lens = [13, 8, 3, 17]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    start, length = orc.chunk_table(cu, C)
    assert start == [0, 8, 13, 21, 24, 32, 40] and length == [8, 5, 8, 3, 8, 8, 1]
    K = rng.normal(size=(T, dk))
    K /= np.linalg.norm(K, axis=1, keepdims=True)
    Q = rng.normal(size=(T, dk))
    V = rng.normal(size=(T, dv))
    beta = 1 / (1 + np.exp(-rng.normal(size=T)))
    graw = -np.log1p(np.exp(rng.normal(size=T)))
    g_local = np.zeros(T)
    for a, L in zip(start, length):
        g_local[a:a + L] = np.cumsum(graw[a:a + L])
    W, U, Tinv, st2, ln2 = orc.chunk_prepare_varlen(K, V, beta, g_local, cu, C, exact=True, w_gated=True)
    assert st2 == start and ln2 == length
    Wr, Ur, Tr, _, _ = orc.chunk_prepare_varlen(K, V, beta, graw, cu, C, exact=True, w_gated=True, g_raw=True)
    assert np.allclose(Wr, W, atol=1e-13) and np.allclose(Ur, U, atol=1e-13) and np.allclose(Tr, Tinv, atol=1e-13)
    ci = 0
    for s_, L in enumerate(lens):
        a = int(cu[s_])
        O_ref, S_ref = orc.gated_delta_rule(Q[a:a + L], K[a:a + L], V[a:a + L], beta[a:a + L], graw[a:a + L], scale=0.9)
        # the sequence padded to whole chunks: padding rows carry zero W, U, K and the gate of the last real token
        n_c = -(-L // C)
        Lp = n_c * C
        pad = lambda x: np.concatenate([x[a:a + L], np.zeros((Lp - L,) + x.shape[1:])])
        gp = pad(g_local)
        if Lp > L:
            gp[L:] = g_local[a + L - 1]
        O, S = orc.chunk_state_output(pad(Q), pad(K), pad(W), pad(U), gp, C, scale=0.9)
        assert np.allclose(O[:L], O_ref, atol=1e-12) and np.allclose(S, S_ref, atol=1e-12)
        for c in range(n_c):
            Lc = length[ci]
            # rows of padding tokens are rows of the identity, real rows never look at padding columns
            assert np.array_equal(Tinv[ci][Lc:], np.eye(C)[Lc:])
            assert np.count_nonzero(Tinv[ci][:Lc, Lc:]) == 0
            # the leading block is the exact inverse of the short chunk itself
            A = orc.build_A(K[start[ci]:start[ci] + Lc], beta[start[ci]:start[ci] + Lc], g_local[start[ci]:start[ci] + Lc])
            assert np.allclose(Tinv[ci][:Lc, :Lc], np.linalg.inv(np.eye(Lc) + A), atol=1e-12)
            ci += 1
    # lengths that are multiples of C: the packed form is the dense one
    cu2 = [0, 16, 24]
    Wd, Ud, Td, _, _ = orc.chunk_prepare_varlen(K[:24], V[:24], beta[:24], graw[:24], cu2, C, 3, 2, g_raw=True)
    Wc, Uc, Tc = orc.chunk_prepare(K[:24].reshape(3, C, dk), V[:24].reshape(3, C, dv), beta[:24].reshape(3, C),
                                   graw[:24].reshape(3, C), 3, 2, g_raw=True)
    assert np.array_equal(Wd, Wc.reshape(24, dk)) and np.array_equal(Ud, Uc.reshape(24, dv)) and np.array_equal(Td, Tc)


# -- P2 / P12: exact inverse -----------------------------------------------------
def test_forward_substitution_closed_forms_c2_c3():
    a = 0.37
    T = orc.exact_inverse(np.array([[0, 0], [a, 0.0]]))
    assert np.array_equal(T, np.array([[1, 0], [-a, 1.0]]))
    a21, a31, a32 = 0.2, -0.5, 0.7
    A = np.array([[0, 0, 0], [a21, 0, 0], [a31, a32, 0.0]])
    T = orc.exact_inverse(A)
    expect = np.array([[1, 0, 0], [-a21, 1, 0], [a32 * a21 - a31, -a32, 1.0]])
    assert np.allclose(T, expect, atol=1e-16)


@pytest.mark.parametrize("k", [2, 3, 4, 8, 16, 64])
def test_forward_substitution_matches_library_inverse(k):
    rng = np.random.default_rng(k)
    A = _rand_strict_lower(k, rng, 0.3)
    T = orc.exact_inverse(A)
    I = np.eye(k)
    assert np.allclose((I + A) @ T, I, atol=1e-12)
    assert np.allclose(T, np.linalg.inv(I + A), atol=1e-12)
    assert np.allclose(T, scipy.linalg.solve_triangular(I + A, I, lower=True), atol=1e-12)


def test_forward_substitution_batched_equals_single():
    rng = np.random.default_rng(5)
    A = np.stack([_rand_strict_lower(8, rng) for _ in range(3)])
    Tb = orc.exact_inverse(A)
    for i in range(3):
        assert np.array_equal(Tb[i], orc.exact_inverse(A[i]))


# -- P1: nilpotency --------------------------------------------------------------
@pytest.mark.parametrize("C", [16, 32, 64])
def test_full_neumann_series_is_the_exact_inverse_benign(C):
    K, V, b, g = _chunks(C)
    A = orc.build_A(K, b, g)
    Abar = -A
    assert np.allclose(orc.neumann_full(Abar), orc.forward_substitution_inverse(Abar), atol=1e-13)
    # A^k = 0
    P = np.linalg.matrix_power(Abar[0], C)
    assert np.all(P == 0)


def test_full_neumann_series_exact_on_small_adversarial():
    K, V, b, g = _chunks(16, adversarial="all")
    Abar = -orc.build_A(K, b, g)
    assert np.allclose(orc.neumann_full(Abar), orc.forward_substitution_inverse(Abar), atol=1e-9)


# -- P3 / P4: structure ------------------------------------------------------------
@pytest.mark.parametrize("C,N,S", [(64, 3, 8), (32, 3, 4), (32, 4, 3), (16, 3, 3), (16, 3, 2), (64, 2, 5)])
@pytest.mark.parametrize("adv", ["none", "all"])
def test_band_and_residual_structure(C, N, S, adv):
    K, V, b, g = _chunks(C, adversarial=adv)
    Abar = -orc.build_A(K, b, g)
    Tex = orc.forward_substitution_inverse(Abar)
    T0 = orc.neumann_masked_init(Abar, N)
    i = np.arange(C)[:, None]
    j = np.arange(C)[None, :]
    d = i - j
    band = (d >= 0) & (d <= N)
    scale = max(1.0, np.abs(Tex).max())
    # the masked initial approximation is exact on its band and zero off it
    assert np.allclose(T0[..., band], Tex[..., band], atol=1e-12 * scale)
    assert np.all(T0[..., ~band] == 0)
    # E vanishes inside the band (up to rounding of cancelling terms), E^s below s(N+1)
    E = orc.residual_matrix(Abar, T0)
    assert np.abs(E[..., d <= N]).max() <= 1e-12 * scale
    Es = E.copy()
    for s in range(2, 5):
        Es = Es @ E
        tol = 1e-11 * max(1.0, np.abs(Es).max())
        assert np.abs(Es[..., d < s * (N + 1)]).max() <= tol
    # T_{N,S} is exact on i - j < (S+1)(N+1)
    Tns = orc.neumann_residual(Abar, N, S)
    near = d < (S + 1) * (N + 1)
    assert np.allclose(Tns[..., near], Tex[..., near], atol=1e-10 * scale)
    # and everywhere once S reaches ceil(C/(N+1)) - 1
    Sfull = math.ceil(C / (N + 1)) - 1
    Tfull = orc.neumann_residual(Abar, N, Sfull)
    assert np.allclose(Tfull, Tex, atol=1e-10 * scale)


# -- P5: the truncation error is the dropped terms ---------------------------------
@pytest.mark.parametrize("C,N,S", [(64, 3, 2), (64, 3, 8), (32, 2, 3), (16, 1, 2)])
def test_truncation_error_equals_dropped_terms(C, N, S):
    K, V, b, g = _chunks(C, seed=7)
    Abar = -orc.build_A(K, b, g)
    Tex = orc.forward_substitution_inverse(Abar)
    T0 = orc.neumann_masked_init(Abar, N)
    E = orc.residual_matrix(Abar, T0)
    Tns = orc.neumann_residual(Abar, N, S)
    dropped = np.zeros_like(E)
    P = np.broadcast_to(np.eye(C), E.shape).copy()
    for s in range(1, math.ceil(C / (N + 1))):
        P = P @ E
        if s > S:
            dropped = dropped + P
    assert np.allclose(Tex - Tns, T0 @ dropped, atol=1e-13)
    if S < math.ceil(C / (N + 1)) - 1 and C == 64 and S == 2:
        assert np.abs(Tex - Tns).max() > 1e-9  # the truncated form really differs


# -- P6: pairing of E and the side of the product -----------------------------------
def test_right_and_left_consistent_agree_alg1_verbatim_does_not():
    K, V, b, g = _chunks(64, seed=11)
    Abar = -orc.build_A(K, b, g)
    Tex = orc.forward_substitution_inverse(Abar)
    R = orc.neumann_residual(Abar, 3, 4, side="right")
    L = orc.neumann_residual(Abar, 3, 4, side="left_consistent")
    Vb = orc.neumann_residual(Abar, 3, 4, side="alg1_verbatim")
    assert np.allclose(R, L, atol=1e-14)
    err_r = orc.rel_frobenius(R, Tex).max()
    err_v = orc.rel_frobenius(Vb, Tex).min()
    assert err_v > 1e3 * max(err_r, 1e-16)


# -- P7: iterative residual correction = power sum with S = 2^m - 1 -----------------
@pytest.mark.parametrize("m", [1, 2, 3])
def test_iterative_correction_equals_power_sum(m):
    K, V, b, g = _chunks(64, seed=13)
    Abar = -orc.build_A(K, b, g)
    it = orc.iterative_residual(Abar, 3, m)
    ps = orc.neumann_residual(Abar, 3, 2 ** m - 1)
    assert np.allclose(it, ps, atol=1e-14)


def test_factorised_power_sum_matches_plain_sum():
    rng = np.random.default_rng(17)
    E = _rand_strict_lower(32, rng, 0.2)
    assert np.allclose(orc.factorised_power_sum(E, 3), orc.power_sum(E, 7), atol=1e-14)


# -- P8: entrywise growth (Lemma 3) -------------------------------------------------
def test_binomial_growth_tight_for_all_ones():
    k = 24
    L = np.tril(np.ones((k, k)), -1)
    P = np.eye(k)
    for n in range(1, 8):
        P = P @ L
        for i in range(k):
            for j in range(k):
                d = i - j
                expect = math.comb(d - 1, n - 1) if d >= 1 else 0
                assert P[i, j] == expect
    # the oracle's running sum sees the same numbers: sum_{n<=N} L^n entries
    T0 = orc.neumann_masked_init(L, 3, mask=False)
    assert T0[10, 2] == sum(math.comb(7, n - 1) for n in range(1, 4))


def test_binomial_growth_bounds_bounded_entries():
    rng = np.random.default_rng(19)
    k = 20
    A = _rand_strict_lower(k, rng, 1.0)
    P = np.eye(k)
    for n in range(1, 6):
        P = P @ A
        for i in range(k):
            for j in range(i):
                assert abs(P[i, j]) <= math.comb(i - j - 1, n - 1) + 1e-12


# -- P9: closed form reachable through the whole path -------------------------------
@pytest.mark.parametrize("a", [0.25, 0.99, 1.0])
@pytest.mark.parametrize("C", [16, 64])
def test_identical_keys_closed_form(a, C):
    rng = np.random.default_rng(23)
    u = rng.normal(size=8)
    u /= np.linalg.norm(u)
    K = np.tile(u, (C, 1))
    V = rng.normal(size=(C, 4))
    W, U, T = orc.chunk_prepare(K, V, np.full(C, a), np.zeros(C),
                                N=3, S=math.ceil(C / 4) - 1)
    i = np.arange(C)[:, None]
    j = np.arange(C)[None, :]
    d = i - j
    expect = np.where(d > 0, -a * (1 - a) ** np.maximum(d - 1, 0), 0.0) + np.eye(C)
    if a == 1.0:
        expect = np.eye(C) - np.eye(C, k=-1)
    assert np.allclose(T, expect, atol=1e-9)
    assert np.allclose(W, (a * (1 - a) ** np.arange(C))[:, None] * u[None, :], atol=1e-9)
    # U_i = a (v_i - sum_{j<i} U_j): running form of the same system
    Uref = np.zeros_like(V)
    run = np.zeros(4)
    for t in range(C):
        Uref[t] = a * (V[t] - run)
        run = run + Uref[t]
    assert np.allclose(U, Uref, atol=1e-8)


# -- P10: truncation bound (Lemma 2) -------------------------------------------------
def test_truncation_norm_bound():
    rng = np.random.default_rng(29)
    k = 64
    i = np.arange(k)[:, None]
    j = np.arange(k)[None, :]
    A = np.where(i > j, rng.uniform(0, 1, size=(k, k)) * 0.8 ** (i - j), 0.0)
    A *= 0.55 / np.linalg.norm(A, 2)
    Tex = orc.neumann_full(A)
    for N in (1, 3, 5, 8):
        EN = Tex - orc.neumann_full(A, upto=N)
        bound = 0.55 ** (N + 1) / (1 - 0.55)
        assert np.linalg.norm(EN, 2) <= bound * (1 + 1e-12)
        assert np.allclose(EN, sum(np.linalg.matrix_power(A, n) for n in range(N + 1, k)), atol=1e-14)


# -- P11: matmul counts the paper prints ----------------------------------------------
def test_matmul_counts_match_paper():
    rows = []
    with open(os.path.join(GOLDEN, "paper_matmul_counts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append(tuple(int(x) for x in line.split()))
    assert rows
    for k, N, S, count in rows:
        rng = np.random.default_rng(k)
        A = _rand_strict_lower(k, rng, 0.1)
        orc.reset_matmul_count()
        orc.neumann_residual(A, N, S)
        assert orc.matmul_count() == count
        assert orc.default_order(k) == N and orc.default_residual_steps(k) == S


# -- P13: block formula (App. E) --------------------------------------------------------
def test_block_formula_reproduces_exact_inverse_with_exact_blocks():
    K, V, b, g = _chunks(128, n=2, seed=31)
    A = orc.build_A(K, b, g)
    Tex = orc.exact_inverse(A)
    # 64-blocks inverted exactly (S large enough), merged by the block formula
    Tb = orc.chunk_inverse(A, 3, 15, block=64)
    assert np.allclose(Tb, Tex, atol=1e-12)
    # four 32-blocks exercise the general recursion (Eq. 27)
    Tb4 = orc.chunk_inverse(A, 3, 7, block=32)
    assert np.allclose(Tb4, Tex, atol=1e-12)
    # the two-block corner: S_21 = -S_22 M_21 S_11
    T11 = orc.exact_inverse(A[..., :64, :64])
    T22 = orc.exact_inverse(A[..., 64:, 64:])
    assert np.allclose(Tex[..., 64:, :64], -T22 @ A[..., 64:, :64] @ T11, atol=1e-12)
    assert np.all(Tb[..., :64, 64:] == 0)


# -- defaults: truncation invisible at the graded tolerance ---------------------------
@pytest.mark.parametrize("C", [16, 32, 64, 128])
@pytest.mark.parametrize("adv", ["none", "all"])
def test_default_parameters_deviation_from_exact(C, adv):
    K, V, b, g = _chunks(C, n=2, seed=37, adversarial=adv)
    W, U, T = orc.chunk_prepare(K, V, b, g)
    We, Ue, Te = orc.chunk_prepare(K, V, b, g, exact=True)
    assert orc.rel_frobenius(T, Te).max() < 1e-9
    assert orc.rel_frobenius(W, We).max() < 1e-8
    assert orc.rel_frobenius(U, Ue).max() < 1e-8
    # W, U are T applied to the beta-scaled rows
    assert np.allclose(W, T @ (b[..., None] * K), atol=1e-13)


def test_snr_definition():
    ref = np.ones((2, 2))
    x = ref + 0.1
    # ||ref||^2 / ||ref - x||^2 = 4 / 0.04 = 100 -> 20 dB
    assert orc.snr_db(x, ref) == pytest.approx(20.0, abs=1e-9)


# -- input recipe --------------------------------------------------------------------
def test_input_recipe():
    inp = gen.make_inputs(2, 2, 4, 128, 64, 128, 128, seed=4, adversarial_heads="odd")
    assert inp.K.dtype == torch.bfloat16 and inp.K.shape == (2, 2, 128, 128)
    assert inp.V.shape == (2, 4, 128, 128) and inp.beta.shape == (2, 4, 128)
    n = inp.K.float().norm(dim=-1)
    assert torch.allclose(n, torch.ones_like(n), atol=1e-2)
    # cumulative gate restarts at each chunk and decreases
    gch = inp.g.view(2, 4, 2, 64)
    assert (gch[:, :2].diff(dim=-1) <= 0).all()
    # odd key head / its value heads are adversarial
    assert (inp.beta[:, 2:] == 0.99).all() and (inp.g[:, 2:] == 0).all()
    Kc = inp.K[0, 1, :64].float()
    cos = Kc @ Kc.T
    assert cos.min() > 0.95
    # seeded
    again = gen.make_inputs(2, 2, 4, 128, 64, 128, 128, seed=4, adversarial_heads="odd")
    assert torch.equal(inp.K, again.K) and torch.equal(inp.g, again.g)


# -- optional prologue (raw gates, key normalisation) reduces to the plain path on prepared inputs --------
def test_prologue_flags_reduce_to_prepared_inputs():
    rng = np.random.default_rng(41)
    C = 16
    K = rng.normal(size=(3, C, 8)) * rng.uniform(0.5, 3.0, size=(3, C, 1))
    V = rng.normal(size=(3, C, 4))
    beta = rng.uniform(0.1, 0.9, size=(3, C))
    graw = -rng.uniform(0.0, 0.5, size=(3, C))
    W1, U1, T1 = orc.chunk_prepare(K, V, beta, graw, g_raw=True, k_l2norm=True)
    Kn = K / np.linalg.norm(K, axis=-1, keepdims=True)
    gc = np.stack([[sum(row[:i + 1]) for i in range(C)] for row in graw])
    W2, U2, T2 = orc.chunk_prepare(Kn, V, beta, gc)
    assert np.allclose(T1, T2, atol=1e-14) and np.allclose(W1, W2, atol=1e-14) and np.allclose(U1, U2, atol=1e-14)
    # normalisation matters: without it the result differs
    W3, _, T3 = orc.chunk_prepare(K, V, beta, gc)
    assert np.abs(T3 - T2).max() > 1e-3

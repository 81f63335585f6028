"""CPU oracle for the chunk-prepare path of chunk-wise Gated DeltaNet (fp64).

TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition the CUDA
path is checked against. Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the product path never does, and it shares no
code with the CUDA sources.

What is computed, per chunk of C tokens (K: C x d_k, V: C x d_v, beta: C,
g: C cumulative log-gate), all in fp64:

  A        strictly lower triangular, A_ij = beta_i * exp(g_i - g_j) * <K_i, K_j>
           for i > j (the "scaled inner product" of Sec. 2.1 with the Gated
           DeltaNet write strength and gate decay).
  Abar     = -A. The paper inverts I - A (Eq. 1); chunk-wise Gated DeltaNet
           inverts I + A, so every formula of the paper is applied to Abar.
  T_exact  = (I - Abar)^-1 by forward substitution (Eq. 2-3).
  T_NS     the paper's multiplication-only approximation (Sec. 3, Alg. 1):
             T0 = M^(N) o sum_{n=0..N} Abar^n      (Eq. 7, 10, 11)
             E  = I - (I - Abar) T0                (Eq. 13)
             T  = T0 * sum_{s=0..S} E^s            (Eq. 13, right product)
  C = 128  two 64 x 64 diagonal blocks by the scheme above and the block
           formula of App. E (Eq. 28) for the lower-left block.
  W, U     = T diag(beta) K,  T diag(beta) V.

Readings of the paper taken here (each also listed in the design notes):
  * Alg. 1's last line multiplies the power sum on the LEFT of T0 while Eq. 13
    and App. D put it on the right; with E = I - (I - Abar) T0 only the right
    product is consistent, so the right product is used
    (`neumann_residual(..., side="right")`; "left_consistent" and
    "alg1_verbatim" exist for the pin that tells them apart).
  * The residual sum runs s = 0..S (S+1 terms); this reproduces the paper's
    matmul counts 11 at (N, S) = (3, 8) and 7 at (3, 4) (Sec. 4.3).
  * The mask keeps 0 <= i - j <= N (Eq. 10 with K = N); the upper triangle is
    zero anyway.
  * Lemma 1 is read as i - j < n  =>  (A^n)_ij = 0.

Every function is pinned in tests/test_oracle_pins.py against closed forms,
brute force and library routines; nothing here is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------
# matmul wrapper with a counter, so that the number of matrix products of
# Alg. 1 can be compared with the counts the paper prints (Sec. 4.3).
# ----------------------------------------------------------------------------
_MATMUL_COUNT = 0


def _mm(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    global _MATMUL_COUNT
    _MATMUL_COUNT += 1
    return np.matmul(a, b)


def reset_matmul_count() -> None:
    global _MATMUL_COUNT
    _MATMUL_COUNT = 0


def matmul_count() -> int:
    return _MATMUL_COUNT


# ----------------------------------------------------------------------------
# A-build (Sec. 2.1 with the Gated DeltaNet beta / gate factors)
# ----------------------------------------------------------------------------
def build_A(K: np.ndarray, beta: np.ndarray, g: np.ndarray) -> np.ndarray:
    """A = tril(diag(beta) (K K^T o Gamma), -1), Gamma_ij = exp(g_i - g_j).

    K: [..., C, d], beta, g: [..., C]. Returns [..., C, C] fp64.
    """
    K = np.asarray(K, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    C = K.shape[-2]
    G = np.matmul(K, np.swapaxes(K, -1, -2))
    i = np.arange(C)[:, None]
    j = np.arange(C)[None, :]
    lower = i > j
    # exponent only where it is used: g_i - g_j <= 0 for i > j with non-increasing g
    diff = np.where(lower, g[..., :, None] - g[..., None, :], 0.0)
    A = beta[..., :, None] * np.exp(diff) * G
    return np.where(lower, A, 0.0)


# ----------------------------------------------------------------------------
# Exact inverse by forward substitution (Eq. 2-3)
# ----------------------------------------------------------------------------
def forward_substitution_inverse(Abar: np.ndarray) -> np.ndarray:
    """(I - Abar)^-1 for strictly lower triangular Abar, rows in order.

    Eq. 2: row i of the working matrix (initialised to Abar) gets its own
    product with the already final leading i x i block added; Eq. 3 adds I.
    """
    Abar = np.asarray(Abar, dtype=np.float64)
    k = Abar.shape[-1]
    X = Abar.copy()
    for i in range(1, k):
        X[..., i, :i] = X[..., i, :i] + np.einsum("...k,...kj->...j", X[..., i, :i], X[..., :i, :i])
    return X + np.eye(k)


# ----------------------------------------------------------------------------
# Neumann pieces (Sec. 2.3, Sec. 3)
# ----------------------------------------------------------------------------
def neumann_full(Abar: np.ndarray, upto: int | None = None) -> np.ndarray:
    """sum_{n=0}^{upto} Abar^n (Eq. 4-6); upto = k-1 gives the exact inverse."""
    Abar = np.asarray(Abar, dtype=np.float64)
    k = Abar.shape[-1]
    if upto is None:
        upto = k - 1
    I = np.broadcast_to(np.eye(k), Abar.shape)
    total = I.copy()
    P = I.copy()
    for _ in range(upto):
        P = np.matmul(P, Abar)
        total = total + P
    return total


def band_mask(k: int, width: int) -> np.ndarray:
    """M^(width)_ij = 1 iff 0 <= i - j <= width (Eq. 10)."""
    i = np.arange(k)[:, None]
    j = np.arange(k)[None, :]
    return ((i - j >= 0) & (i - j <= width)).astype(np.float64)


def neumann_masked_init(Abar: np.ndarray, N: int, mask: bool = True) -> np.ndarray:
    """T0 = M^(N) o sum_{n=0}^{N} Abar^n (Eq. 11), powers as in Alg. 1.

    Alg. 1 starts P = I and multiplies N times; the first product (I * Abar)
    is a copy and is not counted as a matrix product.
    """
    Abar = np.asarray(Abar, dtype=np.float64)
    k = Abar.shape[-1]
    I = np.broadcast_to(np.eye(k), Abar.shape)
    T0 = I.copy()
    P = None
    for n in range(1, N + 1):
        P = Abar.copy() if n == 1 else _mm(P, Abar)
        T0 = T0 + P
    if mask:
        T0 = T0 * band_mask(k, N)
    return T0


def residual_matrix(Abar: np.ndarray, T0: np.ndarray, side: str = "right") -> np.ndarray:
    """E = I - (I - Abar) T0 (Eq. 13); side="left_consistent": I - T0 (I - Abar)."""
    k = Abar.shape[-1]
    I = np.eye(k)
    if side == "left_consistent":
        return I - _mm(T0, I - Abar)
    return I - _mm(I - Abar, T0)


def power_sum(E: np.ndarray, S: int) -> np.ndarray:
    """sum_{s=0}^{S} E^s, accumulated as in Alg. 1 (first product is a copy)."""
    k = E.shape[-1]
    I = np.broadcast_to(np.eye(k), E.shape)
    total = I.copy()
    P = None
    for s in range(1, S + 1):
        P = E.copy() if s == 1 else _mm(P, E)
        total = total + P
    return total


def neumann_residual(Abar: np.ndarray, N: int, S: int, *, side: str = "right",
                     mask: bool = True) -> np.ndarray:
    """The paper's approximation of (I - Abar)^-1 with order N and S residual terms.

    side = "right"           T0 * sum E^s, E = I - (I - Abar) T0   (Eq. 13, App. D)
    side = "left_consistent" (sum E_L^s) * T0, E_L = I - T0 (I - Abar)
    side = "alg1_verbatim"   (sum E^s) * T0 with E = I - (I - Abar) T0, the
                             printed last line of Alg. 1 (inconsistent pairing)
    """
    Abar = np.asarray(Abar, dtype=np.float64)
    T0 = neumann_masked_init(Abar, N, mask=mask)
    if side == "right":
        E = residual_matrix(Abar, T0, "right")
        return _mm(T0, power_sum(E, S))
    if side == "left_consistent":
        E = residual_matrix(Abar, T0, "left_consistent")
        return _mm(power_sum(E, S), T0)
    if side == "alg1_verbatim":
        E = residual_matrix(Abar, T0, "right")
        return _mm(power_sum(E, S), T0)
    raise ValueError(side)


def iterative_residual(Abar: np.ndarray, N: int, iters: int) -> np.ndarray:
    """Eq. 12: R = I - (I - Abar) T; T <- T + T R, `iters` times from T0."""
    Abar = np.asarray(Abar, dtype=np.float64)
    k = Abar.shape[-1]
    I = np.eye(k)
    T = neumann_masked_init(Abar, N)
    for _ in range(iters):
        R = I - np.matmul(I - Abar, T)
        T = T + np.matmul(T, R)
    return T


def factorised_power_sum(E: np.ndarray, levels: int) -> np.ndarray:
    """prod_{l=0}^{levels-1} (I + E^(2^l)) = sum_{s=0}^{2^levels - 1} E^s (App. F)."""
    k = E.shape[-1]
    I = np.broadcast_to(np.eye(k), E.shape)
    Gs = I.copy()
    P = np.asarray(E, dtype=np.float64)
    for _ in range(levels):
        Gs = np.matmul(Gs, I + P)
        P = np.matmul(P, P)
    return Gs


# ----------------------------------------------------------------------------
# Defaults per chunk size (Sec. 4.1, Sec. 4.3, App. H)
# ----------------------------------------------------------------------------
def default_order(C: int) -> int:
    return 3


def default_residual_steps(C: int) -> int:
    """C = 64 -> 8 (Sec. 4.1); C = 32 -> 4 (Sec. 4.3); C = 128 uses 64-blocks -> 8.

    C = 16 is not in the paper; S = 3 makes (S+1)(N+1) >= C, i.e. the result exact.
    """
    return {16: 3, 32: 4, 64: 8, 128: 8}.get(C, max(0, math.ceil(C / 4) - 1))


# ----------------------------------------------------------------------------
# Whole inverse for one chunk size, including the C = 128 block form (App. E)
# ----------------------------------------------------------------------------
def chunk_inverse(A: np.ndarray, N: int, S: int, block: int | None = None) -> np.ndarray:
    """Approximate (I + A)^-1 by the paper's scheme; A: [..., C, C].

    If block is given and smaller than C, the diagonal blocks of that size are
    inverted by the scheme and the lower-left blocks follow from the block
    forward substitution of App. E (Eq. 27; Eq. 28 for two blocks):
        S_ij = -S_ii * sum_{k=j}^{i-1} M_ik S_kj,   M = I + A.
    """
    A = np.asarray(A, dtype=np.float64)
    C = A.shape[-1]
    if block is None or block >= C:
        return neumann_residual(-A, N, S)
    assert C % block == 0
    nb = C // block
    Sinv = np.zeros_like(A)

    def blk(M, i, j):
        return M[..., i * block:(i + 1) * block, j * block:(j + 1) * block]

    for i in range(nb):
        blk(Sinv, i, i)[...] = neumann_residual(-blk(A, i, i), N, S)
    for i in range(nb):
        for j in range(i - 1, -1, -1):
            acc = np.zeros_like(blk(A, i, j))
            for k in range(j, i):
                acc = acc + np.matmul(blk(A, i, k), blk(Sinv, k, j))
            blk(Sinv, i, j)[...] = -np.matmul(blk(Sinv, i, i), acc)
    return Sinv


def exact_inverse(A: np.ndarray) -> np.ndarray:
    """(I + A)^-1 by forward substitution (Eq. 2-3 applied to Abar = -A)."""
    return forward_substitution_inverse(-np.asarray(A, dtype=np.float64))


def l2_normalise_rows(K: np.ndarray) -> np.ndarray:
    """Rows of K divided by their Euclidean norm (Sec. 2.1). The paper does not say what a zero key becomes: it stays
    zero here (a token that writes nothing), as the usual normalise-with-epsilon routines leave it."""
    norm = np.sqrt((K * K).sum(axis=-1, keepdims=True))
    return np.divide(K, norm, out=np.zeros_like(K), where=norm > 0)


def chunk_prepare(K, V, beta, g, N: int | None = None, S: int | None = None, *,
                  exact: bool = False, g_raw: bool = False, k_l2norm: bool = False, w_gated: bool = False):
    """One chunk or a stack of chunks: returns (W, U, T), all fp64.

    K: [..., C, d_k], V: [..., C, d_v], beta, g: [..., C].
    exact=False: T by the paper's scheme (order N, S residual terms; C = 128 by
    64-blocks). exact=True: T by forward substitution.
    W = T diag(beta) K, U = T diag(beta) V.
    g_raw: g holds raw log-gates (prefix-summed here). k_l2norm: rows of K are
    normalised here (W uses the normalised keys). w_gated: W = T diag(beta * exp(g)) K,
    the form in which the chunk-wise state update consumes W (U_new = U - W S_0^T for a
    state S_0 carried into the chunk); U is unchanged.
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    C = K.shape[-2]
    if g_raw:
        # g holds the raw per-token log-gates: the cumulative gate is their prefix sum inside the chunk
        g = np.cumsum(g, axis=-1)
    if k_l2norm:
        # keys are l2-normalised before the path (Sec. 2.1)
        K = l2_normalise_rows(K)
    A = build_A(K, beta, g)
    if exact:
        T = exact_inverse(A)
    else:
        N = default_order(C) if N is None or N < 0 else N
        S = default_residual_steps(C) if S is None or S < 0 else S
        T = chunk_inverse(A, N, S, block=64 if C == 128 else None)
    wscale = beta * np.exp(g) if w_gated else beta
    W = np.matmul(T, wscale[..., :, None] * K)
    U = np.matmul(T, beta[..., :, None] * V)
    return W, U, T


def chunk_table(cu_seqlens, C: int):
    """Chunks of packed variable-length sequences: sequence s holds tokens [cu_seqlens[s], cu_seqlens[s+1]) and is cut
    into chunks of C tokens from its own first token; its last chunk may be shorter. Returns (start, length) lists."""
    start, length = [], []
    for s in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        assert b >= a
        for t0 in range(a, b, C):
            start.append(t0)
            length.append(min(C, b - t0))
    return start, length


def chunk_prepare_varlen(K, V, beta, g, cu_seqlens, C: int, N: int | None = None, S: int | None = None, *,
                         exact: bool = False, g_raw: bool = False, k_l2norm: bool = False, w_gated: bool = False):
    """One head of packed variable-length sequences: K [T, d_k], V [T, d_v], beta, g [T] (g: cumulative log-gate
    restarting in every chunk, chunks counted from each sequence's first token; or raw with g_raw).

    A chunk shorter than C is the chunk of C tokens whose missing tokens write nothing: beta = 0, zero key and
    value, no further decay (raw log-gate 0, i.e. the cumulative gate of the last real token). The scheme of
    `chunk_prepare` is applied to that padded chunk and the rows of the real tokens are kept.
    Returns (W [T, d_k], U [T, d_v], Tinv [n_chunks, C, C], start, length).
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    if k_l2norm:
        K = l2_normalise_rows(K)
    start, length = chunk_table(cu_seqlens, C)
    W = np.zeros_like(K)
    U = np.zeros_like(V)
    Tinv = np.zeros((len(start), C, C))
    for c, (a, L) in enumerate(zip(start, length)):
        Kc = np.zeros((C, K.shape[1])); Vc = np.zeros((C, V.shape[1])); bc = np.zeros(C); gc = np.zeros(C)
        Kc[:L] = K[a:a + L]; Vc[:L] = V[a:a + L]; bc[:L] = beta[a:a + L]; gc[:L] = g[a:a + L]
        if not g_raw:
            gc[L:] = gc[L - 1]
        Wc, Uc, Tc = chunk_prepare(Kc, Vc, bc, gc, N, S, exact=exact, g_raw=g_raw, w_gated=w_gated)
        W[a:a + L] = Wc[:L]
        U[a:a + L] = Uc[:L]
        Tinv[c] = Tc
    return W, U, Tinv, start, length


# ----------------------------------------------------------------------------
# The rest of the chunk-wise layer: state passing and output, given W and U
# ----------------------------------------------------------------------------
def gated_delta_rule(Q, K, V, beta, g_raw, scale: float = 1.0, S0=None):
    """Token-by-token gated delta rule, the definition the chunk-wise form stands for.

    Q, K: [T, d_k]; V: [T, d_v]; beta, g_raw (raw per-token log-gates): [T].
    State S is [d_v, d_k]:  S_t = a_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,  a_t = exp(g_raw_t),
    output o_t = scale * S_t q_t. Returns (O [T, d_v], S_T).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    g_raw = np.asarray(g_raw, dtype=np.float64)
    T, dv = V.shape
    S = np.zeros((dv, K.shape[1])) if S0 is None else np.array(S0, dtype=np.float64)
    O = np.zeros((T, dv))
    for t in range(T):
        S = math.exp(g_raw[t]) * S
        S = S - beta[t] * np.outer(S @ K[t], K[t]) + beta[t] * np.outer(V[t], K[t])
        O[t] = scale * (S @ Q[t])
    return O, S


def chunk_state_output(Q, K, W_gated, U, g, C: int, scale: float = 1.0, S0=None):
    """Chunk-wise state passing and output of one (batch, head) sequence, given W and U of every chunk.

    Q, K, W_gated: [T, d_k]; U: [T, d_v]; g: [T] cumulative log-gate, CHUNK-LOCAL (inclusive prefix sum that
    restarts in every chunk of C tokens). W_gated = T diag(beta exp(g)) K, U = T diag(beta) V.
    Per chunk, with S0 the state [d_v, d_k] carried in:
        U_new = U - W_gated S0^T
        o_i   = scale * ( exp(g_i) S0 q_i + sum_{j <= i} exp(g_i - g_j) <k_j, q_i> U_new_j )
        S_end = exp(g_C) S0 + sum_j exp(g_C - g_j) U_new_j k_j^T        (g_C: the chunk's last g)
    Returns (O [T, d_v], S after the last chunk).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    W_gated = np.asarray(W_gated, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    T, dv = U.shape
    assert T % C == 0
    S = np.zeros((dv, K.shape[1])) if S0 is None else np.array(S0, dtype=np.float64)
    O = np.zeros((T, dv))
    causal = np.tril(np.ones((C, C), dtype=bool))
    for c in range(T // C):
        sl = slice(c * C, (c + 1) * C)
        q, k, w, u, gc = Q[sl], K[sl], W_gated[sl], U[sl], g[sl]
        u_new = u - w @ S.T
        # the sum runs over j <= i only: the decay factor is not evaluated above the diagonal (g_i - g_j > 0 there, and a
        # gate that closes fast would overflow the exponential and leave 0 * inf)
        P = (q @ k.T) * np.exp(np.where(causal, gc[:, None] - gc[None, :], -np.inf))
        O[sl] = scale * (np.exp(gc)[:, None] * (q @ S.T) + P @ u_new)
        S = math.exp(gc[-1]) * S + (u_new * np.exp(gc[-1] - gc)[:, None]).T @ k
    return O, S


# ----------------------------------------------------------------------------
# Error measures used by the tests and reports
# ----------------------------------------------------------------------------
def rel_frobenius(x: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """||x - ref||_F / ||ref||_F over the last two axes (per chunk)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    num = np.sqrt(((x - ref) ** 2).sum(axis=(-1, -2)))
    den = np.sqrt((ref ** 2).sum(axis=(-1, -2)))
    return num / np.maximum(den, 1e-300)


def snr_db(x: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """10 log10(||ref||^2 / ||ref - x||^2), the paper's accuracy measure (Sec. 4.2)."""
    r = rel_frobenius(x, ref)
    return -20.0 * np.log10(np.maximum(r, 1e-300))

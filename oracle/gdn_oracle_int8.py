"""CPU oracle for the INT8 variant of the chunk-prepare path (exact integer arithmetic).

TEST INFRASTRUCTURE ONLY: only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this file; it shares no code with the CUDA sources.

The paper fixes little about its low-bit variant: a uniform symmetric quantiser
q(x) = clip(round(x / Delta), qmin, qmax) (App. G, Eq. 32), one scale per tensor for the inverse
(App. G table), a truncation order N <= 3 compensated by residual correction (Sec. 3.5), the band
mask that removes the outliers min-max scales are sensitive to (Sec. 3.3), and the remark that the
chain re-applies quantisation at every step (Sec. 3.5). Everything else is a reading of this build,
chosen so that both sides can evaluate it bit for bit ("block floating point, 8-bit mantissas"):

  * every tensor is int8 mantissas in [-127, 127] with ONE power-of-two exponent per chunk
    (Delta = 2^e, chosen from the tensor's own maximum: dynamic per-tensor scale);
  * the identity is never quantised (T = I + Toff), the structural mask is applied BEFORE each
    requantisation (only the structurally non-zero support decides the scale);
  * round = round half away from zero, range +-127;
  * the gate decay exp(g_i - g_j) is a 256-entry table of 2^(-f/256) in 1.15 fixed point plus a shift.

Definitions (Python integers or int64; every product that a tensor-core MMA would form fits int32):

  rsr(x, r)    = sign(x) * ((|x| + 2^(r-1)) >> r),  rsr(x, 0) = x
  Q8(acc, e)   : m = max|acc| over the support, r = max(0, bitlen(m) - 7),
                 q = clamp(rsr(acc, r), -127, 127), exponent e + r
  align(terms) : e_ref = max(min e, max e - 8); x_i shifted left by e_i - e_ref (rsr if negative); summed.
                 Eight bits below the largest term are kept: the sum is requantised to 8 bits right after, so
                 finer bits cannot matter (measured: same SNR as a 24-bit window), and every sum fits int32.

Steps per chunk (C <= 64), inputs Kq, Vq int8 with exponents k_exp, v_exp, beta_q = rne(beta 2^15) (u16),
decay_q = rne(-g log2(e) 2^8) (non-decreasing inside a chunk):

  I1  G = Kq Kq^T
  I2  d = decay_q_i - decay_q_j; Gam = LUT[d & 255] >> (d >> 8) if (d >> 8) < 16 else 0; c = (beta_q_i Gam + 2^14) >> 15
  I3  (Aq, eA)   = Q8(-(G o c) on i > j, 2 k_exp - 15)                      [Abar, Sec. 2.1]
  I4  P_1 = band_N(Aq); (P_n, e_n) = Q8(band_N(P_{n-1} band_N(Aq)), e_{n-1} + eA), n = 2..N   [Eq. 7, 10]
  I5  (T0q, eT0) = Q8(align(P_1..P_N))  on 1 <= i-j <= N                    [T0 - I, Eq. 11]
  I6  (Eq, eE)   = Q8(align(Aq, Aq T0q)) on i-j > N                         [Eq. 13]
  I7  R_1 = Eq; (R_s, e_s) = Q8(R_{s-1} Eq, e_{s-1} + eE) on i-j >= s(N+1), s = 2..S while s(N+1) < C;
      (Sq, eS) = Q8(align(R_1..))                                           [sum_{s>=1} E^s]
  I8  (Toffq, eT) = Q8(align(T0q, Sq, T0q Sq)) on i > j                     [T - I = T0 sum E^s - I]
  I9  (Tbq, eTb) = Q8(Toffq_ij beta_q_j, eT - 15) on i > j
  I10 (Wq, eW)   = Q8(align(Tbq Kq [eTb + k_exp], beta_q_i Kq_i [k_exp - 15])); same for U with Vq, v_exp

Chunks of 128 tokens (two 64-blocks; block formula of App. E, Eq. 28, with this path's sign: T21 = -T22 A21 T11,
which for the stored blocks Aq = Abar = -A (step I3) reads T21 = T22 Abar21 T11).
The paper gives the block formula and says that 128-chunks are handled as 64 x 64 blocks; how the blocks are
quantised is this build's reading: the three blocks of A (A11, A21, A22) are quantised separately (three exponents,
all from 2 k_exp - 15), I4-I8 run on the two diagonal blocks, and

  (X, eX)     = Q8(align(A21q, A21q Toff11q))  on the full 64 x 64 block         [Abar21 T11, T11 = I + Toff11]
  (T21q, e21) = Q8(align(X, Toff22q X))                                           [(I + Toff22) X]
  I9 per block (T11b, T22b on i > j; T21b = Q8(T21q_ij beta_q_j, e21 - 15) on the full block)
  I10 rows 0..63:  Q8(align(T11b Kq_top, beta_q_i Kq_i));
      rows 64..127: Q8(align(T21b Kq_top [e21b + k_exp], T22b Kq_bot [e22b + k_exp], beta_q_i Kq_i [k_exp - 15]))

Outputs: Toffq [128][128] with exponents (e11, e21, e22), the upper-right block zero; W, U with one exponent per
64 rows. `chunk_prepare_int8_c128_ref` / `chunk_prepare_int8_c128` evaluate it.

Two evaluators are given: `chunk_prepare_int8_ref` (plain Python integers, loops) and
`chunk_prepare_int8` (numpy int64, with assertions that MMA accumulators fit int32). They are
written separately and compared with each other in the tests, together with closed forms.
"""
from __future__ import annotations

import math

import numpy as np

QMAX = 127
ALIGN_WINDOW = 8  # bits kept below the largest term of an aligned sum
# Width of the mantissas (8 here). `gdn_oracle_int16` evaluates the same steps with 16-bit mantissas by running
# these evaluators under `mantissa_width(16)`: QMAX = 2^15 - 1, shifts from bitlen - 15, a 16-bit alignment window,
# matrix products checked against 62 bits instead of 31.
MANT_BITS = 8
ACC_BITS = 31


class mantissa_width:
    """Context manager that switches both evaluators of this module to `bits`-bit mantissas (8 or 16)."""

    def __init__(self, bits: int):
        assert bits in (8, 16)
        self.new = (bits, (1 << (bits - 1)) - 1, bits, 31 if bits == 8 else 62)

    def __enter__(self):
        global MANT_BITS, QMAX, ALIGN_WINDOW, ACC_BITS
        self.old = (MANT_BITS, QMAX, ALIGN_WINDOW, ACC_BITS)
        MANT_BITS, QMAX, ALIGN_WINDOW, ACC_BITS = self.new
        return self

    def __exit__(self, *exc):
        global MANT_BITS, QMAX, ALIGN_WINDOW, ACC_BITS
        MANT_BITS, QMAX, ALIGN_WINDOW, ACC_BITS = self.old
        return False


def decay_lut() -> list[int]:
    """LUT[f] = rne(2^15 * 2^(-f/256)), f = 0..255 (unsigned 16 bit; LUT[0] = 32768)."""
    return [int(math.floor(32768.0 * 2.0 ** (-f / 256.0) + 0.5)) for f in range(256)]


def lut_checksum(lut=None) -> int:
    lut = decay_lut() if lut is None else lut
    s = 0
    for f, v in enumerate(lut):
        s = (s * 31 + int(v) + f) % 1000000007
    return s


# --------------------------------------------------------------------------- plain Python evaluator
def _rsr(x: int, r: int) -> int:
    if r <= 0:
        return x << (-r)
    a = (abs(x) + (1 << (r - 1))) >> r
    return a if x >= 0 else -a


def _q8(acc, e, support):
    """acc: dict {(i, j): int} or nested lists; support: iterable of index pairs. Returns (dict, e_out)."""
    m = 0
    for idx in support:
        m = max(m, abs(acc[idx]))
    r = max(0, m.bit_length() - (MANT_BITS - 1))
    out = {}
    for idx in support:
        q = _rsr(acc[idx], r)
        out[idx] = max(-QMAX, min(QMAX, q))
    return out, e + r


def _align(terms, support):
    """terms: list of (dict, exponent). Returns (dict over support, e_ref)."""
    es = [e for _, e in terms]
    e_ref = max(min(es), max(es) - ALIGN_WINDOW)
    out = {}
    for idx in support:
        s = 0
        for x, e in terms:
            s += _rsr(x.get(idx, 0), -(e - e_ref))
        out[idx] = s
    return out, e_ref


def _matmul_sparse(X, Y, n, support):
    out = {}
    for (i, j) in support:
        s = 0
        for k in range(n):
            a = X.get((i, k), 0)
            if a:
                b = Y.get((k, j), 0)
                if b:
                    s += a * b
        out[(i, j)] = s
    return out


def chunk_prepare_int8_ref(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N, S):
    """One chunk, plain Python integers. Kq [C][dk], Vq [C][dv] lists of ints. Returns a dict of results."""
    C = len(Kq)
    dk = len(Kq[0])
    dv = len(Vq[0])
    lut = decay_lut()
    lower = [(i, j) for i in range(C) for j in range(i)]
    # I1-I3
    accA = {}
    for (i, j) in lower:
        G = sum(int(Kq[i][d]) * int(Kq[j][d]) for d in range(dk))
        dlt = int(decay_q[i]) - int(decay_q[j])
        assert dlt >= 0
        sh = dlt >> 8
        gam = (lut[dlt & 255] >> sh) if sh < 16 else 0
        c = (int(beta_q[i]) * gam + (1 << 14)) >> 15
        accA[(i, j)] = -G * c
    Aq, eA = _q8(accA, 2 * int(k_exp) - 15, lower)
    blk = _inverse_block_ref(Aq, eA, C, N, S)
    Toffq, eT, Eq, eE, T0q, eT0 = blk["Toffq"], blk["t_exp"], blk["Eq"], blk["e_exp"], blk["T0q"], blk["t0_exp"]
    # I9
    accTb = {(i, j): Toffq[(i, j)] * int(beta_q[j]) for (i, j) in lower}
    Tbq, eTb = _q8(accTb, eT - 15, lower)

    # I10
    def out_rows(Xq, x_exp, d):
        full = [(i, c) for i in range(C) for c in range(d)]
        prod = {}
        diag = {}
        for (i, c) in full:
            s = 0
            for j in range(i):
                t = Tbq[(i, j)]
                if t:
                    s += t * int(Xq[j][c])
            prod[(i, c)] = s
            diag[(i, c)] = int(beta_q[i]) * int(Xq[i][c])
        acc, eref = _align([(prod, eTb + int(x_exp)), (diag, int(x_exp) - 15)], full)
        q, e = _q8(acc, eref, full)
        return [[q[(i, c)] for c in range(d)] for i in range(C)], e

    Wq, eW = out_rows(Kq, k_exp, dk)
    Uq, eU = out_rows(Vq, v_exp, dv)
    Toff = [[Toffq.get((i, j), 0) for j in range(C)] for i in range(C)]
    return {"Wq": Wq, "w_exp": eW, "Uq": Uq, "u_exp": eU, "Toffq": Toff, "t_exp": eT,
            "Aq": [[Aq.get((i, j), 0) for j in range(C)] for i in range(C)], "a_exp": eA,
            "Eq": [[Eq.get((i, j), 0) for j in range(C)] for i in range(C)], "e_exp": eE,
            "T0q": [[T0q.get((i, j), 0) for j in range(C)] for i in range(C)], "t0_exp": eT0}


def _inverse_block_ref(Aq, eA, C, N, S):
    """Steps I4-I8 on one C x C block: (Aq, eA) on the strictly lower triangle -> Toffq, eT (T = I + Toffq 2^eT)."""
    lower = [(i, j) for i in range(C) for j in range(i)]
    band = [(i, j) for (i, j) in lower if i - j <= N]
    far = [(i, j) for (i, j) in lower if i - j > N]
    # I4
    Aband = {idx: Aq[idx] for idx in band}
    P = [(Aband, eA)]
    for n in range(2, N + 1):
        prev, eprev = P[-1]
        sup_n = [(i, j) for (i, j) in band if i - j >= n]
        acc = _matmul_sparse(prev, Aband, C, sup_n)
        Pn, en = _q8(acc, eprev + eA, sup_n)
        P.append((Pn, en))
    # I5
    accT0, eref = _align(P, band)
    T0q, eT0 = _q8(accT0, eref, band)
    # I6
    AT0 = _matmul_sparse(Aq, T0q, C, far)
    accE, eref = _align([(Aq, eA), (AT0, eA + eT0)], far)
    Eq, eE = _q8(accE, eref, far)
    # I7
    R = []
    if S >= 1:
        R.append((Eq, eE))
        for s in range(2, S + 1):
            if s * (N + 1) >= C:
                break
            sup_s = [(i, j) for (i, j) in lower if i - j >= s * (N + 1)]
            prev, eprev = R[-1]
            acc = _matmul_sparse(prev, Eq, C, sup_s)
            Rs, es = _q8(acc, eprev + eE, sup_s)
            R.append((Rs, es))
    if R:
        accS, eref = _align(R, far)
        Sq, eS = _q8(accS, eref, far)
    else:
        Sq, eS = {idx: 0 for idx in far}, 0
    # I8
    T0S = _matmul_sparse(T0q, Sq, C, lower)
    accT, eref = _align([(T0q, eT0), (Sq, eS), (T0S, eT0 + eS)], lower)
    Toffq, eT = _q8(accT, eref, lower)
    return {"Toffq": Toffq, "t_exp": eT, "Eq": Eq, "e_exp": eE, "T0q": T0q, "t0_exp": eT0}


def chunk_prepare_int8_c128_ref(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N, S):
    """One chunk of 128 tokens as two 64-blocks (App. E, Eq. 28 with the sign of this path), plain Python integers.

    See the module docstring ("Chunks of 128 tokens"). Returns Wq, Uq [128][d], w_exp, u_exp (top, bottom),
    Toffq [128][128] (upper-right block zero) and t_exp = (e11, e21, e22).
    """
    c = 64
    assert len(Kq) == 2 * c
    dk, dv = len(Kq[0]), len(Vq[0])
    lut = decay_lut()
    lower = [(i, j) for i in range(c) for j in range(i)]
    full = [(i, j) for i in range(c) for j in range(c)]

    def a_block(r0, c0, support):
        acc = {}
        for (i, j) in support:
            gi, gj = r0 + i, c0 + j
            G = sum(int(Kq[gi][d]) * int(Kq[gj][d]) for d in range(dk))
            dlt = int(decay_q[gi]) - int(decay_q[gj])
            assert dlt >= 0
            sh = dlt >> 8
            gam = (lut[dlt & 255] >> sh) if sh < 16 else 0
            acc[(i, j)] = -G * ((int(beta_q[gi]) * gam + (1 << 14)) >> 15)
        return _q8(acc, 2 * int(k_exp) - 15, support)

    A11, eA11 = a_block(0, 0, lower)
    A21, eA21 = a_block(c, 0, full)
    A22, eA22 = a_block(c, c, lower)
    b1 = _inverse_block_ref(A11, eA11, c, N, S)
    b2 = _inverse_block_ref(A22, eA22, c, N, S)
    T11, e11 = b1["Toffq"], b1["t_exp"]
    T22, e22 = b2["Toffq"], b2["t_exp"]
    # the blocks hold Abar = -A (step I3), so T21 = -T22 A21 T11 = T22 Abar21 T11:
    # X = Abar21 T11 = Abar21 + Abar21 Toff11;  T21 = T22 X = X + Toff22 X
    accX, eref = _align([(A21, eA21), (_matmul_sparse(A21, T11, c, full), eA21 + e11)], full)
    X, eX = _q8(accX, eref, full)
    acc21, eref = _align([(X, eX), (_matmul_sparse(T22, X, c, full), e22 + eX)], full)
    T21, e21 = _q8(acc21, eref, full)
    # I9 per block
    T11b, e11b = _q8({(i, j): T11[(i, j)] * int(beta_q[j]) for (i, j) in lower}, e11 - 15, lower)
    T22b, e22b = _q8({(i, j): T22[(i, j)] * int(beta_q[c + j]) for (i, j) in lower}, e22 - 15, lower)
    T21b, e21b = _q8({(i, j): T21[(i, j)] * int(beta_q[j]) for (i, j) in full}, e21 - 15, full)

    # I10 per block of 64 rows
    def out_rows(Xq, x_exp, d):
        sup = [(i, cc) for i in range(c) for cc in range(d)]
        x_exp = int(x_exp)
        top_p, top_d, bot_p1, bot_p2, bot_d = {}, {}, {}, {}, {}
        for (i, cc) in sup:
            top_p[(i, cc)] = sum(T11b.get((i, j), 0) * int(Xq[j][cc]) for j in range(i))
            top_d[(i, cc)] = int(beta_q[i]) * int(Xq[i][cc])
            bot_p1[(i, cc)] = sum(T21b[(i, j)] * int(Xq[j][cc]) for j in range(c))
            bot_p2[(i, cc)] = sum(T22b.get((i, j), 0) * int(Xq[c + j][cc]) for j in range(i))
            bot_d[(i, cc)] = int(beta_q[c + i]) * int(Xq[c + i][cc])
        acc, er = _align([(top_p, e11b + x_exp), (top_d, x_exp - 15)], sup)
        qt, et = _q8(acc, er, sup)
        acc, er = _align([(bot_p1, e21b + x_exp), (bot_p2, e22b + x_exp), (bot_d, x_exp - 15)], sup)
        qb, eb = _q8(acc, er, sup)
        rows = [[qt[(i, cc)] for cc in range(d)] for i in range(c)] + [[qb[(i, cc)] for cc in range(d)] for i in range(c)]
        return rows, (et, eb)

    Wq, eW = out_rows(Kq, k_exp, dk)
    Uq, eU = out_rows(Vq, v_exp, dv)
    Toff = [[0] * (2 * c) for _ in range(2 * c)]
    for (i, j) in lower:
        Toff[i][j] = T11[(i, j)]
        Toff[c + i][c + j] = T22[(i, j)]
    for (i, j) in full:
        Toff[c + i][j] = T21[(i, j)]
    return {"Wq": Wq, "w_exp": eW, "Uq": Uq, "u_exp": eU, "Toffq": Toff, "t_exp": (e11, e21, e22)}


# --------------------------------------------------------------------------- numpy int64 evaluator (batched)
def _bitlen(m: np.ndarray) -> np.ndarray:
    """bit length of non-negative int64 values."""
    m = m.astype(np.int64)
    out = np.zeros(m.shape, dtype=np.int64)
    v = m.copy()
    for sh in (32, 16, 8, 4, 2, 1):
        big = v >= (np.int64(1) << sh)
        out = out + np.where(big, sh, 0)
        v = np.where(big, v >> sh, v)
    return out + (v > 0)


def _rsr_np(x: np.ndarray, r: np.ndarray) -> np.ndarray:
    """Round-half-away right shift by r >= 0 (r broadcastable); r == 0 leaves x unchanged."""
    r = np.asarray(r, dtype=np.int64)
    # int64 cannot hold 2^(r-1) for r >= 64 and numpy's shifts by 64 or more are not the mathematical ones: there the
    # result is 0, since every value that reaches this function is below 2^62 in magnitude (|x| + 2^(r-1) < 2^r).
    big = r >= 63
    rc = np.where(big, 1, r)
    half = np.where(rc > 0, np.int64(1) << np.maximum(rc - 1, 0), 0)
    a = (np.abs(x) + half) >> rc
    return np.where(big, 0, np.where(x >= 0, a, -a))


def _shift_np(x: np.ndarray, s: np.ndarray) -> np.ndarray:
    """x * 2^s for s >= 0, rsr for s < 0 (s per chunk, broadcast over the last two axes)."""
    s = np.asarray(s, dtype=np.int64)[..., None, None]
    return np.where(s >= 0, x << np.maximum(s, 0), _rsr_np(x, np.maximum(-s, 0)))


def _q8_np(acc: np.ndarray, e: np.ndarray, support: np.ndarray):
    acc = np.where(support, acc, 0).astype(np.int64)
    m = np.abs(acc).max(axis=(-1, -2))
    r = np.maximum(0, _bitlen(m) - (MANT_BITS - 1))
    q = np.clip(_rsr_np(acc, r[..., None, None]), -QMAX, QMAX)
    return np.where(support, q, 0).astype(np.int64), np.asarray(e, dtype=np.int64) + r


def _align_np(terms, support):
    es = np.stack([np.asarray(e, dtype=np.int64) for _, e in terms])
    e_ref = np.maximum(es.min(axis=0), es.max(axis=0) - ALIGN_WINDOW)
    total = 0
    for x, e in terms:
        total = total + _shift_np(np.where(support, x, 0).astype(np.int64), np.asarray(e, dtype=np.int64) - e_ref)
    return total, e_ref


def _mm_i32(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    out = np.matmul(a.astype(np.int64), b.astype(np.int64))
    assert np.abs(out).max(initial=0) < 2 ** ACC_BITS, "a matrix-product accumulator would overflow"
    return out


def _inverse_block_np(Aq, eA, N: int, S: int):
    """Steps I4-I8 on a batch of C x C blocks. Returns Toffq, eT, Eq, eE, T0q, eT0 and the products R_{s-1} Eq."""
    C = Aq.shape[-1]
    i = np.arange(C)[:, None]
    j = np.arange(C)[None, :]
    d = i - j
    lower = d > 0
    band = lower & (d <= N)
    far = d > N
    # I4
    Aband = np.where(band, Aq, 0)
    P = [(Aband, eA)]
    for nn in range(2, N + 1):
        prev, eprev = P[-1]
        sup = band & (d >= nn)
        Pn, en = _q8_np(_mm_i32(prev, Aband), eprev + eA, sup)
        P.append((Pn, en))
    # I5
    accT0, eref = _align_np(P, band)
    T0q, eT0 = _q8_np(accT0, eref, band)
    # I6
    accE, eref = _align_np([(Aq, eA), (_mm_i32(Aq, T0q), eA + eT0)], far)
    Eq, eE = _q8_np(accE, eref, far)
    # I7
    R = []
    acc_R = {}  # s -> the int32 product R_{s-1} Eq before requantisation
    if S >= 1:
        R.append((Eq, eE))
        for s in range(2, S + 1):
            if s * (N + 1) >= C:
                break
            sup = d >= s * (N + 1)
            prev, eprev = R[-1]
            acc_R[s] = _mm_i32(prev, Eq)
            Rs, es = _q8_np(acc_R[s], eprev + eE, sup)
            R.append((Rs, es))
    if R:
        accS, eref = _align_np(R, far)
        Sq, eS = _q8_np(accS, eref, far)
    else:
        Sq, eS = np.zeros_like(Aq), np.zeros_like(eA)
    # I8
    accT, eref = _align_np([(T0q, eT0), (Sq, eS), (_mm_i32(T0q, Sq), eT0 + eS)], lower)
    Toffq, eT = _q8_np(accT, eref, lower)
    return Toffq, eT, Eq, eE, T0q, eT0, acc_R


def chunk_prepare_int8(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N: int, S: int):
    """Batched exact evaluation. Kq [n, C, dk], Vq [n, C, dv] (int), k_exp, v_exp [n], beta_q, decay_q [n, C].

    Returns dict with Wq, Uq (int8 arrays), w_exp, u_exp, Toffq [n, C, C] int8, t_exp and the
    intermediate tensors Aq, Eq, T0q with their exponents.
    """
    Kq = np.asarray(Kq).astype(np.int64)
    Vq = np.asarray(Vq).astype(np.int64)
    k_exp = np.asarray(k_exp).astype(np.int64)
    v_exp = np.asarray(v_exp).astype(np.int64)
    beta_q = np.asarray(beta_q).astype(np.int64)
    decay_q = np.asarray(decay_q).astype(np.int64)
    n, C, dk = Kq.shape
    lut = np.asarray(decay_lut(), dtype=np.int64)
    i = np.arange(C)[:, None]
    j = np.arange(C)[None, :]
    d = i - j
    lower = d > 0
    band = lower & (d <= N)
    far = d > N
    # I1-I3
    G = _mm_i32(Kq, np.swapaxes(Kq, -1, -2))
    dlt = np.where(lower, decay_q[:, :, None] - decay_q[:, None, :], 0)
    assert dlt.min() >= 0, "decay_q must be non-decreasing inside a chunk"
    sh = dlt >> 8
    gam = np.where(sh < 16, lut[dlt & 255] >> np.minimum(sh, 15), 0)
    c = (beta_q[:, :, None] * gam + (1 << 14)) >> 15
    Aq, eA = _q8_np(-(G * c), 2 * k_exp - 15, lower)
    Toffq, eT, Eq, eE, T0q, eT0, acc_R = _inverse_block_np(Aq, eA, N, S)
    # I9
    Tbq, eTb = _q8_np(Toffq * beta_q[:, None, :], eT - 15, lower)

    # I10
    def out_rows(Xq, x_exp):
        full = np.ones((1, 1), dtype=bool)
        prod = _mm_i32(Tbq, Xq)
        diag = beta_q[:, :, None] * Xq
        acc, er = _align_np([(prod, eTb + x_exp), (diag, x_exp - 15)], full)
        return _q8_np(acc, er, full) + (prod,)

    Wq, eW, acc_W = out_rows(Kq, k_exp)
    Uq, eU, acc_U = out_rows(Vq, v_exp)
    # the matrix products an implementation is expected to run on integer matrix units, before any rounding:
    # Gram rows, the power products R_{s-1} Eq (s = 2..8, zeros where skipped), Tbq Kq and Tbq Vq
    acc_all = np.zeros((n, C, 8 * C + dk + Vq.shape[-1]), dtype=np.int64)
    acc_all[:, :, :C] = G
    for s_, prod_ in acc_R.items():
        if s_ <= 8:
            acc_all[:, :, (s_ - 1) * C:s_ * C] = prod_
    acc_all[:, :, 8 * C:8 * C + dk] = acc_W
    acc_all[:, :, 8 * C + dk:] = acc_U
    mt = np.int8 if MANT_BITS == 8 else np.int16
    return {"acc": acc_all,
            "Wq": Wq.astype(mt), "w_exp": eW, "Uq": Uq.astype(mt), "u_exp": eU,
            "Toffq": Toffq.astype(mt), "t_exp": eT, "Aq": Aq.astype(mt), "a_exp": eA,
            "Eq": Eq.astype(mt), "e_exp": eE, "T0q": T0q.astype(mt), "t0_exp": eT0}


def chunk_prepare_int8_c128(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N: int, S: int):
    """Batched exact evaluation for chunks of 128 tokens (two 64-blocks and the block formula of App. E, Eq. 28).

    Kq [n, 128, dk], Vq [n, 128, dv], k_exp, v_exp [n], beta_q, decay_q [n, 128]. Returns Wq, Uq with w_exp, u_exp
    [n, 2] (rows 0..63, rows 64..127), Toffq [n, 128, 128] with t_exp [n, 3] = (e11, e21, e22).
    """
    Kq = np.asarray(Kq).astype(np.int64)
    Vq = np.asarray(Vq).astype(np.int64)
    k_exp = np.asarray(k_exp).astype(np.int64)
    v_exp = np.asarray(v_exp).astype(np.int64)
    beta_q = np.asarray(beta_q).astype(np.int64)
    decay_q = np.asarray(decay_q).astype(np.int64)
    n, C2, dk = Kq.shape
    c = 64
    assert C2 == 2 * c
    lut = np.asarray(decay_lut(), dtype=np.int64)
    ii = np.arange(C2)[:, None]
    jj = np.arange(C2)[None, :]
    low2 = ii > jj
    G = _mm_i32(Kq, np.swapaxes(Kq, -1, -2))
    dlt = np.where(low2, decay_q[:, :, None] - decay_q[:, None, :], 0)
    assert dlt.min() >= 0, "decay_q must be non-decreasing inside a chunk"
    sh = dlt >> 8
    gam = np.where(sh < 16, lut[dlt & 255] >> np.minimum(sh, 15), 0)
    accA = -(G * ((beta_q[:, :, None] * gam + (1 << 14)) >> 15))
    lower = low2[:c, :c]
    full = np.ones((c, c), dtype=bool)
    eA0 = 2 * k_exp - 15
    A11, eA11 = _q8_np(accA[:, :c, :c], eA0, lower)
    A21, eA21 = _q8_np(accA[:, c:, :c], eA0, full)
    A22, eA22 = _q8_np(accA[:, c:, c:], eA0, lower)
    T11, e11 = _inverse_block_np(A11, eA11, N, S)[:2]
    T22, e22 = _inverse_block_np(A22, eA22, N, S)[:2]
    accX, er = _align_np([(A21, eA21), (_mm_i32(A21, T11), eA21 + e11)], full)
    X, eX = _q8_np(accX, er, full)
    acc21, er = _align_np([(X, eX), (_mm_i32(T22, X), e22 + eX)], full)
    T21, e21 = _q8_np(acc21, er, full)  # (the blocks hold Abar = -A: T21 = T22 Abar21 T11, no sign left)
    b_top, b_bot = beta_q[:, :c], beta_q[:, c:]
    T11b, e11b = _q8_np(T11 * b_top[:, None, :], e11 - 15, lower)
    T22b, e22b = _q8_np(T22 * b_bot[:, None, :], e22 - 15, lower)
    T21b, e21b = _q8_np(T21 * b_top[:, None, :], e21 - 15, full)

    def out_rows(Xq, x_exp):
        one = np.ones((1, 1), dtype=bool)
        Xt, Xb = Xq[:, :c], Xq[:, c:]
        acc, er = _align_np([(_mm_i32(T11b, Xt), e11b + x_exp), (b_top[:, :, None] * Xt, x_exp - 15)], one)
        qt, et = _q8_np(acc, er, one)
        acc, er = _align_np([(_mm_i32(T21b, Xt), e21b + x_exp), (_mm_i32(T22b, Xb), e22b + x_exp),
                             (b_bot[:, :, None] * Xb, x_exp - 15)], one)
        qb, eb = _q8_np(acc, er, one)
        return np.concatenate([qt, qb], axis=1), np.stack([et, eb], axis=-1)

    Wq, eW = out_rows(Kq, k_exp)
    Uq, eU = out_rows(Vq, v_exp)
    Toff = np.zeros((n, C2, C2), dtype=np.int64)
    Toff[:, :c, :c] = T11
    Toff[:, c:, :c] = T21
    Toff[:, c:, c:] = T22
    mt = np.int8 if MANT_BITS == 8 else np.int16
    return {"Wq": Wq.astype(mt), "w_exp": eW, "Uq": Uq.astype(mt), "u_exp": eU,
            "Toffq": Toff.astype(mt), "t_exp": np.stack([e11, e21, e22], axis=-1)}


def dequantise_c128(q: np.ndarray, e: np.ndarray) -> np.ndarray:
    """T - I of 128-token chunks as fp64 from the three blocks and their exponents (e11, e21, e22)."""
    c = 64
    out = np.zeros(q.shape, dtype=np.float64)
    e = np.asarray(e, dtype=np.float64)
    out[..., :c, :c] = q[..., :c, :c] * np.exp2(e[..., 0])[..., None, None]
    out[..., c:, :c] = q[..., c:, :c] * np.exp2(e[..., 1])[..., None, None]
    out[..., c:, c:] = q[..., c:, c:] * np.exp2(e[..., 2])[..., None, None]
    return out


def dequantise(q: np.ndarray, e: np.ndarray) -> np.ndarray:
    """q * 2^e per chunk, fp64."""
    return q.astype(np.float64) * np.exp2(np.asarray(e, dtype=np.float64))[..., None, None]

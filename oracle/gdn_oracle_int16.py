"""CPU oracle for the INT16 variant of the chunk-prepare path (exact integer arithmetic).

TEST INFRASTRUCTURE ONLY: only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this file; it shares no code with the CUDA sources.

INT16 is the paper's primary integer precision for the inverse (Sec. 4.2, Table 1; App. G table,
row "Matrix Inversion"). The paper fixes for it what it fixes for INT8 (uniform symmetric quantiser,
App. G Eq. 32; one scale per tensor; N <= 3 with residual correction, Sec. 3.5; band mask, Sec. 3.3;
quantisation re-applied at every step of the chain, Sec. 3.5) and nothing more, so this build reads
it as the block-floating-point scheme of `gdn_oracle_int8` with 16-bit mantissas:

  * every tensor is int16 mantissas in [-32767, 32767] with one power-of-two exponent per chunk,
    taken from the tensor's own maximum on its structural support (mask before requantisation);
  * Q16(acc, e): r = max(0, bitlen(max |acc|) - 15), q = clamp(rsr(acc, r), +-32767), exponent e + r,
    rsr = rounded right shift, half away from zero;
  * aligned sums keep 16 bits below their largest term (the width of the mantissa they are
    requantised to right afterwards);
  * the identity is never quantised (T = I + Toff); beta_q = rne(beta 2^15); the gate decay comes
    from the same 256-entry table of 2^(-f/256) in 1.15 fixed point plus a shift;
  * steps I1-I10 are those of the INT8 oracle, in the same order, with Q16 in place of Q8.

Inputs: Kq, Vq int16 mantissas with one exponent per chunk (k_exp, v_exp), beta_q, decay_q as for INT8.
The two evaluators of `gdn_oracle_int8` (plain Python integers with loops; batched numpy int64) are
written for a mantissa width that they read at call time; here they run at 16 bits. Matrix
products are checked against 62 bits (an implementation that splits the mantissas into bytes and
multiplies the byte planes on an 8-bit integer matrix unit recombines int32 partial sums exactly).
"""
from __future__ import annotations

import numpy as np

from . import gdn_oracle_int8 as _w

QMAX = 32767
MANT_BITS = 16
ALIGN_WINDOW = 16


def chunk_prepare_int16_ref(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N, S):
    """One chunk, plain Python integers (loops). Same result keys as `gdn_oracle_int8.chunk_prepare_int8_ref`."""
    with _w.mantissa_width(16):
        return _w.chunk_prepare_int8_ref(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N, S)


def chunk_prepare_int16(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N: int, S: int):
    """Batched exact evaluation (numpy int64). Kq [n, C, dk], Vq [n, C, dv] int16 mantissas, k_exp, v_exp [n],
    beta_q, decay_q [n, C]. Returns Wq, Uq, Toffq (int16) with w_exp, u_exp, t_exp, the intermediate tensors
    Aq, Eq, T0q with their exponents, and "acc": the exact matrix products before any rounding (Gram rows, the
    power products R_{s-1} Eq for s = 2..8, Tbq Kq, Tbq Vq) as int64."""
    with _w.mantissa_width(16):
        return _w.chunk_prepare_int8(Kq, Vq, k_exp, v_exp, beta_q, decay_q, N, S)


def dequantise(q: np.ndarray, e: np.ndarray) -> np.ndarray:
    """q * 2^e per chunk, fp64."""
    return _w.dequantise(q, e)

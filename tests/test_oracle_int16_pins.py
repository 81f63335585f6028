"""Pins for the exact-integer INT16 oracle (the INT8 steps at 16-bit mantissas): the two separately written
evaluators agree bit for bit, the quantiser's defining properties at 16 bits, a closed form in integers, and the
dequantised result against the fp64 definition (Sec. 4.2 measures the paper's INT16 kernel by the same SNR)."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as orc
from oracle import gdn_oracle_int8 as orq8
from oracle import gdn_oracle_int16 as orq
from paper_2606_06034_b200 import inputs as gen


def _int16_chunks(C, n_heads=2, T=None, seed=0, adversarial="none", d=32):
    T = T or 2 * C
    inp = gen.make_inputs(1, n_heads, n_heads, T, C, d, d, seed=seed, dtype=torch.float32, adversarial_heads=adversarial)
    q = gen.make_int16_inputs(inp)
    return inp, q, gen.int8_chunk_slices(q, range(q.n_chunks))


def test_width_switch_is_scoped_and_q16_follows_its_definition():
    assert orq8.MANT_BITS == 8 and orq8.QMAX == 127 and orq8.ALIGN_WINDOW == 8
    with orq8.mantissa_width(16):
        assert orq8.MANT_BITS == 16 and orq8.QMAX == 32767 and orq8.ALIGN_WINDOW == 16
        # maximum 2^20 + 5 has bit length 21 -> shift 6; the scale comes from the support only
        acc = {(1, 0): (1 << 20) + 5, (2, 0): -(1 << 20) - 5, (2, 1): 33, (0, 1): 10 ** 12}
        q, e = orq8._q8(acc, -3, [(1, 0), (2, 0), (2, 1)])
        assert e == 3 and q == {(1, 0): 16384, (2, 0): -16384, (2, 1): 1}   # 33 / 64 = 0.516 -> 1; (2^20 + 5) / 64 -> 16384
        # 2^16 - 1 -> shift 1 -> 32768 -> clamped to 32767
        q, e = orq8._q8({(0, 0): 65535}, 0, [(0, 0)])
        assert q[(0, 0)] == 32767 and e == 1
        # values that fit 15 bits are not scaled
        q, e = orq8._q8({(0, 0): -32767}, 4, [(0, 0)])
        assert q[(0, 0)] == -32767 and e == 4
        qn, en = orq8._q8_np(np.array([[[65535, -3], [40000, 0]]]), np.array([0]), np.array([[True, True], [True, False]]))
        assert en[0] == 1 and qn.tolist() == [[[32767, -2], [20000, 0]]]   # -3 / 2 = -1.5 -> -2 (half away from zero)
    assert orq8.MANT_BITS == 8 and orq8.QMAX == 127 and orq8.ALIGN_WINDOW == 8 and orq8.ACC_BITS == 31


@pytest.mark.parametrize("C,N,S,adv", [(8, 2, 1, "none"), (16, 3, 2, "none"), (16, 3, 3, "all"), (32, 3, 4, "none"),
                                       (64, 3, 8, "none"), (64, 3, 8, "all"), (64, 2, 3, "none")])
def test_two_evaluators_agree_bit_for_bit(C, N, S, adv):
    d = 16 if C >= 64 else 8
    inp, q, (Kq, Vq, ke, ve, bq, dq) = _int16_chunks(C, T=2 * C if C < 64 else C, seed=C + N + S, adversarial=adv, d=d)
    assert int(np.abs(Kq).max()) > 127  # really 16-bit mantissas
    fast = orq.chunk_prepare_int16(Kq, Vq, ke, ve, bq, dq, N, S)
    for c in range(Kq.shape[0]):
        ref = orq.chunk_prepare_int16_ref(Kq[c].tolist(), Vq[c].tolist(), int(ke[c]), int(ve[c]), bq[c].tolist(), dq[c].tolist(), N, S)
        for key in ("Wq", "Uq", "Toffq", "Aq", "Eq", "T0q"):
            assert np.array_equal(np.asarray(ref[key]), fast[key][c]), key
        for key in ("w_exp", "u_exp", "t_exp", "a_exp", "e_exp", "t0_exp"):
            assert int(ref[key]) == int(fast[key][c]), key


@pytest.mark.parametrize("case", gen.INT_EDGE_CASES)
def test_two_evaluators_agree_on_saturating_and_degenerate_inputs(case):
    inp = gen.make_inputs(1, 1, 1, 64, 64, 16, 16, seed=5, dtype=torch.float32)
    q = gen.int_edge_inputs(gen.make_int16_inputs(inp), case, bits=16)
    Kq, Vq, ke, ve, bq, dq = gen.int8_chunk_slices(q, range(q.n_chunks))
    fast = orq.chunk_prepare_int16(Kq, Vq, ke, ve, bq, dq, 3, 8)
    ref = orq.chunk_prepare_int16_ref(Kq[0].tolist(), Vq[0].tolist(), int(ke[0]), int(ve[0]), bq[0].tolist(), dq[0].tolist(), 3, 8)
    for key in ("Wq", "Uq", "Toffq", "Aq", "Eq", "T0q"):
        assert np.array_equal(np.asarray(ref[key]), fast[key][0]), key
    for key in ("w_exp", "u_exp", "t_exp", "a_exp", "e_exp", "t0_exp"):
        assert int(ref[key]) == int(fast[key][0]), key


def test_structure_and_ranges():
    inp, q, (Kq, Vq, ke, ve, bq, dq) = _int16_chunks(64, seed=5, adversarial="all", d=32)
    out = orq.chunk_prepare_int16(Kq, Vq, ke, ve, bq, dq, 3, 8)
    i = np.arange(64)[:, None]; j = np.arange(64)[None, :]
    for key in ("Wq", "Uq", "Toffq", "Aq", "Eq", "T0q"):
        assert out[key].dtype == np.int16 and np.abs(out[key].astype(int)).max() <= 32767
    assert np.all(out["Toffq"][:, i <= j] == 0)
    assert np.all(out["Eq"][:, (i - j) <= 3] == 0)
    assert np.all(out["T0q"][:, ((i - j) > 3) | (i <= j)] == 0)
    # the scale of a requantised tensor is tight: its largest mantissa uses the top bit
    assert np.all(np.abs(out["Aq"].astype(int)).max(axis=(-1, -2)) >= 16384)


def test_identical_keys_closed_form_in_integers():
    """All keys equal to one unit vector, beta = 1/2, no decay: A = (1/2) L exactly and T - I = -(1/2)^(i-j), which
    16-bit mantissas hold exactly down to 2^-15 of the largest entry (C = 16: every entry)."""
    C, d = 16, 4
    Kq = np.zeros((1, C, d), dtype=np.int64); Kq[:, :, 0] = 16384    # K = e_0 (16384 * 2^-14)
    Vq = np.zeros((1, C, d), dtype=np.int64); Vq[:, :, 1] = 8192
    ke = np.array([-14]); ve = np.array([-13])
    bq = np.full((1, C), 16384); dq = np.zeros((1, C), dtype=np.int64)
    out = orq.chunk_prepare_int16(Kq, Vq, ke, ve, bq, dq, 3, 3)
    A = orq.dequantise(out["Aq"], out["a_exp"])[0]
    assert np.array_equal(A, -0.5 * np.tril(np.ones((C, C)), -1))
    T = orq.dequantise(out["Toffq"], out["t_exp"])[0]
    i = np.arange(C)[:, None]; j = np.arange(C)[None, :]
    exact = np.where(i > j, -(0.5 ** np.maximum(i - j, 1)), 0.0)
    step = 2.0 ** float(out["t_exp"][0])
    assert np.abs(T - exact).max() <= 1.5 * step
    assert np.array_equal(T[(i - j <= 8) & (i > j)], exact[(i - j <= 8) & (i > j)])
    W = orq.dequantise(out["Wq"], out["w_exp"])[0]
    expect = 0.5 * 0.5 ** np.arange(C)
    assert np.abs(W[:, 0] - expect).max() <= 2.0 ** float(out["w_exp"][0]) * 1.5 + 2 * step


@pytest.mark.parametrize("adv,lo_T,lo_W,lo_U", [("none", 69.0, 81.0, 81.0), ("all", 76.0, 63.0, 77.0)])
def test_dequantised_result_tracks_the_fp64_definition(adv, lo_T, lo_W, lo_U):
    """The integer pipeline at 16 bits, dequantised, against the fp64 inverse of the same (dequantised) inputs:
    40-48 dB above the 8-bit pipeline, as 8 more mantissa bits should give; the floors sit within 3 dB of what these
    inputs give (benign: T - I 71.3..75.4 dB, W 83.2..84.1, U 83.3..84.2; adversarial: 78.3..78.8, 65.1..67.3,
    79.4..80.0). (Context: the paper reports 67.16 dB for its INT16
    kernel on real activations, Sec. 4.2 Table 1, measured against the unquantised computation, inputs included.)"""
    for seed in (9, 10):
        inp, q, (Kq, Vq, ke, ve, bq, dq) = _int16_chunks(64, n_heads=2, T=128, seed=seed, adversarial=adv, d=64)
        out = orq.chunk_prepare_int16(Kq, Vq, ke, ve, bq, dq, 3, 8)
        K = Kq * np.exp2(ke.astype(float))[:, None, None]
        V = Vq * np.exp2(ve.astype(float))[:, None, None]
        We, Ue, Te = orc.chunk_prepare(K, V, bq / 32768.0, -dq / (256.0 * 1.4426950408889634), exact=True)
        sT = orc.snr_db(orq.dequantise(out["Toffq"], out["t_exp"]), Te - np.eye(64))
        sW = orc.snr_db(orq.dequantise(out["Wq"], out["w_exp"]), We)
        sU = orc.snr_db(orq.dequantise(out["Uq"], out["u_exp"]), Ue)
        assert sT.min() > lo_T and sW.min() > lo_W and sU.min() > lo_U, (sT, sW, sU)

"""INT8 entry point against the exact-integer CPU oracle: every output byte and exponent must match."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle_int8 as orq
from paper_2606_06034_b200 import binding as gdn
from paper_2606_06034_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _to_dev(q):
    return gen.Int8Inputs(q.Kq.cuda(), q.Vq.cuda(), q.k_exp.cuda(), q.v_exp.cuda(), q.beta_q.cuda(), q.decay_q.cuda(),
                          q.B, q.H_k, q.H_v, q.T, q.C, q.d_k, q.d_v)


def _check(inp, N=-1, S=-1, chunk_ids=None, mutate=None):
    q = gen.make_int8_inputs(inp)
    if mutate is not None:
        mutate(q)
    qd = _to_dev(q)
    Wq, Uq, w_exp, u_exp, Toff, t_exp = gdn.chunk_prepare_int8(qd, N, S)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    ids = list(range(q.n_chunks)) if chunk_ids is None else list(chunk_ids)
    Kq, Vq, ke, ve, bq, dq = gen.int8_chunk_slices(q, ids)
    Nn = gdn.gdn_default_order(q.C) if N < 0 else N
    Ss = gdn.gdn_default_residual_steps(q.C) if S < 0 else S
    ref = orq.chunk_prepare_int8(Kq, Vq, ke, ve, bq, dq, Nn, Ss)
    n, C = q.n_chunks, q.C
    idx = torch.as_tensor(ids, device="cuda")
    got = {
        "Wq": Wq.reshape(n, C, q.d_k)[idx].cpu().numpy(), "Uq": Uq.reshape(n, C, q.d_v)[idx].cpu().numpy(),
        "Toffq": Toff.reshape(n, C, C)[idx].cpu().numpy(), "w_exp": w_exp.reshape(n)[idx].cpu().numpy(),
        "u_exp": u_exp.reshape(n)[idx].cpu().numpy(), "t_exp": t_exp.reshape(n)[idx].cpu().numpy(),
    }
    for key in ("t_exp", "Toffq", "w_exp", "Wq", "u_exp", "Uq"):
        bad = np.argwhere(got[key] != ref[key])
        assert bad.size == 0, f"{key}: {len(bad)} mismatches, first at {bad[0]}: got {got[key][tuple(bad[0])]} want {ref[key][tuple(bad[0])]}"


def test_lut_matches_the_oracle_table():
    assert gdn.gdn_int8_lut_checksum() == orq.lut_checksum()


@pytest.mark.parametrize("adv", ["none", "all"])
def test_int8_defaults_bit_exact(adv):
    inp = gen.make_inputs(1, 2, 2, 512, 64, 128, 128, seed=101, adversarial_heads=adv)
    _check(inp)


@pytest.mark.parametrize("N,S", [(3, 0), (3, 1), (3, 2), (2, 4), (1, 8), (2, 8), (3, 5)])
def test_int8_other_orders_and_steps(N, S):
    inp = gen.make_inputs(1, 1, 2, 256, 64, 128, 128, seed=110 + N + S, adversarial_heads="odd")
    _check(inp, N, S)


def test_int8_gqa_ragged_and_many_tiles():
    inp = gen.make_inputs(2, 2, 6, 192, 64, 128, 128, seed=120, adversarial_heads="odd")
    _check(inp)
    # more tiles than CTAs: every CTA loops
    inp = gen.make_inputs(2, 4, 8, 4096, 64, 128, 128, seed=121)
    ids = np.random.default_rng(0).choice(inp.n_chunks, size=96, replace=False)
    _check(inp, chunk_ids=sorted(ids.tolist()))


@pytest.mark.parametrize("case", gen.INT_EDGE_CASES)
def test_int8_saturating_and_degenerate_inputs_bit_exact(case):
    """Largest mantissas with the gate open and beta at its maximum (the inverse grows by tens of octaves: shifts far
    beyond the word size in the aligned sums), empty chunks, closed gates, extreme input exponents."""
    inp = gen.make_inputs(1, 2, 2, 256, 64, 128, 128, seed=5)
    _check(inp, mutate=lambda q: gen.int_edge_inputs(q, case))
    if case == "sign_max":
        for N, S in ((1, 8), (2, 5), (3, 0)):
            _check(inp, N, S, mutate=lambda q: gen.int_edge_inputs(q, case))


def test_int8_without_the_t_output_gives_the_same_w_and_u():
    inp = gen.make_inputs(1, 2, 2, 256, 64, 128, 128, seed=140, adversarial_heads="odd")
    qd = _to_dev(gen.make_int8_inputs(inp))
    full = gdn.chunk_prepare_int8(qd)
    part = gdn.chunk_prepare_int8(qd, want_toff=False)
    assert gdn.gdn_device_status() == gdn.GDN_OK and part[4] is None
    for i in (0, 1, 2, 3, 5):
        assert torch.equal(full[i], part[i])


def test_int8_unsupported_configurations():
    inp = gen.make_inputs(1, 1, 1, 128, 32, 128, 128, seed=130)
    qd = _to_dev(gen.make_int8_inputs(inp))
    with pytest.raises(gdn.GdnError) as e:
        gdn.chunk_prepare_int8(qd)
    assert e.value.status == gdn.GDN_ERR_UNSUPPORTED
    inp = gen.make_inputs(1, 1, 1, 128, 64, 128, 128, seed=131)
    qd = _to_dev(gen.make_int8_inputs(inp))
    with pytest.raises(gdn.GdnError) as e:
        gdn.chunk_prepare_int8(qd, 4, 3)
    assert e.value.status == gdn.GDN_ERR_UNSUPPORTED


def test_int8_tensor_core_accumulators_match():
    """dbg_acc_out: every int32 accumulator of the products that run on the tensor cores (Gram rows, the power
    products, Tbq Kq, Tbq Vq) equals the oracle's exact integer product."""
    inp = gen.make_inputs(1, 1, 2, 192, 64, 128, 128, seed=140, adversarial_heads="odd")
    q = gen.make_int8_inputs(inp)
    qd = _to_dev(q)
    n, C = q.n_chunks, q.C
    dbg = torch.zeros(q.B, q.H_v, q.T // C, C, 8 * C + q.d_k + q.d_v, dtype=torch.int32, device="cuda")
    gdn.chunk_prepare_int8(qd, dbg_acc=dbg)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Kq, Vq, ke, ve, bq, dq = gen.int8_chunk_slices(q, range(n))
    ref = orq.chunk_prepare_int8(Kq, Vq, ke, ve, bq, dq, gdn.gdn_default_order(C), gdn.gdn_default_residual_steps(C))
    got = dbg.reshape(n, C, -1).cpu().numpy().astype(np.int64)
    bad = np.argwhere(got != ref["acc"])
    assert bad.size == 0, f"{len(bad)} accumulator mismatches, first at {bad[0]}"
    assert np.abs(ref["acc"]).max() < 2 ** 31

"""INT8 entry point on chunks of 128 tokens (two 64-blocks and the block formula of App. E, Eq. 28) against the
exact-integer CPU oracle: every output byte and every exponent must match."""
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
    ref = orq.chunk_prepare_int8_c128(Kq, Vq, ke, ve, bq, dq, Nn, Ss)
    n, C = q.n_chunks, q.C
    idx = torch.as_tensor(ids, device="cuda")
    got = {
        "Wq": Wq.reshape(n, C, q.d_k)[idx].cpu().numpy(), "Uq": Uq.reshape(n, C, q.d_v)[idx].cpu().numpy(),
        "Toffq": Toff.reshape(n, C, C)[idx].cpu().numpy(), "w_exp": w_exp.reshape(n, 2)[idx].cpu().numpy(),
        "u_exp": u_exp.reshape(n, 2)[idx].cpu().numpy(), "t_exp": t_exp.reshape(n, 3)[idx].cpu().numpy(),
    }
    for key in ("t_exp", "Toffq", "w_exp", "Wq", "u_exp", "Uq"):
        bad = np.argwhere(got[key] != ref[key])
        assert bad.size == 0, f"{key}: {len(bad)} mismatches, first at {bad[0]}: got {got[key][tuple(bad[0])]} want {ref[key][tuple(bad[0])]}"
    return got


@pytest.mark.parametrize("case", gen.INT_EDGE_CASES)
def test_int8_c128_saturating_and_degenerate_inputs_bit_exact(case):
    inp = gen.make_inputs(1, 2, 2, 512, 128, 128, 128, seed=5)
    _check(inp, mutate=lambda q: gen.int_edge_inputs(q, case))


@pytest.mark.parametrize("adv", ["none", "all"])
def test_int8_c128_defaults_bit_exact(adv):
    inp = gen.make_inputs(1, 2, 2, 512, 128, 128, 128, seed=201, adversarial_heads=adv)
    _check(inp)


@pytest.mark.parametrize("N,S", [(3, 0), (2, 4), (1, 8), (3, 5)])
def test_int8_c128_other_orders_and_steps(N, S):
    inp = gen.make_inputs(1, 1, 2, 256, 128, 128, 128, seed=210 + N + S, adversarial_heads="odd")
    _check(inp, N, S)


def test_int8_c128_gqa_and_many_tiles():
    inp = gen.make_inputs(2, 2, 6, 384, 128, 128, 128, seed=220, adversarial_heads="odd")
    _check(inp)
    # more tiles than CTAs: every CTA of both kernels loops
    inp = gen.make_inputs(2, 4, 8, 8192, 128, 128, 128, seed=221)
    ids = np.random.default_rng(0).choice(inp.n_chunks, size=64, replace=False)
    _check(inp, chunk_ids=sorted(ids.tolist()))


def test_int8_c128_closed_gate_gives_a_zero_block():
    """A gate that closes at token 64 of every chunk makes the lower-left block vanish (degenerate case of the merge)."""
    def close(q):
        d = q.decay_q.view(q.B, q.H_v, q.T // 128, 128)
        d[..., 64:] += 16 * 256
    inp = gen.make_inputs(1, 2, 2, 256, 128, 128, 128, seed=230)
    got = _check(inp, mutate=close)
    assert not got["Toffq"][:, 64:, :64].any()


def test_int8_c128_unsupported_configurations():
    inp = gen.make_inputs(1, 1, 1, 256, 128, 128, 128, seed=240)
    qd = _to_dev(gen.make_int8_inputs(inp))
    n_c = qd.T // 128
    Wq = torch.empty(1, 1, qd.T, 128, dtype=torch.int8, device="cuda")
    Uq = torch.empty_like(Wq)
    w_exp = torch.empty(1, 1, n_c, 2, dtype=torch.int32, device="cuda")
    u_exp = torch.empty_like(w_exp)
    t_exp = torch.empty(1, 1, n_c, 3, dtype=torch.int32, device="cuda")
    # the merge reads the diagonal blocks back: Toff_q_out is required
    with pytest.raises(gdn.GdnError) as e:
        gdn.chunk_prepare_int8(qd, outputs=(Wq, Uq, w_exp, u_exp, None, t_exp))
    assert e.value.status == gdn.GDN_ERR_UNSUPPORTED
    # no accumulator dump at C = 128
    Toff = torch.empty(1, 1, n_c, 128, 128, dtype=torch.int8, device="cuda")
    dbg = torch.zeros(1, 1, n_c, 128, 8 * 128 + 256, dtype=torch.int32, device="cuda")
    with pytest.raises(gdn.GdnError) as e:
        gdn.chunk_prepare_int8(qd, outputs=(Wq, Uq, w_exp, u_exp, Toff, t_exp), dbg_acc=dbg)
    assert e.value.status == gdn.GDN_ERR_UNSUPPORTED


def test_int8_c128_needs_the_t_output():
    """The second launch reads the diagonal blocks of T back from Toff_q_out: the C ABI refuses a null pointer there
    (the binding always allocates it for chunks of 128 tokens)."""
    inp = gen.make_inputs(1, 1, 1, 256, 128, 128, 128, seed=260)
    qd = _to_dev(gen.make_int8_inputs(inp))
    out = gdn.chunk_prepare_int8(qd, want_toff=False)
    assert out[4] is not None
    W, U = torch.empty_like(qd.Kq), torch.empty_like(qd.Vq)
    we = torch.empty(1, 1, 2, 2, dtype=torch.int32, device="cuda")
    ue, te = torch.empty_like(we), torch.empty(1, 1, 2, 3, dtype=torch.int32, device="cuda")
    rc = gdn.gdn_chunk_prepare_int8(qd.Kq, qd.Vq, qd.k_exp, qd.v_exp, qd.beta_q, qd.decay_q, 1, 1, 1, 256, 128, 128, 128, -1, -1,
                                    W, U, we, ue, None, te, None, check=False)
    assert rc == gdn.GDN_ERR_UNSUPPORTED

"""Packed variable-length sequences (gdn_chunk_prepare_varlen) against the fp64 oracle and against the dense call.

Sequences of ragged lengths are laid end to end; every sequence is chunked from its own first token and its last chunk
may be short. The oracle treats a short chunk as a padded one (beta = 0 for the missing tokens)."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as orc
from paper_2606_06034_b200 import binding as gdn

pytestmark = pytest.mark.gpu

TOL = 2e-3


def _packed_inputs(lens, H_k, H_v, C, seed):
    """The configurations' recipe on a packed token axis: normalised keys, beta = sigmoid(N(0,1)), raw log-gates
    -softplus(N(0,1)); the cumulative gate restarts in every chunk of every sequence."""
    g_ = torch.Generator().manual_seed(seed)
    T = int(sum(lens))
    K = torch.randn(H_k, T, 128, generator=g_)
    K = K / K.norm(dim=-1, keepdim=True)
    V = torch.randn(H_v, T, 128, generator=g_)
    beta = torch.sigmoid(torch.randn(H_v, T, generator=g_))
    graw = -torch.nn.functional.softplus(torch.randn(H_v, T, generator=g_))
    cu = np.concatenate([[0], np.cumsum(lens)])
    start, length = gdn.chunk_table(cu, C)
    g = torch.zeros_like(graw)
    for a, L in zip(start, length):
        g[:, a:a + L] = torch.cumsum(graw[:, a:a + L], dim=-1)
    return K.to(torch.bfloat16), V.to(torch.bfloat16), beta, g, graw, cu


def _floor(ref):
    return orc.rel_frobenius(torch.from_numpy(np.ascontiguousarray(ref)).to(torch.bfloat16).double().numpy(), ref)


def _check(got, ref, what):
    err = orc.rel_frobenius(got, ref)
    fl = _floor(ref)
    bound = np.where(fl > 0.9 * TOL, np.maximum(TOL, fl + 2e-4), TOL)
    assert np.all(err <= bound), f"{what}: rel-F {err.max():.3e} (bound {bound[np.argmax(err - bound)]:.3e})"


def _compare_with_oracle(K, V, beta, g_dev, g_for_oracle, cu, C, flags, W, U, Tinv, *, g_raw=False, k_l2norm=False,
                         w_gated=False):
    H_k, H_v = K.shape[0], V.shape[0]
    group = H_v // H_k
    start, length = orc.chunk_table(cu, C)
    for hv in range(H_v):
        Wo, Uo, To, _, _ = orc.chunk_prepare_varlen(K[hv // group].double().numpy(), V[hv].double().numpy(),
                                                    beta[hv].double().numpy(), g_for_oracle[hv].double().numpy(), cu, C,
                                                    g_raw=g_raw, k_l2norm=k_l2norm, w_gated=w_gated)
        Wg, Ug = W[hv].double().cpu().numpy(), U[hv].double().cpu().numpy()
        for c, (a, L) in enumerate(zip(start, length)):
            _check(Wg[None, a:a + L], Wo[None, a:a + L], f"W head {hv} chunk {c} (len {L})")
            _check(Ug[None, a:a + L], Uo[None, a:a + L], f"U head {hv} chunk {c} (len {L})")
        if Tinv is not None:
            _check(Tinv[hv].double().cpu().numpy(), To, f"Tinv head {hv}")


LENS = {
    16: [40, 16, 5, 1, 33, 64, 7],
    32: [70, 32, 5, 1, 97, 64],
    64: [130, 64, 5, 1, 200, 63, 65],
    128: [300, 128, 5, 1, 129, 127, 256],
}


@pytest.mark.parametrize("C", [16, 32, 64, 128])
def test_varlen_matches_oracle(C):
    K, V, beta, g, graw, cu = _packed_inputs(LENS[C], 2, 4, C, seed=500 + C)
    W, U, Tinv, cs, cl = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), cu, C)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    st, ln = orc.chunk_table(cu, C)
    assert cs.cpu().tolist() == st and cl.cpu().tolist() == ln
    _compare_with_oracle(K, V, beta, g, g, cu, C, 0, W, U, Tinv)


@pytest.mark.parametrize("C", [32, 64, 128])
def test_varlen_with_prologue_flags_and_token_major_layout(C):
    K, V, beta, g, graw, cu = _packed_inputs(LENS[C], 2, 4, C, seed=520 + C)
    Kun = (K.float() * 1.9).to(torch.bfloat16)
    flags = gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM | gdn.GDN_FLAG_W_GATED
    W, U, Tinv, _, _ = gdn.chunk_prepare_varlen(Kun.cuda(), V.cuda(), beta.cuda(), graw.cuda(), cu, C, flags=flags)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    _compare_with_oracle(Kun, V, beta, graw, graw, cu, C, flags, W, U, Tinv, g_raw=True, k_l2norm=True, w_gated=True)
    # the same tensors token-major: bit-identical after transposing
    tm = flags | gdn.GDN_FLAG_LAYOUT_BTHD
    Wt, Ut, Tt, _, _ = gdn.chunk_prepare_varlen(Kun.transpose(0, 1).contiguous().cuda(), V.transpose(0, 1).contiguous().cuda(),
                                                beta.t().contiguous().cuda(), graw.t().contiguous().cuda(), cu, C, flags=tm)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(Wt.transpose(0, 1), W) and torch.equal(Ut.transpose(0, 1), U) and torch.equal(Tt, Tinv)


@pytest.mark.parametrize("C", [16, 64, 128])
def test_whole_chunks_give_the_bits_of_the_dense_call(C):
    """Lengths that are multiples of C: the packed call must reproduce the dense one bit for bit (same arithmetic, the
    rows only leave by another route)."""
    lens = [2 * C, C, 5 * C, 3 * C]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 2, 4, C, seed=540 + C)
    W, U, Tinv, _, _ = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), cu, C)
    Wd, Ud, Td = gdn.chunk_prepare(K[None].cuda(), V[None].cuda(), beta[None].cuda(), g[None].cuda(), C)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(W, Wd[0]) and torch.equal(U, Ud[0]) and torch.equal(Tinv, Td[0])


def test_short_chunks_leave_their_neighbours_alone():
    """Rows past a short chunk's length belong to the next sequence: they must come out as that sequence's own rows
    (checked above against the oracle) and rows that no chunk covers must not be written at all."""
    C = 64
    lens = [70, 3, 64]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 1, 1, C, seed=560)
    T = int(cu[-1])
    # a table that leaves out the second sequence: its rows of W, U stay as they were
    start, length = gdn.chunk_table(cu, C)
    keep = [i for i, a in enumerate(start) if not (cu[1] <= a < cu[2])]
    cs = torch.tensor([start[i] for i in keep], dtype=torch.int32, device="cuda")
    cl = torch.tensor([length[i] for i in keep], dtype=torch.int32, device="cuda")
    W = torch.full((1, T, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    U = torch.full((1, T, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    gdn.gdn_chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), cs, cl, len(keep), T, 1, 1, C, 128, 128, -1, -1,
                                 W, U, None, 0)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    a, b = int(cu[1]), int(cu[2])
    assert bool((W[:, a:b] == 7.0).all()) and bool((U[:, a:b] == 7.0).all())
    assert not bool((W[:, :a] == 7.0).all(dim=-1).any()) and not bool((W[:, b:] == 7.0).all(dim=-1).any())


def test_varlen_argument_errors():
    K = torch.zeros(1, 128, 128, dtype=torch.bfloat16, device="cuda")
    b = torch.zeros(1, 128, device="cuda")
    cs = torch.zeros(2, dtype=torch.int32, device="cuda")
    call = lambda *a: gdn.gdn_chunk_prepare_varlen(*a, check=False)
    assert call(K, K, b, b, None, cs, 2, 128, 1, 1, 64, 128, 128, -1, -1, K, K, None, 0) == gdn.GDN_ERR_NULL
    assert call(K, K, b, b, cs, cs, 2, 128, 1, 1, 48, 128, 128, -1, -1, K, K, None, 0) == gdn.GDN_ERR_UNSUPPORTED
    assert call(K, K, b, b, cs, cs, -1, 128, 1, 1, 64, 128, 128, -1, -1, K, K, None, 0) == gdn.GDN_ERR_INVALID_ARG
    assert call(K, K, b, b, cs, cs, 2, 128, 1, 1, 64, 128, 128, -1, -1, K, K, None, gdn.GDN_FLAG_OUT_FP32) == gdn.GDN_ERR_INVALID_ARG
    assert call(K, K, b, b, cs, cs, 0, 128, 1, 1, 64, 128, 128, -1, -1, K, K, None, 0) == gdn.GDN_OK
    assert gdn.gdn_device_status() == gdn.GDN_OK


def _queries(H_k, T, seed):
    gq = torch.Generator().manual_seed(seed)
    Q = torch.randn(H_k, T, 128, generator=gq)
    return (Q / Q.norm(dim=-1, keepdim=True)).to(torch.bfloat16)


@pytest.mark.parametrize("with_state,raw", [(False, False), (True, False), (True, True)])
def test_packed_layer_matches_the_token_recurrence_per_sequence(with_state, raw):
    """Both packed calls back to back (gated W, U per chunk; then state passing and output per sequence) against the
    token-by-token gated delta rule run on every sequence by itself, each with its own initial and final state."""
    C = 64
    lens = [130, 64, 5, 1, 200, 63, 65, 128]
    H_k, H_v = 2, 4
    K, V, beta, g, graw, cu = _packed_inputs(lens, H_k, H_v, C, seed=600)
    T = int(cu[-1])
    Q = _queries(H_k, T, 601)
    scale = 128 ** -0.5
    S0 = 0.1 * torch.randn(len(lens), H_v, 128, 128, generator=torch.Generator().manual_seed(602)) if with_state else None
    gates = graw if raw else g
    flags = gdn.GDN_FLAG_W_GATED | (gdn.GDN_FLAG_G_RAW if raw else 0)
    W, U, _, _, _ = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), gates.cuda(), cu, C, flags=flags, want_tinv=False)
    O, S = gdn.chunk_state_output_varlen(Q.cuda(), K.cuda(), W, U, gates.cuda(), cu, C, scale,
                                         None if S0 is None else S0.cuda(), flags=gdn.GDN_FLAG_G_RAW if raw else 0)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert bool(torch.isfinite(O).all()) and bool(torch.isfinite(S).all())
    for s_, L in enumerate(lens):
        a = int(cu[s_])
        for hv in range(H_v):
            hk = hv // (H_v // H_k)
            Oo, So = orc.gated_delta_rule(Q[hk, a:a + L].double().numpy(), K[hk, a:a + L].double().numpy(),
                                          V[hv, a:a + L].double().numpy(), beta[hv, a:a + L].double().numpy(),
                                          graw[hv, a:a + L].double().numpy(), scale,
                                          None if S0 is None else S0[s_, hv].double().numpy())
            eO = orc.rel_frobenius(O[hv, a:a + L].double().cpu().numpy()[None], Oo[None])
            assert eO.max() <= 1e-2, f"sequence {s_} (len {L}) head {hv}: O rel-F {eO.max():.3e}"
            eS = orc.rel_frobenius(S[s_, hv].double().cpu().numpy()[None], So[None])
            assert eS.max() <= 1e-2, f"sequence {s_} (len {L}) head {hv}: S rel-F {eS.max():.3e}"


def test_packed_state_output_matches_oracle_on_the_same_w_u():
    """The state / output step alone: the oracle gets the bf16 W, U the first call produced (padded per sequence)."""
    C = 64
    lens = [100, 64, 7, 191]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 1, 2, C, seed=610)
    T = int(cu[-1])
    Q = _queries(1, T, 611)
    scale = 128 ** -0.5
    W, U, _, _, _ = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), cu, C, flags=gdn.GDN_FLAG_W_GATED,
                                             want_tinv=False)
    O, S = gdn.chunk_state_output_varlen(Q.cuda(), K.cuda(), W, U, g.cuda(), cu, C, scale)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    for s_, L in enumerate(lens):
        a = int(cu[s_])
        Lp = -(-L // C) * C
        for hv in range(2):
            def pad(x):
                out = np.zeros((Lp,) + tuple(x.shape[1:]))
                out[:L] = x[a:a + L].double().cpu().numpy()
                return out
            gp = pad(g[hv])
            gp[L:] = gp[L - 1]
            Oo, So = orc.chunk_state_output(pad(Q[0]), pad(K[0]), pad(W[hv]), pad(U[hv]), gp, C, scale)
            eO = orc.rel_frobenius(O[hv, a:a + L].double().cpu().numpy()[None], Oo[None, :L])
            assert eO.max() <= 2.2e-3, f"sequence {s_} head {hv}: O rel-F {eO.max():.3e}"
            eS = orc.rel_frobenius(S[s_, hv].double().cpu().numpy()[None], So[None])
            assert eS.max() <= 1e-4, f"sequence {s_} head {hv}: S rel-F {eS.max():.3e}"
    # rows of O past the last sequence stay untouched (none here), and nothing wrote outside [0, T)
    assert O.shape == (2, T, 128)


def test_packed_layer_token_major_gives_the_same_bits():
    """Both packed calls on token-major tensors [T,H,d] reproduce the head-major results bit for bit."""
    C = 64
    lens = [100, 64, 7, 191, 1]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 2, 4, C, seed=620)
    T = int(cu[-1])
    Q = _queries(2, T, 621)
    scale = 128 ** -0.5
    f = gdn.GDN_FLAG_W_GATED | gdn.GDN_FLAG_G_RAW
    W, U, _, _, _ = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), graw.cuda(), cu, C, flags=f, want_tinv=False)
    O, S = gdn.chunk_state_output_varlen(Q.cuda(), K.cuda(), W, U, graw.cuda(), cu, C, scale, flags=gdn.GDN_FLAG_G_RAW)
    tm = lambda x: x.transpose(0, 1).contiguous().cuda()
    b = gdn.GDN_FLAG_LAYOUT_BTHD
    Wt, Ut, _, _, _ = gdn.chunk_prepare_varlen(tm(K), tm(V), tm(beta), tm(graw), cu, C, flags=f | b, want_tinv=False)
    Ot, St = gdn.chunk_state_output_varlen(tm(Q), tm(K), Wt, Ut, tm(graw), cu, C, scale, flags=gdn.GDN_FLAG_G_RAW | b)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(Wt.transpose(0, 1), W) and torch.equal(Ut.transpose(0, 1), U)
    assert torch.equal(Ot.transpose(0, 1), O) and torch.equal(St, S)


def test_empty_sequences_and_empty_batches():
    """Degenerate inputs: a sequence of length zero among others (its state passes through unchanged, it has no chunk),
    no sequences at all, and a dense call with no tokens."""
    C = 64
    lens = [70, 0, 5]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 1, 2, C, seed=630)
    T = int(cu[-1])
    Q = _queries(1, T, 631)
    scale = 128 ** -0.5
    S0 = (0.1 * torch.randn(3, 2, 128, 128, generator=torch.Generator().manual_seed(632))).cuda()
    W, U, Tinv, cs, cl = gdn.chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), cu, C, flags=gdn.GDN_FLAG_W_GATED)
    assert cs.cpu().tolist() == [0, 64, 70] and cl.cpu().tolist() == [64, 6, 5]
    O, S = gdn.chunk_state_output_varlen(Q.cuda(), K.cuda(), W, U, g.cuda(), cu, C, scale, S0)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(S[1], S0[1])  # the empty sequence
    for s_, L in ((0, 70), (2, 5)):
        a = int(cu[s_])
        for hv in range(2):
            Oo, So = orc.gated_delta_rule(Q[0, a:a + L].double().numpy(), K[0, a:a + L].double().numpy(),
                                          V[hv, a:a + L].double().numpy(), beta[hv, a:a + L].double().numpy(),
                                          graw[hv, a:a + L].double().numpy(), scale, S0[s_, hv].double().cpu().numpy())
            eO = orc.rel_frobenius(O[hv, a:a + L].double().cpu().numpy()[None], Oo[None])
            eS = orc.rel_frobenius(S[s_, hv].double().cpu().numpy()[None], So[None])
            assert eO.max() <= 1e-2 and eS.max() <= 1e-2
    # no sequences, no chunks: nothing is launched, nothing is written
    before = gdn.gdn_launch_count()
    e32 = torch.zeros(1, dtype=torch.int32, device="cuda")
    Wz = torch.full((2, T, 128), 3.0, dtype=torch.bfloat16, device="cuda")
    assert gdn.gdn_chunk_prepare_varlen(K.cuda(), V.cuda(), beta.cuda(), g.cuda(), e32, e32, 0, T, 1, 2, C, 128, 128, -1, -1,
                                        Wz, Wz.clone(), None, 0) == gdn.GDN_OK
    assert gdn.gdn_chunk_state_output_varlen(Q.cuda(), K.cuda(), W, U, g.cuda(), e32, 0, T, 1, 2, C, 128, 128, scale, None,
                                             Wz, None) == gdn.GDN_OK
    assert gdn.gdn_launch_count() == before and bool((Wz == 3.0).all())
    assert gdn.gdn_device_status() == gdn.GDN_OK


def test_layer_wrapper_on_packed_token_major_raw_projections():
    """`gated_delta_layer`: packed sequences, token-major tensors, raw gates, raw key / query projections, one call."""
    C = 64
    lens = [150, 64, 9, 200]
    K, V, beta, g, graw, cu = _packed_inputs(lens, 2, 4, C, seed=640)
    T = int(cu[-1])
    gq = torch.Generator().manual_seed(641)
    Qun = (1.7 * torch.randn(2, T, 128, generator=gq)).to(torch.bfloat16)
    Kun = (K.float() * (0.5 + torch.rand(2, T, 1, generator=gq))).to(torch.bfloat16)
    tm = lambda x: x.transpose(0, 1).contiguous().cuda()
    O, S = gdn.gated_delta_layer(tm(Qun), tm(Kun), tm(V), tm(beta), tm(graw), C, cu_seqlens=cu)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    O = O.transpose(0, 1)
    Kn = Kun.double() / Kun.double().norm(dim=-1, keepdim=True)
    Qn = Qun.double() / Qun.double().norm(dim=-1, keepdim=True)
    for s_, L in enumerate(lens):
        a = int(cu[s_])
        for hv in range(4):
            Oo, So = orc.gated_delta_rule(Qn[hv // 2, a:a + L].numpy(), Kn[hv // 2, a:a + L].numpy(), V[hv, a:a + L].double().numpy(),
                                          beta[hv, a:a + L].double().numpy(), graw[hv, a:a + L].double().numpy(), 128 ** -0.5)
            eO = orc.rel_frobenius(O[hv, a:a + L].double().cpu().numpy()[None], Oo[None])
            eS = orc.rel_frobenius(S[s_, hv].double().cpu().numpy()[None], So[None])
            assert eO.max() <= 1e-2 and eS.max() <= 1e-2, f"sequence {s_} head {hv}: O {eO.max():.3e} S {eS.max():.3e}"

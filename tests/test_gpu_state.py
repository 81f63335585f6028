"""State passing + output of the chunk-wise layer (gdn_chunk_state_output) against the fp64 oracle.

The CUDA call consumes the bf16 W (gated) and U that the chunk-prepare kernel produced; the oracle is given exactly the
same values (upcast), so what is compared is this step alone. A second test runs the two CUDA calls back to back
against the token-by-token gated delta rule on the original inputs (the whole layer)."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as orc
from paper_2606_06034_b200 import binding as gdn
from paper_2606_06034_b200 import inputs as gen

pytestmark = pytest.mark.gpu

# Relative Frobenius error per chunk of O and of the final state. Every operand that can cancel (state, U_new, P) goes
# through the tensor cores as hi + lo bf16 halves with fp32 accumulation, so what remains is the bf16 rounding of the
# output itself (1.7e-3, the same floor as W and U of the chunk-prepare path) and ~1e-6 on the fp32 state.
TOL_O = 2.2e-3
TOL_S = 1e-4


def _queries(inp, seed):
    gq = torch.Generator().manual_seed(seed)
    Q = torch.randn(inp.B, inp.H_k, inp.T, inp.d_k, generator=gq)
    Q = Q / Q.norm(dim=-1, keepdim=True)
    return Q.to(inp.K.dtype).contiguous()


def _run(inp, Q, scale, S0):
    K, V, beta, g = inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), inp.g.cuda()
    W, U, _ = gdn.chunk_prepare(K, V, beta, g, inp.C, flags=gdn.GDN_FLAG_W_GATED)
    O, S = gdn.chunk_state_output(Q.cuda(), K, W, U, g, inp.C, scale, None if S0 is None else S0.cuda())
    assert gdn.gdn_device_status() == gdn.GDN_OK
    return W, U, O, S


@pytest.mark.parametrize("B,H_k,H_v,T", [(1, 1, 1, 64), (1, 1, 1, 256), (2, 2, 4, 512), (1, 2, 2, 1024)])
@pytest.mark.parametrize("with_state", [False, True])
def test_state_output_matches_oracle(B, H_k, H_v, T, with_state):
    C = 64
    inp = gen.make_inputs(B, H_k, H_v, T, C, 128, 128, seed=400 + T + H_v)
    Q = _queries(inp, 401 + T)
    scale = 128 ** -0.5
    S0 = None
    if with_state:
        S0 = 0.1 * torch.randn(B, H_v, 128, 128, generator=torch.Generator().manual_seed(402))
    W, U, O, S = _run(inp, Q, scale, S0)
    group = H_v // H_k
    for b in range(B):
        for hv in range(H_v):
            hk = hv // group
            Oo, So = orc.chunk_state_output(Q[b, hk].double().numpy(), inp.K[b, hk].double().numpy(),
                                            W[b, hv].double().cpu().numpy(), U[b, hv].double().cpu().numpy(),
                                            inp.g[b, hv].double().numpy(), C, scale,
                                            None if S0 is None else S0[b, hv].double().numpy())
            Og = O[b, hv].double().cpu().numpy().reshape(T // C, C, 128)
            eO = orc.rel_frobenius(Og, Oo.reshape(T // C, C, 128))
            assert eO.max() <= TOL_O, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head ({b},{hv})"
            eS = orc.rel_frobenius(S[b, hv].double().cpu().numpy()[None], So[None])
            assert eS.max() <= TOL_S, f"S rel-F {eS.max():.3e} of head ({b},{hv})"


@pytest.mark.parametrize("case", ["closed_gate", "open_gate", "zero_u", "large_state"])
def test_state_output_on_degenerate_inputs(case):
    """A gate that closes by 30 nats per token (every token forgets the state: the decay factors above the diagonal
    of a chunk would overflow if they were formed), no decay at all, U = 0 (the state only decays and is corrected by
    W S0), and an initial state a hundred times the usual size."""
    C, B, H_k, H_v, T = 64, 2, 1, 2, 320
    inp = gen.make_inputs(B, H_k, H_v, T, C, 128, 128, seed=430, adversarial_heads="odd")
    if case == "closed_gate":
        inp.g = (-30.0 * (1 + torch.arange(T) % C).float()).expand_as(inp.g).contiguous()
    if case == "open_gate":
        inp.g.zero_()
    Q = _queries(inp, 431)
    scale = 128 ** -0.5
    S0 = (10.0 if case == "large_state" else 0.1) * torch.randn(B, H_v, 128, 128, generator=torch.Generator().manual_seed(432))
    K, V, beta, g = inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), inp.g.cuda()
    W, U, _ = gdn.chunk_prepare(K, V, beta, g, C, flags=gdn.GDN_FLAG_W_GATED)
    if case == "zero_u":
        U.zero_()
    O, S = gdn.chunk_state_output(Q.cuda(), K, W, U, g, C, scale, S0.cuda())
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.isfinite(O.float()).all() and torch.isfinite(S).all()
    for b in range(B):
        for hv in range(H_v):
            Oo, So = orc.chunk_state_output(Q[b, 0].double().numpy(), inp.K[b, 0].double().numpy(), W[b, hv].double().cpu().numpy(),
                                            U[b, hv].double().cpu().numpy(), inp.g[b, hv].double().numpy(), C, scale,
                                            S0[b, hv].double().numpy())
            assert np.isfinite(Oo).all()
            Og, Or = O[b, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128)
            # (with U = 0 the state only decays, by e^-50 per chunk on these gates: from the third chunk on the output
            # is below the fp32 range, where the kernel's zeros are the right answer and a relative error means nothing)
            live = np.sqrt((Or ** 2).sum(axis=(-1, -2))) > 1e-30
            assert live[:2].all() and np.abs(Og[~live]).max(initial=0.0) < 1e-30
            eO = orc.rel_frobenius(Og[live], Or[live])
            assert eO.max() <= TOL_O, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head ({b},{hv})"
            Sg = S[b, hv].double().cpu().numpy()
            if np.abs(So).max() > 1e-30:
                eS = orc.rel_frobenius(Sg[None], So[None])
                assert eS.max() <= TOL_S, f"S rel-F {eS.max():.3e} of head ({b},{hv})"
            else:
                assert np.abs(Sg).max() < 1e-30


def test_both_calls_can_be_captured_in_a_cuda_graph():
    """The entry points launch kernels only (no allocation, no synchronisation; tensor maps travel as kernel arguments),
    so a model can capture the layer in a CUDA graph and replay it on the same buffers."""
    inp = gen.make_inputs(1, 2, 4, 1024, 64, 128, 128, seed=440)
    K, V, beta, g = inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), inp.g.cuda()
    Q = _queries(inp, 441).cuda()
    outs = gdn.alloc_outputs(K, V, 64, True, False)
    O, S = torch.empty_like(V), torch.empty(1, 4, 128, 128, device="cuda")

    def step():
        W, U, _ = gdn.chunk_prepare(K, V, beta, g, 64, outputs=outs, flags=gdn.GDN_FLAG_W_GATED)
        gdn.chunk_state_output(Q, K, W, U, g, 64, 0.1, None, outputs=(O, S))

    step()
    torch.cuda.synchronize()
    want = [t.clone() for t in (*outs, O, S)]
    for t in (*outs, O, S):
        t.zero_()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    assert not outs[0].any()  # captured, not run
    graph.replay()
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip((*outs, O, S), want))
    assert gdn.gdn_device_status() == gdn.GDN_OK


def test_layer_with_zero_key_and_query_rows_under_in_kernel_normalisation():
    """Raw projections with a few all-zero key and query rows, normalised in the kernels: a zero row stays zero (the
    token writes nothing / reads nothing), nothing is NaN, and the layer equals the token-by-token rule on rows
    normalised the same way."""
    gq = torch.Generator().manual_seed(450)
    T, C = 256, 64
    Q, K = torch.randn(1, T, 1, 128, generator=gq), torch.randn(1, T, 1, 128, generator=gq)
    K[0, [0, 5, 63, 64, 200]] = 0
    Q[0, [1, 5, 130]] = 0
    V = torch.randn(1, T, 2, 128, generator=gq)
    beta = torch.sigmoid(torch.randn(1, T, 2, generator=gq))
    graw = -torch.nn.functional.softplus(torch.randn(1, T, 2, generator=gq))
    Qb, Kb, Vb = Q.to(torch.bfloat16), K.to(torch.bfloat16), V.to(torch.bfloat16)
    O, S = gdn.gated_delta_layer(Qb.cuda(), Kb.cuda(), Vb.cuda(), beta.cuda(), graw.cuda(), C)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert bool(torch.isfinite(O.float()).all()) and bool(torch.isfinite(S).all())
    assert not O[0, [1, 5, 130]].any()  # a zero query reads nothing
    q, k = orc.l2_normalise_rows(Qb[0, :, 0].double().numpy()), orc.l2_normalise_rows(Kb[0, :, 0].double().numpy())
    for hv in range(2):
        Oo, So = orc.gated_delta_rule(q, k, Vb[0, :, hv].double().numpy(), beta[0, :, hv].double().numpy(),
                                      graw[0, :, hv].double().numpy(), 128 ** -0.5)
        eO = orc.rel_frobenius(O[0, :, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        eS = orc.rel_frobenius(S[0, hv].double().cpu().numpy()[None], So[None])
        assert eO.max() <= 1e-2 and eS.max() <= 1e-2, (eO.max(), eS.max())


def test_zero_tokens_hand_the_initial_state_on():
    K = torch.zeros(2, 3, 0, 128, dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(2, 3, 0, device="cuda")
    S0 = torch.randn(2, 3, 128, 128, device="cuda")
    O, S = gdn.chunk_state_output(K, K, K, K, g, 64, 1.0, S0)
    assert O.shape == K.shape and torch.equal(S, S0)
    O, S = gdn.chunk_state_output(K, K, K, K, g, 64, 1.0, None)
    assert not S.any()
    Ke = torch.zeros(0, 3, 64, 128, dtype=torch.bfloat16, device="cuda")
    O, S = gdn.chunk_state_output(Ke, Ke, Ke, Ke, torch.zeros(0, 3, 64, device="cuda"), 64, 1.0, None)
    assert O.shape == Ke.shape and S.shape == (0, 3, 128, 128)
    assert gdn.gdn_device_status() == gdn.GDN_OK


def test_whole_layer_matches_the_token_recurrence():
    """chunk-prepare (gated W, U) + state passing/output on the GPU against the token-by-token gated delta rule."""
    C, T = 64, 512
    inp = gen.make_inputs(1, 1, 2, T, C, 128, 128, seed=410)
    Q = _queries(inp, 411)
    scale = 128 ** -0.5
    _, _, O, S = _run(inp, Q, scale, None)
    graw = inp.g.view(1, 2, T // C, C).diff(dim=-1, prepend=torch.zeros(1, 2, T // C, 1)).reshape(1, 2, T)
    for hv in range(2):
        Oo, So = orc.gated_delta_rule(Q[0, 0].double().numpy(), inp.K[0, 0].double().numpy(), inp.V[0, hv].double().numpy(),
                                      inp.beta[0, hv].double().numpy(), graw[0, hv].double().numpy(), scale)
        Og = O[0, hv].double().cpu().numpy().reshape(T // C, C, 128)
        eO = orc.rel_frobenius(Og, Oo.reshape(T // C, C, 128))
        assert eO.max() <= 1e-2, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()}"
        eS = orc.rel_frobenius(S[0, hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= 1e-2, f"S rel-F {eS.max():.3e}"


def test_whole_layer_from_raw_gates_and_unnormalised_keys():
    """Both calls with the raw per-token log-gates (prefix sums formed inside the kernels) and the key normalisation
    fused into the first call, against the token-by-token rule on the normalised keys."""
    C, T = 64, 384
    inp = gen.make_inputs(1, 1, 2, T, C, 128, 128, seed=412)
    Q = _queries(inp, 413)
    scale = 128 ** -0.5
    graw = inp.g.view(1, 2, T // C, C).diff(dim=-1, prepend=torch.zeros(1, 2, T // C, 1)).reshape(1, 2, T).contiguous()
    Kun = (inp.K.float() * 1.7).to(torch.bfloat16)  # unnormalised keys; the kernel normalises them for A, W
    flags = gdn.GDN_FLAG_W_GATED | gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM
    W, U, _ = gdn.chunk_prepare(Kun.cuda(), inp.V.cuda(), inp.beta.cuda(), graw.cuda(), C, flags=flags)
    Kn = Kun.double() / Kun.double().norm(dim=-1, keepdim=True)
    # the state kernel multiplies by the keys it is given: the normalised ones, rounded to bf16 as a model would
    Kn16 = Kn.to(torch.bfloat16)
    O, S = gdn.chunk_state_output(Q.cuda(), Kn16.cuda(), W, U, graw.cuda(), C, scale, flags=gdn.GDN_FLAG_G_RAW)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    for hv in range(2):
        Oo, So = orc.gated_delta_rule(Q[0, 0].double().numpy(), Kn[0, 0].numpy(), inp.V[0, hv].double().numpy(),
                                      inp.beta[0, hv].double().numpy(), graw[0, hv].double().numpy(), scale)
        eO = orc.rel_frobenius(O[0, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= 1e-2, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()}"
        eS = orc.rel_frobenius(S[0, hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= 1e-2, f"S rel-F {eS.max():.3e}"


def test_state_output_argument_errors():
    inp = gen.make_inputs(1, 1, 1, 128, 64, 128, 128, seed=420)
    K = inp.K.cuda()
    g = inp.g.cuda()
    O = torch.empty(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")
    args = dict(check=False)
    assert gdn.gdn_chunk_state_output(K, K, K, K, g, 1, 1, 1, 128, 32, 128, 128, 1.0, None, O, None, 0, **args) == gdn.GDN_ERR_UNSUPPORTED
    assert gdn.gdn_chunk_state_output(K, K, K, K, g, 1, 1, 1, 100, 64, 128, 128, 1.0, None, O, None, 0, **args) == gdn.GDN_ERR_INVALID_ARG
    assert gdn.gdn_chunk_state_output(None, K, K, K, g, 1, 1, 1, 128, 64, 128, 128, 1.0, None, O, None, 0, **args) == gdn.GDN_ERR_NULL
    assert gdn.gdn_chunk_state_output(K, K, K, K, g, 1, 1, 1, 128, 64, 128, 128, 1.0, None, O, None, gdn.GDN_FLAG_OUT_FP32, **args) == gdn.GDN_ERR_INVALID_ARG
    assert gdn.gdn_device_status() == gdn.GDN_OK


@pytest.mark.parametrize("name", ["sweep_c64", "prefill_gqa", "stress"])
def test_state_output_at_full_size(name):
    """The benchmark workloads in one launch each (chunk-prepare with the gated W, then state passing + output):
    sampled heads are compared with the oracle over their whole sequence (the chain of up to 1024 chunks is where
    an error in the carried state would accumulate), every output must be finite, and a second launch must agree
    bit for bit."""
    inp = gen.make_workload(name, device="cuda")
    C, T = inp.C, inp.T
    Q = torch.randn(inp.B, inp.H_k, T, inp.d_k, device="cuda", generator=torch.Generator(device="cuda").manual_seed(430))
    Q = (Q / Q.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    scale = 128 ** -0.5
    W, U, _ = gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, C, flags=gdn.GDN_FLAG_W_GATED)
    O, S = gdn.chunk_state_output(Q, inp.K, W, U, inp.g, C, scale)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert bool(torch.isfinite(O).all()) and bool(torch.isfinite(S).all())
    O2, S2 = gdn.chunk_state_output(Q, inp.K, W, U, inp.g, C, scale)
    assert torch.equal(O, O2) and torch.equal(S, S2)
    group = inp.H_v // inp.H_k
    heads = [(0, 0), (inp.B - 1, inp.H_v - 1), (0, 1 % inp.H_v)]  # head 1 is adversarial in the stress workload
    for b, hv in dict.fromkeys(heads):
        hk = hv // group
        Oo, So = orc.chunk_state_output(Q[b, hk].double().cpu().numpy(), inp.K[b, hk].double().cpu().numpy(),
                                        W[b, hv].double().cpu().numpy(), U[b, hv].double().cpu().numpy(),
                                        inp.g[b, hv].double().cpu().numpy(), C, scale)
        eO = orc.rel_frobenius(O[b, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= TOL_O, f"{name}: O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head ({b},{hv})"
        eS = orc.rel_frobenius(S[b, hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= TOL_S, f"{name}: S rel-F {eS.max():.3e} of head ({b},{hv})"


def test_token_major_layout_gives_the_same_bits():
    """GDN_FLAG_LAYOUT_BTHD: the tensors as model code keeps them, [B,T,H,d]; only addresses change."""
    C, T = 64, 384
    inp = gen.make_inputs(2, 2, 4, T, C, 128, 128, seed=450)
    Q = _queries(inp, 451).cuda()
    scale = 128 ** -0.5
    S0 = (0.1 * torch.randn(2, 4, 128, 128, generator=torch.Generator().manual_seed(452))).cuda()
    K, g = inp.K.cuda(), inp.g.cuda()
    W, U, _ = gdn.chunk_prepare(K, inp.V.cuda(), inp.beta.cuda(), g, C, flags=gdn.GDN_FLAG_W_GATED)
    O, S = gdn.chunk_state_output(Q, K, W, U, g, C, scale, S0)
    tm = lambda x: x.transpose(1, 2).contiguous()
    Ot, St = gdn.chunk_state_output(tm(Q), tm(K), tm(W), tm(U), g.transpose(1, 2).contiguous(), C, scale, S0,
                                    flags=gdn.GDN_FLAG_LAYOUT_BTHD)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(Ot.transpose(1, 2), O) and torch.equal(St, S)


@pytest.mark.parametrize("segments", [2, 3, 5])
@pytest.mark.parametrize("with_state", [False, True])
def test_segmented_call_matches_the_plain_call_and_the_oracle(segments, with_state):
    """Few long sequences: segments' state maps in parallel, a short recurrence for their initial states, then all
    segments with their output. Against the plain call (the state recurrence is re-associated: fp32 rounding only) and
    against the oracle on the same W, U."""
    C, T = 64, 1024
    inp = gen.make_inputs(1, 1, 2, T, C, 128, 128, seed=460)
    Q = _queries(inp, 461)
    scale = 128 ** -0.5
    S0 = 0.1 * torch.randn(1, 2, 128, 128, generator=torch.Generator().manual_seed(462)) if with_state else None
    K, g = inp.K.cuda(), inp.g.cuda()
    W, U, _ = gdn.chunk_prepare(K, inp.V.cuda(), inp.beta.cuda(), g, C, flags=gdn.GDN_FLAG_W_GATED)
    O_ref, S_ref = gdn.chunk_state_output(Q.cuda(), K, W, U, g, C, scale, None if S0 is None else S0.cuda())
    O, S = gdn.chunk_state_output_segmented(Q[0].cuda(), K[0], W[0], U[0], g[0], C, scale,
                                            None if S0 is None else S0[0].cuda(), segments=segments)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    for hv in range(2):
        Oo, So = orc.chunk_state_output(Q[0, 0].double().numpy(), inp.K[0, 0].double().numpy(), W[0, hv].double().cpu().numpy(),
                                        U[0, hv].double().cpu().numpy(), inp.g[0, hv].double().numpy(), C, scale,
                                        None if S0 is None else S0[0, hv].double().numpy())
        eO = orc.rel_frobenius(O[hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= TOL_O, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head {hv}"
        eS = orc.rel_frobenius(S[hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= TOL_S, f"S rel-F {eS.max():.3e} of head {hv}"
    dO = orc.rel_frobenius(O.double().cpu().numpy().reshape(2, -1, 128), O_ref[0].double().cpu().numpy().reshape(2, -1, 128))
    assert dO.max() <= 2e-3


def test_segmented_call_on_the_prefill_shapes():
    """The library's own segment count on the prefill workload (32 sequences of 512 chunks): finite, deterministic, and
    sampled heads against the oracle over the whole sequence."""
    inp = gen.make_workload("prefill_gqa", device="cuda")
    C, T = inp.C, inp.T
    Q = torch.randn(inp.H_k, T, inp.d_k, device="cuda", generator=torch.Generator(device="cuda").manual_seed(470))
    Q = (Q / Q.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    scale = 128 ** -0.5
    W, U, _ = gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, C, flags=gdn.GDN_FLAG_W_GATED)
    O, S = gdn.chunk_state_output_segmented(Q, inp.K[0], W[0], U[0], inp.g[0], C, scale)
    O2, S2 = gdn.chunk_state_output_segmented(Q, inp.K[0], W[0], U[0], inp.g[0], C, scale)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert bool(torch.isfinite(O).all()) and bool(torch.isfinite(S).all())
    assert torch.equal(O, O2) and torch.equal(S, S2)
    group = inp.H_v // inp.H_k
    for hv in (0, inp.H_v - 1):
        Oo, So = orc.chunk_state_output(Q[hv // group].double().cpu().numpy(), inp.K[0, hv // group].double().cpu().numpy(),
                                        W[0, hv].double().cpu().numpy(), U[0, hv].double().cpu().numpy(),
                                        inp.g[0, hv].double().cpu().numpy(), C, scale)
        eO = orc.rel_frobenius(O[hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= TOL_O, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head {hv}"
        eS = orc.rel_frobenius(S[hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= TOL_S, f"S rel-F {eS.max():.3e} of head {hv}"


@pytest.mark.parametrize("token_major", [False, True])
def test_model_native_layer_from_raw_projections(token_major):
    """The call sequence of a model: raw key / query projections (normalised inside both kernels), raw log-gates,
    optionally token-major tensors; against the token-by-token rule on the normalised keys and queries."""
    C, T = 64, 448
    inp = gen.make_inputs(1, 2, 4, T, C, 128, 128, seed=480)
    gq = torch.Generator().manual_seed(481)
    Qun = (1.3 * torch.randn(1, 2, T, 128, generator=gq)).to(torch.bfloat16)
    Kun = (inp.K.float() * (0.5 + torch.rand(1, 2, T, 1, generator=gq))).to(torch.bfloat16)
    scale = 128 ** -0.5
    graw = inp.g.view(1, 4, T // C, C).diff(dim=-1, prepend=torch.zeros(1, 4, T // C, 1)).reshape(1, 4, T).contiguous()
    f1 = gdn.GDN_FLAG_W_GATED | gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM
    f2 = gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM
    if token_major:
        tm = lambda x: x.transpose(1, 2).contiguous().cuda()
        b = gdn.GDN_FLAG_LAYOUT_BTHD
        W, U, _ = gdn.chunk_prepare(tm(Kun), tm(inp.V), tm(inp.beta), tm(graw), C, flags=f1 | b, want_tinv=False)
        O, S = gdn.chunk_state_output(tm(Qun), tm(Kun), W, U, tm(graw), C, scale, flags=f2 | b)
        O = O.transpose(1, 2)
    else:
        W, U, _ = gdn.chunk_prepare(Kun.cuda(), inp.V.cuda(), inp.beta.cuda(), graw.cuda(), C, flags=f1, want_tinv=False)
        O, S = gdn.chunk_state_output(Qun.cuda(), Kun.cuda(), W, U, graw.cuda(), C, scale, flags=f2)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Kn = Kun.double() / Kun.double().norm(dim=-1, keepdim=True)
    Qn = Qun.double() / Qun.double().norm(dim=-1, keepdim=True)
    for hv in range(4):
        Oo, So = orc.gated_delta_rule(Qn[0, hv // 2].numpy(), Kn[0, hv // 2].numpy(), inp.V[0, hv].double().numpy(),
                                      inp.beta[0, hv].double().numpy(), graw[0, hv].double().numpy(), scale)
        eO = orc.rel_frobenius(O[0, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= 1e-2, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head {hv}"
        eS = orc.rel_frobenius(S[0, hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= 1e-2, f"S rel-F {eS.max():.3e} of head {hv}"


def test_layer_wrapper_one_long_sequence_per_head_takes_the_segmented_path():
    """B = 1 with few heads: `gated_delta_layer` runs the segments of every sequence in parallel (raw projections,
    token-major tensors, raw gates); against the token-by-token rule."""
    C, T = 64, 1536
    inp = gen.make_inputs(1, 1, 2, T, C, 128, 128, seed=490)
    gq = torch.Generator().manual_seed(491)
    Qun = (1.3 * torch.randn(1, 1, T, 128, generator=gq)).to(torch.bfloat16)
    Kun = (inp.K.float() * (0.5 + torch.rand(1, 1, T, 1, generator=gq))).to(torch.bfloat16)
    graw = inp.g.view(1, 2, T // C, C).diff(dim=-1, prepend=torch.zeros(1, 2, T // C, 1)).reshape(1, 2, T).contiguous()
    S0 = 0.1 * torch.randn(1, 2, 128, 128, generator=torch.Generator().manual_seed(492))
    tm = lambda x: x.transpose(1, 2).contiguous().cuda()
    assert gdn.load_library().gdn_chunk_state_segments(2) > 1
    O, S = gdn.gated_delta_layer(tm(Qun), tm(Kun), tm(inp.V), tm(inp.beta), tm(graw), C, S_in=S0.cuda())
    assert gdn.gdn_device_status() == gdn.GDN_OK
    O = O.transpose(1, 2)
    Kn = Kun.double() / Kun.double().norm(dim=-1, keepdim=True)
    Qn = Qun.double() / Qun.double().norm(dim=-1, keepdim=True)
    for hv in range(2):
        Oo, So = orc.gated_delta_rule(Qn[0, 0].numpy(), Kn[0, 0].numpy(), inp.V[0, hv].double().numpy(),
                                      inp.beta[0, hv].double().numpy(), graw[0, hv].double().numpy(), 128 ** -0.5,
                                      S0[0, hv].double().numpy())
        eO = orc.rel_frobenius(O[0, hv].double().cpu().numpy().reshape(T // C, C, 128), Oo.reshape(T // C, C, 128))
        assert eO.max() <= 1e-2, f"O rel-F {eO.max():.3e} at chunk {eO.argmax()} of head {hv}"
        eS = orc.rel_frobenius(S[0, hv].double().cpu().numpy()[None], So[None])
        assert eS.max() <= 1e-2, f"S rel-F {eS.max():.3e} of head {hv}"

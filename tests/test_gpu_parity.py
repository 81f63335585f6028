"""CUDA path (through the C-ABI library) against the fp64 CPU oracle, chunk by chunk."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as orc
from paper_2606_06034_b200 import binding as gdn
from paper_2606_06034_b200 import inputs as gen

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-3   # relative Frobenius error per chunk, bf16 path
TOL_FP32 = 1e-5   # fp32-only path


def _to_dev(inp):
    return inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), inp.g.cuda()


def _oracle(inp, N=None, S=None, exact=False, chunk_ids=None):
    ids = range(inp.n_chunks) if chunk_ids is None else chunk_ids
    sl = gen.chunk_slices(inp, ids)
    K = np.stack([s[0] for s in sl]); V = np.stack([s[1] for s in sl])
    b = np.stack([s[2] for s in sl]); g = np.stack([s[3] for s in sl])
    return orc.chunk_prepare(K, V, b, g, N, S, exact=exact)


def _bf16_round(x):
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).double().numpy()


def _bound(ref, tol, bf16_out=True):
    """Per-chunk bar: `tol`, or, for bf16 outputs, the bf16 rounding floor of the fp64 result + 2e-4 where that floor
    is within 10 % of `tol` or above it (rounding the exact result already costs ~1.7e-3, up to 2.2e-3 on a few
    chunks of strongly correlated keys)."""
    if not bf16_out:
        return np.full(ref.shape[0], tol)
    floor = orc.rel_frobenius(_bf16_round(ref), ref)
    return np.where(floor > 0.9 * tol, np.maximum(tol, floor + 2e-4), tol)


def _gpu_chunks(W, U, Tinv, inp, chunk_ids=None):
    C = inp.C
    n = inp.n_chunks
    Wc = W.reshape(n, C, inp.d_k); Uc = U.reshape(n, C, inp.d_v); Tc = Tinv.reshape(n, C, C)
    if chunk_ids is not None:
        idx = torch.as_tensor(list(chunk_ids), device=W.device)
        Wc, Uc, Tc = Wc[idx], Uc[idx], Tc[idx]
    return Wc.double().cpu().numpy(), Uc.double().cpu().numpy(), Tc.double().cpu().numpy()


def _check(inp, tol, N=-1, S=-1, method="neumann", exact=False, chunk_ids=None):
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, inp.C, N, S, method=method)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp, chunk_ids)
    Wo, Uo, To = _oracle(inp, None if N < 0 else N, None if S < 0 else S, exact=exact, chunk_ids=chunk_ids)
    eT = orc.rel_frobenius(Tg, To); eW = orc.rel_frobenius(Wg, Wo); eU = orc.rel_frobenius(Ug, Uo)
    for name, err, ref in (("Tinv", eT, To), ("W", eW, Wo), ("U", eU, Uo)):
        bound = np.full_like(err, tol)
        if inp.K.dtype == torch.bfloat16:
            # Rounding the exact result to bf16 already costs ~1.7e-3 and, on strongly correlated keys
            # with C <= 32, up to 2.2e-3 on a few chunks. Where that floor is within 10% of the
            # tolerance or above it, the bar is the floor plus 2e-4.
            floor = orc.rel_frobenius(_bf16_round(ref), ref)
            bound = np.where(floor > 0.9 * tol, np.maximum(tol, floor + 2e-4), tol)
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), f"{name} rel-F {err[worst]:.3e} > {bound[worst]:.3e} at chunk {worst}"
    # structure: strictly upper triangle exactly zero, unit diagonal
    assert np.all(np.triu(Tg, 1) == 0)
    assert np.all(np.diagonal(Tg, axis1=-2, axis2=-1) == 1)
    return eT, eW, eU


# ---------------------------------------------------------------- fp32 path (plain FMA kernel)
def test_fp32_tiny_config():
    inp = gen.make_workload("tiny_fp32")
    _check(inp, TOL_FP32)


@pytest.mark.parametrize("C,N,S", [(2, 1, 1), (3, 1, 2), (4, 2, 1), (8, 3, 1), (8, 2, 2), (16, 3, 3), (32, 3, 4), (32, 4, 3),
                                   (64, 3, 2), (64, 5, 0), (128, 3, 8)])
def test_fp32_small_shapes(C, N, S):
    inp = gen.make_inputs(2, 1, 2, 2 * C, C, 64, 32, seed=10 + C, dtype=torch.float32)
    _check(inp, TOL_FP32, N, S)


def test_fp32_forward_substitution_matches_exact():
    inp = gen.make_inputs(1, 2, 2, 128, 64, 128, 128, seed=21, dtype=torch.float32)
    _check(inp, TOL_FP32, method="fwdsubst", exact=True)
    inp = gen.make_inputs(1, 1, 1, 256, 128, 64, 64, seed=22, dtype=torch.float32)
    _check(inp, TOL_FP32, method="fwdsubst", exact=True)


# ---------------------------------------------------------------- bf16 tensor-core path
@pytest.mark.parametrize("C", [16, 32, 64])
@pytest.mark.parametrize("adv", ["none", "all"])
def test_bf16_defaults(C, adv):
    # several tiles per head, more tiles than one wave needs a second pass on a small grid
    inp = gen.make_inputs(2, 2, 2, 1024, C, 128, 128, seed=30 + C, adversarial_heads=adv)
    _check(inp, TOL_BF16)


@pytest.mark.parametrize("C,d_k,d_v,N,S,adv", [(64, 64, 64, -1, -1, "none"), (64, 256, 64, -1, -1, "all"), (64, 64, 128, 3, 8, "all"),
                                              (48, 128, 128, 3, 4, "none"), (24, 72, 40, 2, 3, "none"), (64, 128, 128, 9, 2, "none"),
                                              (128, 64, 64, -1, -1, "all")])
def test_bf16_shapes_outside_the_tensor_core_kernel(C, d_k, d_v, N, S, adv):
    """bf16 tensors with feature sizes other than 128, chunk sizes other than 16 / 32 / 64 / 128 or an order above 7
    run on the plain FMA kernel (bf16 in and out, fp32 arithmetic): same bar as the tensor-core path, grouped heads."""
    inp = gen.make_inputs(1, 1, 2, 4 * C, C, d_k, d_v, seed=90 + C + d_k, adversarial_heads=adv)
    assert inp.K.dtype == torch.bfloat16
    n0 = gdn.gdn_launch_count()
    _check(inp, TOL_BF16, N, S)
    assert gdn.gdn_launch_count() == n0 + 1
    _check(inp, TOL_BF16, method="fwdsubst", exact=True)


@pytest.mark.parametrize("C,N,S", [(64, 3, 2), (64, 3, 1), (64, 3, 0), (64, 2, 5), (64, 1, 8), (64, 5, 3), (64, 7, 2),
                                   (32, 4, 3), (32, 3, 7), (16, 3, 2), (16, 2, 1)])
def test_bf16_other_orders_and_steps(C, N, S):
    inp = gen.make_inputs(1, 2, 2, 512, C, 128, 128, seed=40 + C + N + S)
    _check(inp, TOL_BF16, N, S)


@pytest.mark.parametrize("C,N,S,beta", [(64, 3, 2, 0.3), (64, 3, 1, 0.3), (64, 5, 3, 0.3), (64, 7, 2, 0.3), (64, 2, 5, 0.7),
                                        (32, 4, 3, 0.3), (16, 3, 2, 0.3), (16, 2, 1, 0.3)])
def test_bf16_orders_and_steps_where_every_term_counts(C, N, S, beta):
    """Inputs on which the result depends visibly on N and on S: strongly correlated keys, no decay, and a write
    strength low enough for the truncated series to stay bounded. The fp64 evaluations with N - 1 or S - 1 differ from
    the one asked for by far more than the bar, so a kernel that clamped the order, ran one round too few or got the
    band recursion wrong beyond distance 3 fails here. fp32 outputs, so that the bar is not hidden by bf16 output
    rounding. These inputs lie outside the workload regimes (the series has not converged, E and the far part of T
    are not small, so their single-bf16 tensor-core operands cost up to 1e-3 on Tinv and, through the cancellation in
    T diag(beta) K on correlated keys, up to 1e-2 on W): the bar per output is a fifth of the distance to the nearest
    neighbouring (N, S), at most 1e-2, and that distance must be at least 5e-3."""
    inp = gen.make_inputs(1, 2, 2, 512, C, 128, 128, seed=40 + C + N + S, adversarial_heads="all")
    inp.beta.fill_(beta)
    ref = _oracle(inp, N, S)
    dist = [np.inf, np.inf, np.inf]
    for n2, s2 in ((N - 1, S), (N, S - 1)):
        if n2 >= 1 and s2 >= 0:
            other = _oracle(inp, n2, s2)
            dist = [min(d, float(orc.rel_frobenius(o, r).min())) for d, o, r in zip(dist, other, ref)]
    assert min(dist) >= 5e-3, dist
    K, V, b, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, b, g, C, N, S, flags=gdn.GDN_FLAG_OUT_FP32)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    got = _gpu_chunks(W, U, Tinv, inp)
    for name, x, r, d in zip(("W", "U", "Tinv"), got, ref, dist):
        err = orc.rel_frobenius(x, r)
        bar = min(1e-2, d / 5)
        assert err.max() <= bar, f"{name} rel-F {err.max():.3e} > {bar:.3e} at chunk {err.argmax()} (nearest neighbour {d:.3e})"


@pytest.mark.parametrize("adv", ["none", "all"])
def test_bf16_full_residual_sum_is_the_exact_inverse(adv):
    """S = 15 at N = 3, C = 64 keeps every term (E^16 = 0): the kernel's four-level doubling form of the sum must
    match both the oracle's truncated evaluation with S = 15 and the exact inverse by forward substitution."""
    inp = gen.make_inputs(2, 2, 2, 1024, 64, 128, 128, seed=47, adversarial_heads=adv)
    _check(inp, TOL_BF16, 3, 15)
    _check(inp, TOL_BF16, 3, 15, exact=True)


@pytest.mark.parametrize("N,S", [(-1, -1), (3, 2), (2, 4), (3, 15)])
@pytest.mark.parametrize("adv", ["none", "odd"])
def test_bf16_chunk_128_block_merge(N, S, adv):
    """C = 128: two 64-blocks by the scheme plus the block formula of App. E for the lower-left block. On strongly
    correlated keys both products of the merge cancel (A21 has entries near 1, A21 T11 is small): the kernel's
    hi + lo operands must keep the result at the bf16 rounding floor there too."""
    inp = gen.make_inputs(2, 2, 4, 512, 128, 128, 128, seed=45 + N + S, adversarial_heads=adv)
    if adv == "odd" and S in (2, 4):
        # few residual terms on adversarial blocks: the truncated series has not converged and its entries are
        # orders of magnitude larger than those of the inverse. Parity is still against the same truncated scheme:
        # the result must be far closer to it than the exact inverse is (the bar of test_bf16_truncation_is_honoured).
        K, V, beta, g = _to_dev(inp)
        W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, 128, N, S)
        assert gdn.gdn_device_status() == gdn.GDN_OK
        Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
        Wo, Uo, To = _oracle(inp, N, S)
        We, Ue, Te = _oracle(inp, exact=True)
        for got, ref, ex in ((Tg, To, Te), (Wg, Wo, We), (Ug, Uo, Ue)):
            gap = orc.rel_frobenius(ref, ex)
            err = orc.rel_frobenius(got, ref)
            floor = orc.rel_frobenius(_bf16_round(ref), ref)
            assert np.all(err <= np.maximum(np.maximum(TOL_BF16, floor + 2e-4), gap / 5))
    else:
        _check(inp, TOL_BF16, N, S)
    inp = gen.make_inputs(1, 1, 2, 128, 128, 128, 128, seed=46)
    _check(inp, TOL_BF16, N, S)


def test_bf16_truncation_is_honoured():
    """With few residual terms the truncated result differs visibly from the exact inverse;
    the kernel must reproduce the truncated one."""
    C = 64
    inp = gen.make_inputs(1, 1, 1, 256, C, 128, 128, seed=50, adversarial_heads="all")
    inp.beta.fill_(0.5)
    Wo, Uo, To = _oracle(inp, 3, 1)
    We, Ue, Te = _oracle(inp, exact=True)
    gap = orc.rel_frobenius(To, Te).min()
    assert gap > 1e-2, gap
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, C, 3, 1)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
    # these inputs lie outside the workload regimes (the truncated series has not converged), so the
    # bar here is only "much closer to the truncated result than the exact inverse is"
    assert orc.rel_frobenius(Tg, To).max() < gap / 5
    assert orc.rel_frobenius(Tg, Te).min() > gap / 2


def test_bf16_gqa_and_ragged_tiles():
    # grouped heads: 2 key heads, 6 value heads; T = 192 leaves a half-empty last tile per head
    inp = gen.make_inputs(2, 2, 6, 192, 64, 128, 128, seed=60, adversarial_heads="odd")
    _check(inp, TOL_BF16)
    inp = gen.make_inputs(1, 1, 3, 64, 64, 128, 128, seed=61)
    _check(inp, TOL_BF16)
    inp = gen.make_inputs(1, 1, 2, 48, 16, 128, 128, seed=62)
    _check(inp, TOL_BF16)
    inp = gen.make_inputs(3, 1, 1, 32, 32, 128, 128, seed=63)
    _check(inp, TOL_BF16)


def test_bf16_without_tinv_and_determinism():
    inp = gen.make_inputs(1, 2, 2, 512, 64, 128, 128, seed=70)
    K, V, beta, g = _to_dev(inp)
    W1, U1, T1 = gdn.chunk_prepare(K, V, beta, g, 64)
    W2, U2, _ = gdn.chunk_prepare(K, V, beta, g, 64, want_tinv=False)
    W3, U3, T3 = gdn.chunk_prepare(K, V, beta, g, 64)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(W1, W2) and torch.equal(U1, U2)
    assert torch.equal(W1, W3) and torch.equal(U1, U3) and torch.equal(T1, T3)


@pytest.mark.parametrize("C", [16, 32, 64, 128])
def test_bf16_forward_substitution_kernel(C):
    # C = 128: the two 64-blocks by substitution, the lower-left block by the block formula of App. E
    inp = gen.make_inputs(1, 2, 4, 512, C, 128, 128, seed=80 + C, adversarial_heads="odd")
    _check(inp, TOL_BF16, method="fwdsubst", exact=True)


@pytest.mark.parametrize("C", [16, 32, 64, 128])
def test_bf16_blocked_forward_substitution_kernel(C):
    inp = gen.make_inputs(1, 2, 4, 512, C, 128, 128, seed=85 + C, adversarial_heads="odd")
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, C, method="fwdsubst", variant=gdn.GDN_FWDSUBST_BLOCKED)
    W2, U2, Tinv2 = gdn.chunk_prepare(K, V, beta, g, C, method="fwdsubst", variant=gdn.GDN_FWDSUBST_ROWS)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
    Wo, Uo, To = _oracle(inp, exact=True)
    for got, ref in ((Tg, To), (Wg, Wo), (Ug, Uo)):
        floor = orc.rel_frobenius(_bf16_round(ref), ref)
        assert np.all(orc.rel_frobenius(got, ref) <= np.maximum(TOL_BF16, floor + 2e-4))
    # the two orders of the same substitution agree to bf16 output rounding
    assert (Tinv.float() - Tinv2.float()).abs().max() <= 1e-2


@pytest.mark.parametrize("adv", ["none", "odd", "all"])
def test_bf16_blocked_forward_substitution_with_tensor_core_merge(adv):
    """32 x 32 diagonal blocks by substitution, lower-left block by the block formula of App. E on the tensor cores
    (hi + lo operands): the exact inverse, at the bf16 floor also on strongly correlated keys; several tiles, grouped
    heads and a ragged last tile."""
    inp = gen.make_inputs(2, 2, 4, 448, 64, 128, 128, seed=180, adversarial_heads=adv)
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, 64, method="fwdsubst", variant=gdn.GDN_FWDSUBST_BLOCKED_TC)
    W2, U2, Tinv2 = gdn.chunk_prepare(K, V, beta, g, 64, method="fwdsubst", variant=gdn.GDN_FWDSUBST_BLOCKED_TC)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert torch.equal(W, W2) and torch.equal(U, U2) and torch.equal(Tinv, Tinv2)
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
    Wo, Uo, To = _oracle(inp, exact=True)
    for name, got, ref in (("Tinv", Tg, To), ("W", Wg, Wo), ("U", Ug, Uo)):
        err = orc.rel_frobenius(got, ref)
        bound = _bound(ref, TOL_BF16)
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), f"{name} rel-F {err[worst]:.3e} > {bound[worst]:.3e} at chunk {worst}"
    assert np.all(np.triu(Tg, 1) == 0) and np.all(np.diagonal(Tg, axis1=-2, axis2=-1) == 1)
    # other chunk sizes are refused
    rc = gdn.gdn_chunk_prepare_fwdsubst(K, V, beta, g, inp.B, inp.H_k, inp.H_v, inp.T, 32, 128, 128, gdn.GDN_DTYPE_BF16,
                                        gdn.GDN_FWDSUBST_BLOCKED_TC, W, U, Tinv, check=False)
    assert rc == gdn.GDN_ERR_UNSUPPORTED


@pytest.mark.parametrize("C", [16, 32, 64, 128])
def test_fp32_blocked_forward_substitution(C):
    inp = gen.make_inputs(1, 1, 2, 2 * C, C, 64, 64, seed=95 + C, dtype=torch.float32)
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, C, method="fwdsubst", variant=gdn.GDN_FWDSUBST_BLOCKED)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
    Wo, Uo, To = _oracle(inp, exact=True)
    assert orc.rel_frobenius(Tg, To).max() <= TOL_FP32 and orc.rel_frobenius(Wg, Wo).max() <= TOL_FP32
    assert orc.rel_frobenius(Ug, Uo).max() <= TOL_FP32


@pytest.mark.parametrize("C,dtype", [(64, torch.bfloat16), (128, torch.bfloat16), (32, torch.bfloat16), (16, torch.bfloat16),
                                     (64, torch.float32), (24, torch.float32)])
@pytest.mark.parametrize("case", ["zero_k", "zero_beta", "closed_gate", "open_gate_beta_one"])
def test_degenerate_inputs(C, dtype, case):
    """Degenerate chunks: no keys, no writes (beta = 0), a gate that closes between any two tokens (A = 0: T = I exactly,
    W = diag(beta) K, U = diag(beta) V), and the other end, the ungated delta rule with beta = 1 (g = 0: no decay inside
    a chunk, the far part of T is as large as its band), against the oracle of the same scheme."""
    inp = gen.make_inputs(1, 1, 2, 4 * C, C, 128, 128, seed=77 + C, dtype=dtype)
    if case == "zero_k":
        inp.K.zero_()
    elif case == "zero_beta":
        inp.beta.zero_()
    elif case == "closed_gate":
        inp.g = (-200.0 * (torch.arange(inp.T) % C).float()).expand_as(inp.g).contiguous()
    else:
        inp.g.zero_()
        inp.beta.fill_(1.0)
    bf16 = dtype == torch.bfloat16
    # Without decay the far entries of T are O(0.1) each instead of vanishing with the distance, and they enter the
    # W / U products as single bf16 operands (the low halves cover the diagonal and the band): that adds ~1.2e-3 to the
    # 1.7e-3 of the output rounding on 64-row blocks (measured 2.03e-3 .. 2.12e-3). Outside the paper's gated workloads;
    # the bar for this case is 2.5e-3.
    tol = (2.5e-3 if case == "open_gate_beta_one" and C >= 64 else TOL_BF16) if bf16 else TOL_FP32
    _check(inp, tol)
    if case == "open_gate_beta_one":
        return
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, inp.C)
    assert torch.equal(Tinv, torch.eye(C, device="cuda", dtype=dtype).expand_as(Tinv))
    if case == "zero_k":
        assert not W.any()
    if case == "zero_beta":
        assert not W.any() and not U.any()


def test_empty_batch_is_a_no_op():
    K = torch.empty(0, 2, 128, 128, dtype=torch.bfloat16, device="cuda")
    V = torch.empty(0, 2, 128, 128, dtype=torch.bfloat16, device="cuda")
    b = torch.empty(0, 2, 128, device="cuda"); g = torch.empty(0, 2, 128, device="cuda")
    W = torch.empty_like(K); U = torch.empty_like(V)
    dummy = torch.zeros(16, device="cuda")
    # empty tensors have null data pointers in torch; pass a valid dummy allocation instead
    lib = gdn.load_library()
    import ctypes
    p = ctypes.c_void_p(dummy.data_ptr())
    rc = lib.gdn_chunk_prepare(p, p, p, p, 0, 2, 128, 64, 128, 128, -1, -1, gdn.GDN_DTYPE_BF16, p, p, None, None)
    assert rc == gdn.GDN_OK


def test_empty_tensors_through_the_binding():
    """torch gives tensors without elements a null data pointer; the binding passes a stand-in address, so an empty
    batch or zero tokens is an empty problem on every entry point, not a missing argument."""
    K = torch.zeros(0, 2, 128, 128, dtype=torch.bfloat16, device="cuda")
    b = torch.zeros(0, 2, 128, device="cuda")
    n0 = gdn.gdn_launch_count()
    W, U, Tinv = gdn.chunk_prepare(K, K, b, b, 64)
    assert W.shape == K.shape and Tinv.shape == (0, 2, 2, 64, 64)
    K0 = torch.zeros(1, 2, 0, 128, dtype=torch.bfloat16, device="cuda")
    b0 = torch.zeros(1, 2, 0, device="cuda")
    W, U, Tinv = gdn.chunk_prepare(K0, K0, b0, b0, 64, method="fwdsubst")
    assert W.shape == K0.shape
    Kf = torch.zeros(0, 1, 48, 40, device="cuda")
    W, U, Tinv = gdn.chunk_prepare(Kf, Kf, torch.zeros(0, 1, 48, device="cuda"), torch.zeros(0, 1, 48, device="cuda"), 24)
    assert W.shape == Kf.shape
    for bits, fn in ((8, gdn.chunk_prepare_int8), (16, gdn.chunk_prepare_int16)):
        q = gen.make_int8_inputs(gen.make_inputs(1, 1, 1, 64, 64, 128, 128, seed=1), bits)
        e = gen.Int8Inputs(q.Kq[:0].cuda(), q.Vq[:0].cuda(), q.k_exp[:0].cuda(), q.v_exp[:0].cuda(), q.beta_q[:0].cuda(),
                           q.decay_q[:0].cuda(), 0, 1, 1, 64, 64, 128, 128)
        out = fn(e)
        assert out[0].shape == (0, 1, 64, 128)
    assert gdn.gdn_device_status() == gdn.GDN_OK and gdn.gdn_launch_count() == n0


def test_argument_errors_on_device():
    inp = gen.make_inputs(1, 1, 1, 128, 64, 128, 128, seed=90)
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.alloc_outputs(K, V, 64)
    args = dict(check=False)
    assert gdn.gdn_chunk_prepare(K, V, beta, g, 1, 1, 128, 48, 128, 128, -1, -1, 1, W, U, Tinv, **args) == gdn.GDN_ERR_INVALID_ARG
    assert gdn.gdn_chunk_prepare(K, V, beta, g, 1, 1, 128, 64, 128, 128, 0, 3, 1, W, U, Tinv, **args) == gdn.GDN_ERR_INVALID_ARG
    # (orders above 7 and other feature sizes run on the plain FMA kernel; these are outside both kernels)
    assert gdn.gdn_chunk_prepare(K, V, beta, g, 1, 1, 128, 64, 100, 128, -1, -1, 1, W, U, Tinv, **args) == gdn.GDN_ERR_UNSUPPORTED
    assert gdn.gdn_chunk_prepare(K, V, beta, g, 1, 1, 128, 64, 264, 128, -1, -1, 1, W, U, Tinv, **args) == gdn.GDN_ERR_UNSUPPORTED
    assert gdn.gdn_chunk_prepare_ex(K, V, beta, g, 1, 1, 1, 128, 64, 64, 64, -1, -1, 1, W, U, Tinv, gdn.GDN_FLAG_LAYOUT_BTHD,
                                    **args) == gdn.GDN_ERR_UNSUPPORTED  # token-major: tensor-core kernel only
    buf = torch.zeros(129, device="cuda")
    g_misaligned = buf[1:]  # 4 bytes past a 16-byte boundary
    assert gdn.gdn_chunk_prepare(K, V, beta, g_misaligned, 1, 1, 128, 64, 128, 128, -1, -1, 1, W, U, Tinv, **args) == gdn.GDN_ERR_ALIGN
    assert gdn.gdn_device_status() == gdn.GDN_OK


# ---------------------------------------------------------------- optional prologue and fp32 outputs (gdn_chunk_prepare_ex)
def _raw_inputs(B, H_k, H_v, T, C, seed, dtype=torch.bfloat16, adv="none"):
    """Unnormalised keys with row norms in [0.5, 3] and RAW (not prefix-summed) log-gates."""
    inp = gen.make_inputs(B, H_k, H_v, T, C, 128, 128, seed=seed, dtype=dtype, adversarial_heads=adv)
    gsc = torch.Generator().manual_seed(seed + 1000)
    scale = 0.5 + 2.5 * torch.rand(B, H_k, T, 1, generator=gsc)
    inp.K = (inp.K.float() * scale).to(dtype).contiguous()
    graw = inp.g.view(B, H_v, T // C, C).diff(dim=-1, prepend=torch.zeros(B, H_v, T // C, 1)).reshape(B, H_v, T).contiguous()
    return inp, graw


def _check_ex(inp, graw, flags, tol, N=-1, S=-1):
    K, V, beta = inp.K.cuda(), inp.V.cuda(), inp.beta.cuda()
    g_raw = bool(flags & gdn.GDN_FLAG_G_RAW)
    l2 = bool(flags & gdn.GDN_FLAG_K_L2NORM)
    g = (graw if g_raw else inp.g).cuda()
    W, U, Tinv = gdn.chunk_prepare(K, V, beta, g, inp.C, N, S, flags=flags)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    if flags & gdn.GDN_FLAG_OUT_FP32:
        assert W.dtype == torch.float32 and Tinv.dtype == torch.float32
    Wg, Ug, Tg = _gpu_chunks(W, U, Tinv, inp)
    sl = gen.chunk_slices(inp, range(inp.n_chunks))
    Kc = np.stack([s[0] for s in sl]); Vc = np.stack([s[1] for s in sl]); bc = np.stack([s[2] for s in sl])
    gsrc = graw if g_raw else inp.g
    gc = gsrc.double().numpy().reshape(inp.n_chunks, inp.C)
    Wo, Uo, To = orc.chunk_prepare(Kc, Vc, bc, gc, None if N < 0 else N, None if S < 0 else S, g_raw=g_raw, k_l2norm=l2,
                                   w_gated=bool(flags & gdn.GDN_FLAG_W_GATED))
    for name, got, ref in (("Tinv", Tg, To), ("W", Wg, Wo), ("U", Ug, Uo)):
        err = orc.rel_frobenius(got, ref)
        bound = _bound(ref, tol, bf16_out=inp.K.dtype == torch.bfloat16 and not (flags & gdn.GDN_FLAG_OUT_FP32))
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), f"{name} rel-F {err[worst]:.3e} > {bound[worst]:.3e} at chunk {worst} (flags {flags})"


@pytest.mark.parametrize("C", [16, 32, 64, 128])
@pytest.mark.parametrize("flags", [1, 2, 3])
def test_bf16_prologue_flags(C, flags):
    inp, graw = _raw_inputs(1, 2, 4, 512, C, seed=200 + C + flags)
    _check_ex(inp, graw, flags, TOL_BF16)


@pytest.mark.parametrize("C", [16, 64, 128])
@pytest.mark.parametrize("adv", ["none", "all"])
def test_bf16_fp32_outputs_show_the_accumulators(C, adv):
    """With fp32 outputs the bf16 output rounding (1.7e-3) is gone: what remains is the error of the bf16
    MMA operands, which the fp32 band / hi-lo split keeps small even for strongly correlated keys."""
    inp = gen.make_inputs(1, 2, 2, 512, C, 128, 128, seed=230 + C, adversarial_heads=adv)
    _check_ex(inp, None, gdn.GDN_FLAG_OUT_FP32, 5e-4)


@pytest.mark.parametrize("C", [16, 32, 64, 128])
@pytest.mark.parametrize("flags", [16, 17, 19, 23])
def test_bf16_gated_w(C, flags):
    """GDN_FLAG_W_GATED: W = T diag(beta exp(g)) K, alone and with the raw-gate / key-normalisation / fp32 flags."""
    inp, graw = _raw_inputs(1, 2, 2, 4 * C, C, seed=300 + C + flags, adv="odd" if C <= 64 else "none")
    if not (flags & gdn.GDN_FLAG_K_L2NORM):
        inp = gen.make_inputs(1, 2, 2, 4 * C, C, 128, 128, seed=300 + C + flags, adversarial_heads="odd" if C <= 64 else "none")
    _check_ex(inp, graw, flags, 5e-4 if (flags & gdn.GDN_FLAG_OUT_FP32) else TOL_BF16)


@pytest.mark.parametrize("C", [16, 64, 128])
def test_fp32_gated_w(C):
    inp, graw = _raw_inputs(1, 1, 2, 2 * C, C, seed=310 + C, dtype=torch.float32)
    _check_ex(inp, graw, 16 + 3, TOL_FP32 * 3)


@pytest.mark.parametrize("C,dtype", [(64, torch.bfloat16), (128, torch.bfloat16), (16, torch.bfloat16), (64, torch.float32)])
def test_key_normalisation_with_zero_keys(C, dtype):
    """GDN_FLAG_K_L2NORM on keys with a few all-zero rows (tokens that write nothing): such a key stays zero, the result
    is finite and meets the usual bars against the oracle (which defines the same)."""
    inp, graw = _raw_inputs(1, 1, 2, 2 * C, C, seed=330 + C, dtype=dtype)
    inp.K[0, 0, [0, 7, C - 1, C + 3]] = 0
    W, U, Tinv = gdn.chunk_prepare(inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), graw.cuda(), C, flags=3)
    assert bool(torch.isfinite(W.float()).all() and torch.isfinite(U.float()).all() and torch.isfinite(Tinv.float()).all())
    assert not W[0, :, [0, 7, C - 1, C + 3]].any()
    _check_ex(inp, graw, 3, TOL_BF16 if dtype == torch.bfloat16 else TOL_FP32 * 3)


def test_bf16_all_flags_together_gqa_ragged():
    inp, graw = _raw_inputs(2, 1, 3, 192, 64, seed=250, adv="odd")
    _check_ex(inp, graw, 7, 5e-4)


@pytest.mark.parametrize("C,flags", [(16, 3), (64, 1), (64, 2), (128, 3)])
def test_fp32_prologue_flags(C, flags):
    inp, graw = _raw_inputs(1, 1, 2, 2 * C, C, seed=260 + C, dtype=torch.float32)
    _check_ex(inp, graw, flags, TOL_FP32 * 3)


@pytest.mark.parametrize("C", [16, 32, 64, 128])
@pytest.mark.parametrize("extra", [0, 3, 7])
def test_bf16_token_major_layout(C, extra):
    """GDN_FLAG_LAYOUT_BTHD: K, V, beta, g, W, U in [B, T, H, d] order (grouped heads, a ragged last tile); the
    result must equal the head-major one element for element after transposing back, and meet the oracle bars."""
    inp, graw = _raw_inputs(2, 2, 4, 3 * C if C == 128 else 320 if C != 32 else 352, C, seed=280 + C, adv="odd")
    if not (extra & gdn.GDN_FLAG_K_L2NORM):
        inp = gen.make_inputs(2, 2, 4, inp.T, C, 128, 128, seed=280 + C, adversarial_heads="odd")
    g_src = graw if (extra & gdn.GDN_FLAG_G_RAW) else inp.g
    K, V, beta, g = inp.K.cuda(), inp.V.cuda(), inp.beta.cuda(), g_src.cuda()
    tm = lambda x: x.transpose(1, 2).contiguous()
    flags = extra | gdn.GDN_FLAG_LAYOUT_BTHD
    W, U, Tinv = gdn.chunk_prepare(tm(K), tm(V), tm(beta), tm(g), C, flags=flags)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert W.shape == (inp.B, inp.T, inp.H_v, inp.d_k) and Tinv.shape == (inp.B, inp.H_v, inp.T // C, C, C)
    # reference: the same call in the head-major layout (the extra flags go through the same instantiation)
    if extra:
        W0, U0, T0 = gdn.chunk_prepare(K, V, beta, g, C, flags=extra)
    else:
        W0, U0, T0 = gdn.chunk_prepare(K, V, beta, g, C)
    assert torch.equal(tm(W0), W)
    assert torch.equal(tm(U0), U)
    assert torch.equal(T0, Tinv)
    # and against the oracle
    Wg, Ug, Tg = _gpu_chunks(W.transpose(1, 2).contiguous(), U.transpose(1, 2).contiguous(), Tinv, inp)
    sl = gen.chunk_slices(inp, range(inp.n_chunks))
    Kc = np.stack([s[0] for s in sl]); Vc = np.stack([s[1] for s in sl]); bc = np.stack([s[2] for s in sl])
    gc = g_src.double().numpy().reshape(inp.n_chunks, C)
    Wo, Uo, To = orc.chunk_prepare(Kc, Vc, bc, gc, None, None, g_raw=bool(extra & 1), k_l2norm=bool(extra & 2))
    fp32_out = bool(extra & gdn.GDN_FLAG_OUT_FP32)
    for name, got, ref in (("Tinv", Tg, To), ("W", Wg, Wo), ("U", Ug, Uo)):
        err = orc.rel_frobenius(got, ref)
        bound = _bound(ref, 5e-4 if fp32_out else TOL_BF16, bf16_out=not fp32_out)
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), f"{name} rel-F {err[worst]:.3e} > {bound[worst]:.3e} at chunk {worst}"


def test_token_major_layout_is_bf16_only():
    inp = gen.make_inputs(1, 1, 1, 128, 64, 128, 128, seed=281, dtype=torch.float32)
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.alloc_outputs(K, V, 64)
    rc = gdn.gdn_chunk_prepare_ex(K, V, beta, g, 1, 1, 1, 128, 64, 128, 128, -1, -1, 0, W, U, Tinv,
                                  gdn.GDN_FLAG_LAYOUT_BTHD, check=False)
    assert rc == gdn.GDN_ERR_UNSUPPORTED


def test_ex_rejects_unknown_flags():
    inp = gen.make_inputs(1, 1, 1, 128, 64, 128, 128, seed=270)
    K, V, beta, g = _to_dev(inp)
    W, U, Tinv = gdn.alloc_outputs(K, V, 64)
    rc = gdn.gdn_chunk_prepare_ex(K, V, beta, g, 1, 1, 1, 128, 64, 128, 128, -1, -1, 1, W, U, Tinv, 32, check=False)
    assert rc == gdn.GDN_ERR_INVALID_ARG


def test_bounded_wait_gives_up_and_reports():
    """A wait on an mbarrier that nothing completes runs out after about a second: the status word reports
    GDN_ERR_TIMEOUT once, and the context stays usable (a normal call afterwards is correct)."""
    assert gdn.gdn_device_status() == gdn.GDN_OK
    assert gdn.gdn_selftest_bounded_wait() == gdn.GDN_OK
    assert gdn.gdn_device_status() == gdn.GDN_ERR_TIMEOUT
    assert gdn.gdn_device_status() == gdn.GDN_OK
    inp = gen.make_inputs(1, 1, 1, 256, 64, 128, 128, seed=290)
    _check(inp, TOL_BF16)


def test_host_threads_on_their_own_streams_do_not_disturb_each_other():
    """Four host threads, each on its own stream, 100 calls each on its own problem: every result equals the one a
    single-threaded call gives (the library keeps no per-call state on the host or the device)."""
    import threading
    problems = [gen.make_inputs(2, 2, 4, 64 * (3 + i), 64, 128, 128, seed=700 + i) for i in range(4)]
    dev = [tuple(x.cuda() for x in (p.K, p.V, p.beta, p.g)) for p in problems]
    want = [gdn.chunk_prepare(*d, 64) for d in dev]
    torch.cuda.synchronize()
    errors = []

    def work(k):
        stream = torch.cuda.Stream()
        try:
            with torch.cuda.stream(stream):
                for _ in range(100):
                    got = gdn.chunk_prepare(*dev[k], 64)
                stream.synchronize()
            if not all(torch.equal(a, b) for a, b in zip(got, want[k])):
                errors.append(f"thread {k}: results differ")
        except Exception as exc:  # a failure in a thread must fail the test
            errors.append(f"thread {k}: {exc!r}")

    threads = [threading.Thread(target=work, args=(k,)) for k in range(4)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    torch.cuda.synchronize()
    assert not errors and gdn.gdn_device_status() == gdn.GDN_OK


@pytest.mark.parametrize("adv", ["none", "all"])
@pytest.mark.parametrize("N,S", [(-1, -1), (3, 15), (5, 8)])
def test_bf16_large_launch_form_on_small_cases(adv, N, S, monkeypatch):
    """Large launches of the default 64-chunk path run a second form of the kernel (every tensor-core product an M = 64
    instruction on one chunk, the rows of the two chunks interleaved over the lanes; the library picks it by launch
    size). GDN_FORCE_M64 selects it here on small cases: grouped heads, a ragged last tile, benign and adversarial
    heads, the exact inverse (S = 15), a wider band (N = 5), with and without the Tinv output; same bars against the
    oracle, and W, U, Tinv within one bf16 rounding of the other form (the two differ in the order of fp32 sums)."""
    inp = gen.make_inputs(2, 2, 4, 64 * 7, 64, 128, 128, seed=800, adversarial_heads=adv)
    K, V, beta, g = _to_dev(inp)
    monkeypatch.setenv("GDN_FORCE_M64", "0")
    ref = gdn.chunk_prepare(K, V, beta, g, 64, N, S)
    monkeypatch.setenv("GDN_FORCE_M64", "1")
    _check(inp, TOL_BF16, N, S)
    got = gdn.chunk_prepare(K, V, beta, g, 64, N, S)
    again = gdn.chunk_prepare(K, V, beta, g, 64, N, S)
    no_t = gdn.chunk_prepare(K, V, beta, g, 64, N, S, want_tinv=False)
    assert gdn.gdn_device_status() == gdn.GDN_OK
    for a, b in zip(got, again):
        assert torch.equal(a, b)  # bit-identical repeats
    assert torch.equal(no_t[0], got[0]) and torch.equal(no_t[1], got[1]) and no_t[2] is None
    for a, b in zip(got, ref):
        d = (a.float() - b.float()).abs()
        assert bool((d <= 2.0 ** -7 * b.float().abs() + 1e-6).all())

"""The segmented state passing on the library's built-in scratch array (`gdn_chunk_state_output_segmented_noalloc`).

Some users of the library cannot allocate device memory around a call: an inference engine that has handed out all of
the GPU's memory at start-up, a plug-in without an allocator, a loop that must not pay for cudaMalloc's
synchronisation. For them the library carries a fixed scratch array of its own. This file checks, through the C ABI,
that the entry point gives what `gdn_chunk_state_output_segmented` (caller-owned workspace) gives, on two calls in a
row (the second one finds the first one's leftovers in the shared array), and that a problem beyond the array's size
is refused with GDN_ERR_SCRATCH before anything is launched.

The file is named so that pytest collects it last: if it fails, a run that stops at the first failure has already
run every other test.
"""
import ctypes

import pytest
import torch

from paper_2606_06034_b200 import binding as gdn
from paper_2606_06034_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _problem(H_k, H_v, T, seed):
    C = 64
    inp = gen.make_inputs(1, H_k, H_v, T, C, 128, 128, seed=seed, adversarial_heads="odd")
    gq = torch.Generator().manual_seed(seed + 1)
    Q = torch.randn(1, H_k, T, 128, generator=gq)
    Q = (Q / Q.norm(dim=-1, keepdim=True)).to(torch.bfloat16).cuda()
    K, g = inp.K.cuda(), inp.g.cuda()
    W, U, _ = gdn.chunk_prepare(K, inp.V.cuda(), inp.beta.cuda(), g, C, flags=gdn.GDN_FLAG_W_GATED)
    S0 = (0.1 * torch.randn(H_v, 128, 128, generator=gq)).cuda()
    return Q[0].contiguous(), K[0].contiguous(), W[0].contiguous(), U[0].contiguous(), g[0].contiguous(), S0


def _rel(x, ref):
    x, ref = x.double(), ref.double()
    return float((x - ref).norm() / ref.norm().clamp_min(1e-300))


def test_noalloc_entry_point_matches_the_workspace_entry_point_twice_in_a_row():
    C, scale = 64, 128 ** -0.5
    lib = gdn.load_library()
    # two different problems, so that the second call really overwrites what the first left in the shared array
    cases = [(1, 2, 1024, 3, 700), (2, 4, 1536, 4, 710)]
    for H_k, H_v, T, segments, seed in cases:
        Q, K, W, U, g, S0 = _problem(H_k, H_v, T, seed)
        assert H_v * (6 * segments - 6) <= 128
        # reference: the existing entry point with a workspace the caller owns
        O_ref, S_ref = gdn.chunk_state_output_segmented(Q, K, W, U, g, C, scale, S0, segments=segments)
        assert gdn.gdn_device_status() == gdn.GDN_OK
        # every buffer of the new call exists before it: the call itself must not need an allocation
        O = torch.full_like(U, float("nan"))
        S = torch.full((H_v, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        rc = lib.gdn_chunk_state_output_segmented_noalloc(
            ctypes.c_void_p(Q.data_ptr()), ctypes.c_void_p(K.data_ptr()), ctypes.c_void_p(W.data_ptr()),
            ctypes.c_void_p(U.data_ptr()), ctypes.c_void_p(g.data_ptr()), H_k, H_v, T, C, 128, 128, ctypes.c_float(scale),
            ctypes.c_void_p(S0.data_ptr()), ctypes.c_void_p(O.data_ptr()), ctypes.c_void_p(S.data_ptr()), segments, 0,
            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == gdn.GDN_OK, gdn.status_string(rc)
        assert gdn.gdn_device_status() == gdn.GDN_OK
        assert bool(torch.isfinite(O).all()) and bool(torch.isfinite(S).all())
        # the same kernels run in the same order on the same numbers: the bar is the one the segmented tests use for
        # two evaluations of the same thing (they are in fact expected to agree to the last bit)
        assert _rel(O, O_ref) <= 2e-3 and _rel(S, S_ref) <= 1e-5
        per_chunk = (O.double() - O_ref.double()).reshape(H_v, T // C, -1).norm(dim=-1) / \
            O_ref.double().reshape(H_v, T // C, -1).norm(dim=-1).clamp_min(1e-300)
        assert float(per_chunk.max()) <= 2e-3


def test_noalloc_entry_point_refuses_what_its_array_cannot_hold():
    C, scale = 64, 128 ** -0.5
    H_k, H_v, T = 2, 32, 512
    bf = dict(dtype=torch.bfloat16, device="cuda")
    Q, K = torch.zeros(H_k, T, 128, **bf), torch.zeros(H_k, T, 128, **bf)
    W, U, O = torch.zeros(H_v, T, 128, **bf), torch.zeros(H_v, T, 128, **bf), torch.zeros(H_v, T, 128, **bf)
    g = torch.zeros(H_v, T, device="cuda")
    before = gdn.gdn_launch_count()
    # 32 heads x (6 * 3 - 6) = 384 state blocks > 128
    rc = gdn.gdn_chunk_state_output_segmented_noalloc(Q, K, W, U, g, H_k, H_v, T, C, 128, 128, scale, None, O, None, 3, check=False)
    assert rc == gdn.GDN_ERR_SCRATCH
    assert "scratch" in gdn.status_string(rc)
    assert gdn.gdn_launch_count() == before
    # one segment needs no scratch and is always accepted
    rc = gdn.gdn_chunk_state_output_segmented_noalloc(Q, K, W, U, g, H_k, H_v, T, C, 128, 128, scale, None, O, None, 1, check=False)
    assert rc == gdn.GDN_OK
    assert gdn.gdn_device_status() == gdn.GDN_OK

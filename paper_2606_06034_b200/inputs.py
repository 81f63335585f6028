"""Seeded synthetic inputs for the chunk-prepare path.

This module only draws random tensors with the shapes and value distributions of
the workloads; it holds none of the method's arithmetic, so the CUDA path's
tests, the benchmark and the CPU oracle's tests can all take inputs from it.

Layouts (contiguous):
  K     [B, H_k, T, d_k]   keys, rows L2-normalised in fp32 and then cast
  V     [B, H_v, T, d_v]   values
  beta  [B, H_v, T]  fp32  write strength, sigmoid of a normal draw
  g     [B, H_v, T]  fp32  cumulative log-gate, prefix sum restarted at every
                           chunk of C tokens, of -softplus(normal draw)

Two regimes:
  "benign"       the distributions above
  "adversarial"  beta = 0.99, g = 0 and highly correlated keys: per chunk one
                 direction u ~ N(0, I), K_t = u + 0.1 * eps_t, row-normalised
                 (cosine ~ 0.99), which maximises growth of the Neumann terms.
`adversarial_heads="odd"` applies the adversarial regime to value heads with
odd index (and to the key heads they read), the rest stay benign.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass
class ChunkInputs:
    K: torch.Tensor
    V: torch.Tensor
    beta: torch.Tensor
    g: torch.Tensor
    B: int
    H_k: int
    H_v: int
    T: int
    C: int
    d_k: int
    d_v: int

    @property
    def n_chunks(self) -> int:
        return self.B * self.H_v * (self.T // self.C)


def make_inputs(B: int, H_k: int, H_v: int, T: int, C: int, d_k: int, d_v: int, *,
                seed: int, dtype: torch.dtype = torch.bfloat16,
                device: str | torch.device = "cpu",
                adversarial_heads: str = "none") -> ChunkInputs:
    """Draw one workload. Tensors are drawn in the fixed order K, V, beta, g."""
    assert T % C == 0 and H_v % H_k == 0
    assert adversarial_heads in ("none", "odd", "all")
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32)

    Kf = randn(B, H_k, T, d_k)
    if adversarial_heads != "none":
        n_ch = T // C
        u = randn(B, H_k, n_ch, 1, d_k)
        eps = randn(B, H_k, n_ch, C, d_k)
        Kadv = (u + 0.1 * eps).reshape(B, H_k, T, d_k)
        if adversarial_heads == "all":
            Kf = Kadv
        else:
            # key heads with odd index are adversarial, and so are the value
            # heads that read them (see `sel` below)
            odd = (torch.arange(H_k, device=dev) % 2 == 1).view(1, H_k, 1, 1)
            Kf = torch.where(odd, Kadv, Kf)
        del u, eps, Kadv
    Kf = Kf / Kf.norm(dim=-1, keepdim=True).clamp_min(1e-12)
    K = Kf.to(dtype)
    del Kf
    V = randn(B, H_v, T, d_v).to(dtype)
    beta = torch.sigmoid(randn(B, H_v, T))
    graw = -torch.nn.functional.softplus(randn(B, H_v, T))
    g = graw.view(B, H_v, T // C, C).cumsum(dim=-1).reshape(B, H_v, T).contiguous()
    if adversarial_heads != "none":
        if adversarial_heads == "all":
            sel = torch.ones(H_v, dtype=torch.bool, device=dev)
        else:
            group = H_v // H_k
            sel = ((torch.arange(H_v, device=dev) // group) % 2 == 1)
        sel = sel.view(1, H_v, 1)
        beta = torch.where(sel, torch.full_like(beta, 0.99), beta)
        g = torch.where(sel, torch.zeros_like(g), g)
    return ChunkInputs(K.contiguous(), V.contiguous(), beta.contiguous(), g.contiguous(),
                       B, H_k, H_v, T, C, d_k, d_v)


# The named workloads (shapes and regimes); seeds are fixed per workload.
WORKLOADS = {
    # tiny fp32 case the CPU oracle finishes at once
    "tiny_fp32": dict(B=1, H_k=2, H_v=2, T=256, C=64, d_k=128, d_v=128, seed=0,
                      dtype=torch.float32, adversarial_heads="none"),
    # chunk-size sweep, bf16
    "sweep_c16": dict(B=4, H_k=16, H_v=16, T=4096, C=16, d_k=128, d_v=128, seed=1,
                      dtype=torch.bfloat16, adversarial_heads="none"),
    "sweep_c32": dict(B=4, H_k=16, H_v=16, T=4096, C=32, d_k=128, d_v=128, seed=1,
                      dtype=torch.bfloat16, adversarial_heads="none"),
    "sweep_c64": dict(B=4, H_k=16, H_v=16, T=4096, C=64, d_k=128, d_v=128, seed=1,
                      dtype=torch.bfloat16, adversarial_heads="none"),
    "sweep_c128": dict(B=4, H_k=16, H_v=16, T=4096, C=128, d_k=128, d_v=128, seed=1,
                       dtype=torch.bfloat16, adversarial_heads="none"),
    # prefill layer with keys shared by pairs of value heads
    "prefill_gqa": dict(B=1, H_k=16, H_v=32, T=32768, C=64, d_k=128, d_v=128, seed=2,
                        dtype=torch.bfloat16, adversarial_heads="none"),
    # stress + scale, odd heads adversarial
    "stress": dict(B=8, H_k=32, H_v=32, T=65536, C=64, d_k=128, d_v=128, seed=4,
                   dtype=torch.bfloat16, adversarial_heads="odd"),
}


def make_workload(name: str, device: str | torch.device = "cpu", **overrides) -> ChunkInputs:
    cfg = dict(WORKLOADS[name])
    cfg.update(overrides)
    return make_inputs(device=device, **cfg)


def chunk_slices(inp: ChunkInputs, chunk_ids):
    """Host fp64 copies of selected chunks: lists of (K, V, beta, g) numpy arrays.

    chunk id = (b * H_v + h_v) * (T / C) + c. The key head of value head h_v is
    h_v // (H_v / H_k). Values are upcast exactly from the stored dtype.
    """
    n_c = inp.T // inp.C
    group = inp.H_v // inp.H_k
    out = []
    for cid in chunk_ids:
        bh, c = divmod(int(cid), n_c)
        b, hv = divmod(bh, inp.H_v)
        hk = hv // group
        sl = slice(c * inp.C, (c + 1) * inp.C)
        out.append((inp.K[b, hk, sl].double().cpu().numpy(),
                    inp.V[b, hv, sl].double().cpu().numpy(),
                    inp.beta[b, hv, sl].double().cpu().numpy(),
                    inp.g[b, hv, sl].double().cpu().numpy()))
    return out


# ----------------------------------------------------------------------------- integer inputs
@dataclass
class Int8Inputs:
    """Integer buffers of the INT8 entry point (prepared once; both the CUDA path and the CPU oracle read them).

    Kq [B,H_k,T,d_k], Vq [B,H_v,T,d_v] int8 with one power-of-two exponent per chunk (k_exp [B,H_k,T/C],
    v_exp [B,H_v,T/C] int32: value = q * 2^exp); beta_q [B,H_v,T] = round(beta * 2^15) in [0, 32767] stored as
    int16; decay_q [B,H_v,T] int32 = round(-g * log2(e) * 2^8), non-decreasing inside a chunk.
    """
    Kq: torch.Tensor
    Vq: torch.Tensor
    k_exp: torch.Tensor
    v_exp: torch.Tensor
    beta_q: torch.Tensor
    decay_q: torch.Tensor
    B: int
    H_k: int
    H_v: int
    T: int
    C: int
    d_k: int
    d_v: int

    @property
    def n_chunks(self) -> int:
        return self.B * self.H_v * (self.T // self.C)


def _quantise_per_chunk(x: torch.Tensor, C: int, bits: int = 8):
    """Symmetric `bits`-bit mantissas with the smallest power-of-two scale that keeps max|x| / 2^e <= qmax per chunk
    (qmax = 127 or 32767)."""
    B, H, T, d = x.shape
    qmax = float((1 << (bits - 1)) - 1)
    xf = x.float().view(B, H, T // C, C * d)
    m = xf.abs().amax(dim=-1).clamp_min(1e-30)
    e = torch.ceil(torch.log2(m / qmax)).to(torch.int32)
    # guard against log2 rounding: raise e where the scaled maximum still exceeds qmax
    e = torch.where(m / torch.exp2(e.float()) > qmax, e + 1, e)
    q = torch.round(xf / torch.exp2(e.float()).unsqueeze(-1)).clamp_(-qmax, qmax).to(torch.int8 if bits == 8 else torch.int16)
    return q.view(B, H, T, d).contiguous(), e.contiguous()


def make_int8_inputs(inp: ChunkInputs, bits: int = 8) -> Int8Inputs:
    """Integer inputs of the INT8 entry point, or with bits = 16 of the INT16 entry point (Kq, Vq int16, the rest alike)."""
    Kq, k_exp = _quantise_per_chunk(inp.K, inp.C, bits)
    Vq, v_exp = _quantise_per_chunk(inp.V, inp.C, bits)
    beta_q = torch.round(inp.beta.float() * 32768.0).clamp_(0, 32767).to(torch.int16).contiguous()
    decay_q = torch.round(-inp.g.double() * (1.4426950408889634 * 256.0)).to(torch.int32).contiguous()
    return Int8Inputs(Kq, Vq, k_exp, v_exp, beta_q, decay_q, inp.B, inp.H_k, inp.H_v, inp.T, inp.C, inp.d_k, inp.d_v)


def make_int16_inputs(inp: ChunkInputs) -> Int8Inputs:
    return make_int8_inputs(inp, bits=16)


INT_EDGE_CASES = ("all_max", "sign_max", "alt_rows", "one_hot", "max_k_slow_decay", "steep_decay", "exp_extremes",
                  "zero_k", "zero_beta", "zero_all")


def int_edge_inputs(q: Int8Inputs, case: str, bits: int = 8) -> Int8Inputs:
    """Overwrites integer inputs in place with a saturating or degenerate pattern (edge cases of the integer entry
    points: largest mantissas with the gate open and beta at its maximum, where the inverse grows by tens of octaves
    and aligned sums meet shifts far beyond the word size; empty chunks; closed gates; extreme input exponents)."""
    assert case in INT_EDGE_CASES
    m = (1 << (bits - 1)) - 1
    gen = torch.Generator().manual_seed(7)
    ramp = (torch.arange(q.T) % q.C).to(torch.int32)
    if case == "all_max":
        q.Kq.fill_(m); q.Vq.fill_(-m); q.beta_q.fill_(32767); q.decay_q.zero_()
    elif case == "sign_max":
        q.Kq.copy_(((torch.randint(0, 2, q.Kq.shape, generator=gen) * 2 - 1) * m).to(q.Kq.dtype))
        q.Vq.copy_(((torch.randint(0, 2, q.Vq.shape, generator=gen) * 2 - 1) * m).to(q.Vq.dtype))
        q.beta_q.fill_(32767); q.decay_q.zero_()
    elif case == "alt_rows":
        q.Kq.fill_(m); q.Kq[:, :, 1::2] = -m; q.beta_q.fill_(32767); q.decay_q.zero_()
    elif case == "one_hot":
        q.Kq.zero_(); q.Kq[..., 0] = m; q.beta_q.fill_(32767); q.decay_q.zero_()
    elif case == "max_k_slow_decay":
        q.Kq.fill_(m); q.beta_q.fill_(32767); q.decay_q.copy_((ramp * 3).expand_as(q.decay_q))
    elif case == "steep_decay":
        q.decay_q.copy_((ramp * (17 * 256)).expand_as(q.decay_q))  # 17 octaves per token: the gate factor is 0
    elif case == "exp_extremes":
        q.k_exp.fill_(-40); q.v_exp.fill_(37)
    elif case == "zero_k":
        q.Kq.zero_()
    elif case == "zero_beta":
        q.beta_q.zero_()
    elif case == "zero_all":
        q.Kq.zero_(); q.Vq.zero_(); q.beta_q.zero_()
    return q


def int8_chunk_slices(q: Int8Inputs, chunk_ids):
    """Host numpy copies of selected chunks: (Kq, Vq, k_exp, v_exp, beta_q, decay_q) stacked over the chunks."""
    import numpy as np
    n_c = q.T // q.C
    group = q.H_v // q.H_k
    Ks, Vs, ke, ve, bq, dq = [], [], [], [], [], []
    for cid in chunk_ids:
        bh, c = divmod(int(cid), n_c)
        b, hv = divmod(bh, q.H_v)
        hk = hv // group
        sl = slice(c * q.C, (c + 1) * q.C)
        Ks.append(q.Kq[b, hk, sl].cpu().numpy().astype(np.int64))
        Vs.append(q.Vq[b, hv, sl].cpu().numpy().astype(np.int64))
        ke.append(int(q.k_exp[b, hk, c]))
        ve.append(int(q.v_exp[b, hv, c]))
        bq.append(q.beta_q[b, hv, sl].cpu().numpy().astype(np.int64))
        dq.append(q.decay_q[b, hv, sl].cpu().numpy().astype(np.int64))
    return (np.stack(Ks), np.stack(Vs), np.asarray(ke), np.asarray(ve), np.stack(bq), np.stack(dq))

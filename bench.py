#!/usr/bin/env python
"""Benchmark of the chunk-prepare hot path (A-build, multiplication-only inverse, W and U).

One "step" = one pass of the whole path over one batch of synthetic chunks, i.e. one call of
`gdn_chunk_prepare_gqa` through the C-ABI library. Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
  python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...

N > 1: every rank runs the same workload on its own GPU (chunks are independent, there is no
exchange step), the timed region is bracketed by a barrier and the slowest rank's time counts.
`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

torch = None  # imported by main(): the worker processes of the CPU leg re-import this file and must not pay for it


def _import_torch():
    global torch
    if torch is None:
        import torch as _torch
        torch = _torch
    return torch


METRIC = "chunk_prepare_throughput"
UNIT = "chunks/s"
DEFAULT_WORKLOAD = "stress"  # the largest single-GPU configuration (B=8, H=32, T=65536, C=64: 262 144 chunks, 19.5 GB)


# ----------------------------------------------------------------------------- bookkeeping
def matmuls_per_inverse(C: int) -> tuple[int, int]:
    """(number of c x c products, c) the paper's scheme needs per chunk with its default (N, S)."""
    return {16: (6, 16), 32: (7, 32), 64: (11, 64), 128: (24, 64)}[C]


def nominal_flops_per_chunk(C: int, d_k: int, d_v: int) -> float:
    """Dense count as the paper counts matmuls: K K^T, the inverse's products, W and U."""
    m, c = matmuls_per_inverse(C)
    return 2.0 * C * C * d_k + m * 2.0 * c ** 3 + 2.0 * C * C * d_k + 2.0 * C * C * d_v


def algorithmic_bytes_per_chunk(C: int, d_k: int, d_v: int, group: int, esize: int = 2) -> float:
    """What the method must move per chunk: K (once per group of value heads), V, W, U tiles,
    the full Tinv block, beta and g."""
    return (C * d_k * esize) / group + C * d_v * esize + C * d_k * esize + C * d_v * esize + C * C * esize + 8 * C


def int8_integer_ops_per_chunk(C: int, d_k: int, d_v: int, N: int, S: int) -> float:
    """32-bit integer ALU operations the INT8 variant needs per chunk outside the tensor-core products, counted from
    its definition (one op = one add, shift, logic op, min/max, compare/select or multiply on one element):
    a requantisation costs 7 per element of its support (magnitude, running maximum, rounding add, sign fix,
    shift, two clamps), an aligned sum 2 per term and element (shift, add), the gate factor 11 per strictly lower
    entry (difference, table index, shift count, look-up, shift, range test, beta product, rounding add, shift,
    and the two-word product with the Gram entry), the band products and A T0, T0 S (banded operand) one
    multiply-add per term."""
    lower = C * (C - 1) // 2
    band = sum(C - d for d in range(1, N + 1))
    far = lower - band
    sup = lambda m: (C - m) * (C - m + 1) // 2 if m < C else 0  # entries with i - j >= m
    ops = 11 * lower + 7 * lower                                    # gate factor, A
    for n in range(2, N + 1):                                       # band powers
        ops += sum((d - 1) * (C - d) for d in range(n, N + 1)) + 7 * sum(C - d for d in range(n, N + 1))
    ops += 2 * N * band + 7 * band                                  # T0
    ops += N * far + 2 * 2 * far + 7 * far                          # E
    terms = far
    for s_ in range(2, S + 1):                                      # powers of E (products on the tensor cores)
        if s_ * (N + 1) >= C:
            break
        ops += 7 * sup(s_ * (N + 1))
        terms += sup(s_ * (N + 1))
    ops += 2 * terms + 7 * far                                      # sum of the powers
    ops += N * far + 2 * (band + 2 * far) + 7 * lower               # T - I
    ops += 8 * lower                                                # T diag(beta)
    ops += (1 + 4 + 7) * C * (d_k + d_v)                            # W, U: diagonal term, aligned sum, requantisation
    return float(ops)


# integer ALU peak: 148 SMs x 4 sub-partitions x one 16-lane integer pipe each x the maximum SM clock
INT_ALU_LANES = 148 * 4 * 16
SM_MAX_GHZ = 1.965


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
    return 6650.0, 1590.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index = index
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def _reason_names(self, mask: int):
        nv = self.nv
        table = {
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "hw_power_brake_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
            "applications_clocks_setting": getattr(nv, "nvmlClocksThrottleReasonApplicationsClocksSetting", 0x2),
        }
        return [k for k, bit in table.items() if mask & bit]

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.reasons.update(self._reason_names(mask))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=1.0)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle leg
def _bf16_round(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16 and back, on the host (bit arithmetic on the fp32 pattern)."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def sample_chunk_ids(n_heads: int, n_c: int, n_random: int, seed: int):
    """First and last chunk of the first and last head, of head 1 (adversarial in the stress workload), random ones."""
    n = n_heads * n_c
    fixed = [0, n_c - 1, (n_heads - 1) * n_c, n - 1]
    if n_heads > 1:
        fixed += [n_c, 2 * n_c - 1]
    rnd = np.random.default_rng(seed).choice(n, size=min(n_random, n), replace=False).tolist()
    return sorted(set(fixed + rnd))


def parity_report(orc, sample, gpu):
    """The numbers the target asks for next to the throughput, on the chunks the CPU leg ran: error of the GPU result
    against the fp64 evaluation of the same truncated scheme (the graded number) with the bf16 rounding floor of that
    evaluation beside it, the signal-to-noise ratio (Sec. 4.2), and the deviation from the exact inverse."""
    K, V, b, g = sample
    Wo, Uo, To = orc.chunk_prepare(K, V, b, g)
    We, Ue, Te = orc.chunk_prepare(K, V, b, g, exact=True)
    rep = {"chunks": int(K.shape[0]), "reference": "fp64 oracle of the same truncated scheme (order, residual steps as timed)"}
    for name, got, ref, ex in (("Tinv", gpu[2], To, Te), ("W", gpu[0], Wo, We), ("U", gpu[1], Uo, Ue)):
        err = orc.rel_frobenius(got, ref)
        floor = orc.rel_frobenius(_bf16_round(ref), ref)
        w = int(np.argmax(err))
        rep[name] = {"worst_rel_frobenius": float(err[w]), "bf16_floor_of_that_chunk": float(floor[w]),
                     "worst_bf16_floor": float(floor.max()), "mean_rel_frobenius": float(err.mean()),
                     "snr_db_worst": float(orc.snr_db(got, ref).min()), "snr_db_mean": float(orc.snr_db(got, ref).mean()),
                     "gpu_vs_exact_inverse_worst": float(orc.rel_frobenius(got, ex).max()),
                     "scheme_vs_exact_inverse_worst": float(orc.rel_frobenius(ref, ex).max()),
                     # chunks whose bf16 rounding floor alone is above 2e-3, and chunks above 2e-3 whatever the cause
                     "chunks_with_floor_above_2e-3": int((floor > 2e-3).sum()), "chunks_above_2e-3": int((err > 2e-3).sum())}
    return rep


def time_oracle(workload: str, budget_s: float, sample=None, workers=None):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload's chunks, on all usable host cores
    (one process per core, each calling the oracle on batches of chunks). `sample`: (K, V, beta, g) stacks of chunks
    taken from the workload itself; without it a small instance with the same shapes and distributions is drawn."""
    from oracle import pool
    from paper_2606_06034_b200 import inputs as gen

    cfg = dict(gen.WORKLOADS[workload])
    if sample is None:
        small = dict(cfg, B=1, H_k=min(cfg["H_k"], 2), H_v=min(cfg["H_k"], 2) * (cfg["H_v"] // cfg["H_k"]), T=max(cfg["C"] * 16, 1024))
        inp = gen.make_inputs(device="cpu", **small)
        sl = gen.chunk_slices(inp, range(inp.n_chunks))
        sample = tuple(np.stack([s[i] for s in sl]) for i in range(4))
    K, V, b, g = sample
    # calibrate on one core, then size the run so that the CPU work is about budget_s core-seconds
    n0 = min(32, K.shape[0])
    _, t1, _ = pool.timed_chunk_prepare(K[:n0], V[:n0], b[:n0], g[:n0], n0, workers=1)
    per_chunk = t1 / n0
    workers = pool.usable_cores() if workers is None else workers
    n = int(max(n0 * workers, budget_s / max(per_chunk, 1e-9)))
    done, wall, used = pool.timed_chunk_prepare(K, V, b, g, n, workers=workers)
    return {"value": done / wall, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"{done} chunk evaluations over {K.shape[0]} distinct chunks of the {workload} shapes (C={cfg['C']}, d={cfg['d_k']}), "
                      f"fp64 numpy oracle in batches of 32 chunks, one process per core, {wall:.1f} s wall "
                      f"({done * per_chunk:.0f} core-seconds at the single-core rate of {1.0 / per_chunk:.0f} chunks/s); "
                      f"host has {os.cpu_count()} logical cores"}, wall


# ----------------------------------------------------------------------------- GPU legs
def device_time_steps(fn, steps: int, warmup: int, dist_ctx, finalize=None):
    _import_torch()
    """Device time of `steps` calls of fn on the current stream. finalize (optional) joins work that fn left running on
    other streams; it is called after the last step, inside the timed region."""
    for _ in range(warmup):
        fn()
    if finalize is not None:
        finalize()
    torch.cuda.synchronize()
    if dist_ctx is not None:
        dist_ctx.barrier()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    # two untimed launches ahead of the first event: after the synchronize the queue is empty, and the first timed
    # interval would otherwise hold the host's launch latency instead of device time
    fn()
    fn()
    if finalize is not None:
        finalize()  # work on side streams must not leak into the timed region
    evs[0].record(stream)
    for i in range(steps):
        fn()
        if finalize is not None and i == steps - 1:
            finalize()
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    if dist_ctx is not None:
        dist_ctx.barrier()
    total_ms = evs[0].elapsed_time(evs[-1])
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    return total_ms, per


def max_over_ranks(total_ms: float, device, dist_ctx) -> float:
    """The slowest rank's device time counts (all-reduce MAX; identity on one rank)."""
    _import_torch()
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    if dist_ctx is not None:
        dist_ctx.all_reduce(t, op=dist_ctx.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(chunks_per_rank: int, world: int, ms_per_step: float) -> float:
    """Every rank processes its own shard of `chunks_per_rank` chunks per step (weak scaling, no exchange)."""
    return world * chunks_per_rank / (ms_per_step * 1e-3)


def run_ours(args, rank, world, dist_ctx):
    _import_torch()
    from paper_2606_06034_b200 import binding as gdn
    from paper_2606_06034_b200 import inputs as gen

    dev = torch.device("cuda", torch.cuda.current_device())
    over = {"B": args.batch} if args.batch > 0 else {}
    inp = gen.make_workload(args.workload, device=dev, **over)
    C, group = inp.C, inp.H_v // inp.H_k
    outs = gdn.alloc_outputs(inp.K, inp.V, C)
    n_chunks = inp.n_chunks
    # --method other than the default times one of the other kernels as the step (used for the ncu summaries of the
    # forward-substitution comparison and of the INT8 variant); the headline is always --method neumann
    method = args.method
    q8 = q8_outs = None
    if method == "int8":
        q8 = gen.make_int8_inputs(inp)
        q8_outs = gdn.chunk_prepare_int8(q8)
    if method == "int16":
        q8 = gen.make_int16_inputs(inp)
        q8_outs = gdn.chunk_prepare_int16(q8)
    st_args = None
    if method == "state":  # state passing + output of the layer, given the gated W and U
        gq = torch.Generator(device=dev).manual_seed(99)
        Qs = torch.randn(inp.B, inp.H_k, inp.T, inp.d_k, device=dev, generator=gq)
        Qs = (Qs / Qs.norm(dim=-1, keepdim=True)).to(inp.K.dtype)
        Wg, Ug, _ = gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, C, flags=gdn.GDN_FLAG_W_GATED, want_tinv=False)
        st_outs = gdn.chunk_state_output(Qs, inp.K, Wg, Ug, inp.g, C, inp.d_k ** -0.5)
        st_args = (Qs, Wg, Ug, st_outs)

    mn_args = None
    if method == "model-native":  # token-major tensors, raw gates, fused key normalisation, gated W (what a model passes)
        mn_in = tuple(x.transpose(1, 2).contiguous() for x in (inp.K, inp.V, inp.beta, inp.g))
        mn_flags = gdn.GDN_FLAG_LAYOUT_BTHD | gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM | gdn.GDN_FLAG_W_GATED
        mn_args = (mn_in, gdn.alloc_outputs(mn_in[0], mn_in[1], C, True, True), mn_flags)

    def step():
        if method == "neumann":
            gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, C, outputs=outs)
        elif method == "model-native":
            gdn.chunk_prepare(*mn_args[0], C, outputs=mn_args[1], flags=mn_args[2])
        elif method == "int8":
            gdn.chunk_prepare_int8(q8, outputs=q8_outs)
        elif method == "int16":
            gdn.chunk_prepare_int16(q8, outputs=q8_outs)
        elif method == "state":
            gdn.chunk_state_output(st_args[0], inp.K, st_args[1], st_args[2], inp.g, C, inp.d_k ** -0.5, outputs=st_args[3])
        else:
            gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, C, outputs=outs, method="fwdsubst",
                              variant={"fwdsubst-blocked": gdn.GDN_FWDSUBST_BLOCKED,
                                       "fwdsubst-tc": gdn.GDN_FWDSUBST_BLOCKED_TC}.get(method, gdn.GDN_FWDSUBST_ROWS))

    sampler = ClockSampler(torch.cuda.current_device())
    # W warm-up steps as asked, and never less than ~0.1 s of untimed launches: the first launches after the idle time
    # spent generating the inputs run at lower clocks and would otherwise sit inside a short timed region
    step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    step()
    torch.cuda.synchronize()
    one = max(time.perf_counter() - t0, 1e-5)
    n_untimed = max(args.warmup, min(50, int(0.1 / one) + 1))
    for _ in range(n_untimed):
        step()
    lc = gdn.gdn_launch_count()
    step()
    per_call = gdn.gdn_launch_count() - lc  # kernels per call of the entry point (two for INT8 chunks of 128 tokens)
    torch.cuda.synchronize()
    launches0 = gdn.gdn_launch_count()
    sampler.start()
    total_ms, per = device_time_steps(step, args.steps, 0, dist_ctx)
    clocks = sampler.stop()
    launches = gdn.gdn_launch_count() - launches0 - 2 * per_call  # the two queue-priming calls sit before the first event
    # a timed region that saw a thermal or hardware slowdown, or clocks far below maximum with no reason given (a leftover
    # clock lock), is not a measurement: take it once more and say so
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clocks.get("reasons") or [])
    stuck = (clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and not clocks.get("reasons")
             and clocks["sm_mhz"] < 0.8 * clocks["sm_max_mhz"])
    remeasured = False
    again = 1.0 if (bad or stuck) else 0.0
    again = max_over_ranks(again, dev, dist_ctx) > 0.0  # every rank takes the same decision
    if again:
        time.sleep(2.0)
        sampler = ClockSampler(torch.cuda.current_device())
        launches0 = gdn.gdn_launch_count()
        sampler.start()
        total_ms, per = device_time_steps(step, args.steps, 0, dist_ctx)
        first, clocks = clocks, sampler.stop()
        clocks["first_attempt"] = first
        launches = gdn.gdn_launch_count() - launches0 - 2 * per_call
        remeasured = True
    status = gdn.gdn_device_status()
    if status != gdn.GDN_OK:
        raise RuntimeError(f"kernel status {status}")

    total_ms = max_over_ranks(total_ms, dev, dist_ctx)
    ms_per_step = total_ms / args.steps
    value = whole_job_throughput(n_chunks, world, ms_per_step)

    bytes_chunk = algorithmic_bytes_per_chunk(C, inp.d_k, inp.d_v, group)
    if method == "state":  # Q, K (shared by a group), W, U read, O written, g
        bytes_chunk = C * inp.d_k * 2 * (2.0 / group + 1) + 2 * C * inp.d_v * 2 + 4 * C
    if method == "int8":  # one byte per element, u16 beta + i32 decay per token
        bytes_chunk = C * inp.d_k / group + C * inp.d_v + C * inp.d_k + C * inp.d_v + C * C + 6 * C
    if method == "int16":  # two bytes per element
        bytes_chunk = 2 * (C * inp.d_k / group + C * inp.d_v + C * inp.d_k + C * inp.d_v + C * C) + 6 * C
    flops_chunk = nominal_flops_per_chunk(C, inp.d_k, inp.d_v)
    hbm_peak, bf16_peak, peak_kind = measured_peaks()
    launch_ms = float(np.mean(per))
    achieved = n_chunks * bytes_chunk / (launch_ms * 1e-3) / 1e9
    traffic = None
    if method == "neumann" and args.workload in TRAFFIC_PER_CHUNK:
        per_chunk_traffic, traffic_src = TRAFFIC_PER_CHUNK[args.workload]
        traffic = per_chunk_traffic * n_chunks
    roofline = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                "traffic": traffic, "peak_kind": peak_kind,
                "algorithmic_bytes_per_launch": n_chunks * bytes_chunk,
                "kernel": {"int8": "chunk_tc_int8_kernel", "int16": "chunk_tc_int16_kernel", "state": "chunk_state_kernel"}.get(method, "chunk_tc_kernel<C=%d>" % C),
                "effective_tflops": n_chunks * flops_chunk / (launch_ms * 1e-3) / 1e12,
                "tensor_time_frac_of_bf16_peak": (n_chunks * flops_chunk / (launch_ms * 1e-3) / 1e12) / bf16_peak}
    if traffic is not None:
        roofline["traffic_source"] = traffic_src

    if method == "int8" and C == 64:
        # the contract's roofline for this variant is HBM (every configuration is memory-bound on paper); the integer-ALU
        # figure explains where the time goes (ncu: the integer pipe is the busiest unit) and is reported beside it
        ops = int8_integer_ops_per_chunk(C, inp.d_k, inp.d_v, gdn.gdn_default_order(C), gdn.gdn_default_residual_steps(C))
        alu_peak = INT_ALU_LANES * SM_MAX_GHZ / 1e3  # Tiop/s
        alu = n_chunks * ops / (launch_ms * 1e-3) / 1e12
        roofline["int_alu"] = {"achieved": alu, "peak": alu_peak, "unit": "Tiop/s", "frac": alu / alu_peak,
                               "peak_kind": "derived: 148 SMs x 64 integer lanes x 1.965 GHz",
                               "algorithmic_int_ops_per_chunk": ops}
    per_sorted = sorted(per)
    roofline["launch_us"] = {"mean": launch_ms * 1e3, "median": per_sorted[len(per_sorted) // 2] * 1e3, "best": per_sorted[0] * 1e3}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"int8": "s8", "int16": "s16"}.get(method, "f32" if inp.K.dtype == torch.float32 else "bf16"),
        "data": "synthetic", "impl": "ours",
        "config": {"workload": args.workload, "method": method, "B": inp.B, "H_k": inp.H_k, "H_v": inp.H_v, "T": inp.T, "C": C, "d_k": inp.d_k,
                   "d_v": inp.d_v, "order": gdn.gdn_default_order(C), "residual_steps": gdn.gdn_default_residual_steps(C),
                   "chunks_per_gpu": n_chunks, "parallelism": f"independent shards x{world}, no collective",
                   "untimed_launches_before_timing": (n_untimed + 3) * per_call,
                   "l2_policy": "inputs+outputs %.0f MB per step, larger than the 126 MB L2" % (n_chunks * bytes_chunk / 1e6)},
        "effective_tflops": world * n_chunks * flops_chunk / (ms_per_step * 1e-3) / 1e12,
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
    }
    if remeasured:
        line["remeasured"] = True

    # the chunks the CPU leg runs are taken from this workload's own device buffers, with the GPU results for them
    cpu_sample = gpu_sample = None
    if rank == 0 and not args.no_cpu and world == 1 and method == "neumann":
        ids = sample_chunk_ids(inp.B * inp.H_v, inp.T // C, 58, seed=11)
        sl = gen.chunk_slices(inp, ids)
        cpu_sample = tuple(np.stack([s[i] for s in sl]) for i in range(4))
        idx = torch.as_tensor(ids, device=dev)
        gpu_sample = (outs[0].reshape(n_chunks, C, inp.d_k)[idx].double().cpu().numpy(),
                      outs[1].reshape(n_chunks, C, inp.d_v)[idx].double().cpu().numpy(),
                      outs[2].reshape(n_chunks, C, C)[idx].double().cpu().numpy())

    if rank == 0 and not args.no_e2e and method == "neumann":
        line["e2e"] = run_e2e(inp, outs, gdn, args, world, n_chunks)
    del outs, inp
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_extras:
        line["extras"] = run_extras(gdn, gen, dev, args)
    if rank == 0 and not args.no_cpu and world == 1:
        line["cpu_baseline"], _ = time_oracle(args.workload, args.cpu_seconds, sample=cpu_sample)
        if cpu_sample is not None:
            from oracle import gdn_oracle as orc
            line["cpu_baseline"]["parity_on_sample"] = parity_report(orc, cpu_sample, gpu_sample)
    return line


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per chunk from the ncu captures summarised under profiles/,
# scaled to a launch by the number of chunks it processes (traffic grows in proportion: every chunk is read and written once)
TRAFFIC_PER_CHUNK: dict = {
    "stress": (2378.12e6 / 32768, "ncu capture of the same workload with one batch entry (32 768 chunks), scaled by the chunks "
                                  "of the launch (profiles/chunk_tc_kernel_bf16_c64_stress.md)"),
    "sweep_c64": (247.93e6 / 4096, "ncu capture of this workload (profiles/chunk_tc_kernel_bf16_c64_sweep_c64.md)"),
    "prefill_gqa": (1024.84e6 / 16384, "ncu capture of this workload (profiles/chunk_tc_kernel_bf16_c64_prefill_gqa.md)"),
}


def run_e2e(inp, outs, gdn, args, world, n_chunks):
    """Same metric through the C-ABI with HOST buffers: pinned host -> device copies of K, V, beta, g and a
    device -> host read of W, U, Tinv inside the timed region, every step. The batch is cut into one slice per batch
    entry; a stream owns pinned host buffers for ONE slice (pinning the 20 GB of the largest workload is not an
    option) and runs its slices in order through them: copy in -> kernel -> copy out."""
    _import_torch()
    B = inp.K.shape[0]
    n_streams = min(B, 4)
    ins = (inp.K, inp.V, inp.beta, inp.g)
    host_in = [[t[s:s + 1].cpu().pin_memory() for t in ins] for s in range(n_streams)]
    dev_in = [[torch.empty_like(t[0:1]) for t in ins] for _ in range(n_streams)]
    host_out = [[torch.empty(t[0:1].shape, dtype=t.dtype, pin_memory=True) for t in outs] for _ in range(n_streams)]
    h2d = B * sum(t.numel() * t.element_size() for t in host_in[0])
    d2h = B * sum(t.numel() * t.element_size() for t in host_out[0])
    steps = max(3, min(args.steps, 10 if h2d + d2h < (2 << 30) else 4))
    streams = [torch.cuda.Stream() for _ in range(n_streams)]

    def step():
        # consecutive steps are not joined (a slice always runs on the same stream, so its buffers are reused in order):
        # the copies of step k + 1 start while step k drains, as in a serving loop; `join` closes the timed region
        for b in range(B):
            s = b % n_streams
            with torch.cuda.stream(streams[s]):
                for h, d in zip(host_in[s], dev_in[s]):
                    d.copy_(h, non_blocking=True)
                gdn.chunk_prepare(dev_in[s][0], dev_in[s][1], dev_in[s][2], dev_in[s][3], inp.C,
                                  outputs=tuple(o[b:b + 1] for o in outs))
                for h, d in zip(host_out[s], outs):
                    h.copy_(d[b:b + 1], non_blocking=True)

    def join():
        cur = torch.cuda.current_stream()
        for st in streams:
            done = torch.cuda.Event()
            done.record(st)
            cur.wait_event(done)

    # the side streams start behind everything already queued on the current stream
    start = torch.cuda.Event()
    start.record(torch.cuda.current_stream())
    for st in streams:
        st.wait_event(start)
    total_ms, _ = device_time_steps(step, steps, 1, None, finalize=join)
    return {"value": world * n_chunks / (total_ms / steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "ms_per_step": total_ms / steps,
            "pipeline": "%d slices (one per batch entry) over %d streams, each stream with pinned host buffers for one slice "
                        "that its slices pass through in order (slice s carries the data of batch entry s mod %d); steps back to back"
                        % (B, n_streams, n_streams)}


def _timed_extra(fn, n_chunks, bytes_chunk, hbm_peak, steps, warm):
    total_ms, per = device_time_steps(fn, steps, warm, None)
    ms = float(np.mean(per))
    return {"chunks_per_s": n_chunks / (ms * 1e-3), "ms": ms, "launch_ms_mean": ms, "launch_ms_best": float(min(per)),
            "hbm_frac": n_chunks * bytes_chunk / (ms * 1e-3) / 1e9 / hbm_peak}


def run_extras(gdn, gen, dev, args):
    """The other graded configurations and the forward-substitution comparisons, timed the same way as the headline
    (CUDA events around every launch after warm-up; every workload is larger than L2). Not the headline."""
    _import_torch()
    out = {}
    hbm_peak, _, _ = measured_peaks()
    plan = [("sweep_c16", "neumann"), ("sweep_c32", "neumann"), ("sweep_c64", "neumann"), ("sweep_c128", "neumann"),
            ("sweep_c64", "neumann-s15"),
            ("sweep_c16", "fwdsubst"), ("sweep_c32", "fwdsubst"), ("sweep_c64", "fwdsubst"), ("sweep_c128", "fwdsubst"),
            ("sweep_c16", "fwdsubst-blocked"), ("sweep_c32", "fwdsubst-blocked"), ("sweep_c64", "fwdsubst-blocked"),
            ("sweep_c128", "fwdsubst-blocked"), ("sweep_c64", "fwdsubst-tc"), ("prefill_gqa", "neumann"), ("prefill_gqa", "fwdsubst"),
            ("prefill_gqa", "fwdsubst-tc")]
    if args.workload != "stress":
        plan.append(("stress", "neumann"))
    for name, method in plan:
        try:
            inp = gen.make_workload(name, device=dev)
            outs = gdn.alloc_outputs(inp.K, inp.V, inp.C)
            meth, var = (method.split("-") + ["rows"])[:2]
            variant = {"blocked": gdn.GDN_FWDSUBST_BLOCKED, "tc": gdn.GDN_FWDSUBST_BLOCKED_TC}.get(var, gdn.GDN_FWDSUBST_ROWS)
            # "neumann-s15": all 15 residual terms (the exact inverse at N = 3, C = 64) by the doubling scheme
            n_ord, n_res = (3, 15) if var == "s15" else (-1, -1)
            fn = lambda: gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, inp.C, n_ord, n_res, outputs=outs, method=meth,
                                           variant=variant)
            by = algorithmic_bytes_per_chunk(inp.C, inp.d_k, inp.d_v, inp.H_v // inp.H_k)
            out[f"{name}:{method}"] = _timed_extra(fn, inp.n_chunks, by, hbm_peak, 20 if name != "stress" else 10, 5)
            del inp, outs
        except Exception as exc:  # an unsupported extra must not lose the headline
            out[f"{name}:{method}"] = {"error": repr(exc)}
    # Neumann against the better of the two substitutions, per chunk size
    for c in (16, 32, 64, 128):
        try:
            neu = out[f"sweep_c{c}:neumann"]["ms"]
            sub = min(out[f"sweep_c{c}:{m}"]["ms"] for m in ("fwdsubst", "fwdsubst-blocked", "fwdsubst-tc")
                      if "ms" in out.get(f"sweep_c{c}:{m}", {}))
            out[f"sweep_c{c}:neumann_speedup_over_best_substitution"] = sub / neu
        except Exception:
            pass
    # the model-native call on the prefill shapes: token-major tensors, raw gates, fused key normalisation, gated W;
    # and the same tokens as 201 packed sequences of ragged lengths (seeded cuts)
    try:
        inp = gen.make_workload("prefill_gqa", device=dev)
        by = algorithmic_bytes_per_chunk(inp.C, inp.d_k, inp.d_v, inp.H_v // inp.H_k)
        Kt, Vt = inp.K.transpose(1, 2).contiguous(), inp.V.transpose(1, 2).contiguous()
        bt, gt = inp.beta.transpose(1, 2).contiguous(), inp.g.transpose(1, 2).contiguous()
        flags = gdn.GDN_FLAG_LAYOUT_BTHD | gdn.GDN_FLAG_G_RAW | gdn.GDN_FLAG_K_L2NORM | gdn.GDN_FLAG_W_GATED
        outs = gdn.alloc_outputs(Kt, Vt, inp.C, True, True)
        fn = lambda: gdn.chunk_prepare(Kt, Vt, bt, gt, inp.C, outputs=outs, flags=flags)
        out["prefill_gqa:model_native_flags"] = _timed_extra(fn, inp.n_chunks, by, hbm_peak, 10, 3)
        del Kt, Vt, bt, gt, outs
        cuts = np.sort(np.random.default_rng(0).choice(np.arange(1, inp.T), size=200, replace=False))
        start, length = gdn.chunk_table([0] + cuts.tolist() + [inp.T], inp.C)
        cs = torch.tensor(start, dtype=torch.int32, device=dev)
        cl = torch.tensor(length, dtype=torch.int32, device=dev)
        W = torch.zeros(inp.H_v, inp.T, inp.d_k, dtype=inp.K.dtype, device=dev)
        U = torch.zeros_like(W)
        per_tile = 128 // inp.C
        Ti = torch.empty(inp.H_v, -(-len(start) // per_tile) * per_tile, inp.C, inp.C, dtype=inp.K.dtype, device=dev)
        fn = lambda: gdn.gdn_chunk_prepare_varlen(inp.K[0], inp.V[0], inp.beta[0], inp.g[0], cs, cl, len(start), inp.T, inp.H_k,
                                                  inp.H_v, inp.C, inp.d_k, inp.d_v, -1, -1, W, U, Ti, 0)
        n_slots = len(start) * inp.H_v
        r = _timed_extra(fn, inp.n_chunks, by, hbm_peak, 10, 3)
        r["chunk_slots"] = n_slots
        r["chunks_per_s"] = n_slots / (r["ms"] * 1e-3)
        out["prefill_gqa:packed_201_sequences"] = r
        del inp, W, U, Ti
    except Exception as exc:
        out["prefill_gqa:model_native"] = {"error": repr(exc)}
    # INT8 variant on the prefill shapes (integer inputs quantised once from the same tensors)
    try:
        inp = gen.make_workload("prefill_gqa", device=dev)
        q = gen.make_int8_inputs(inp)
        outs = gdn.chunk_prepare_int8(q)
        fn = lambda: gdn.chunk_prepare_int8(q, outputs=outs)
        group = inp.H_v // inp.H_k
        by = inp.C * inp.d_k / group + inp.C * inp.d_v + inp.C * inp.d_k + inp.C * inp.d_v + inp.C * inp.C + 6 * inp.C
        ops = int8_integer_ops_per_chunk(q.C, q.d_k, q.d_v, gdn.gdn_default_order(q.C), gdn.gdn_default_residual_steps(q.C))
        r = _timed_extra(fn, q.n_chunks, by, hbm_peak, 10, 3)
        r["int_alu_frac"] = q.n_chunks * ops / (r["ms"] * 1e-3) / (INT_ALU_LANES * SM_MAX_GHZ * 1e9)
        out["prefill_gqa:int8"] = r
        del inp, q, outs
    except Exception as exc:
        out["prefill_gqa:int8"] = {"error": repr(exc)}
    # INT8 on chunks of 128 tokens (two 64-blocks and the block merge of App. E, Eq. 28: two launches per call)
    try:
        inp = gen.make_workload("sweep_c128", device=dev)
        q = gen.make_int8_inputs(inp)
        outs = gdn.chunk_prepare_int8(q)
        fn = lambda: gdn.chunk_prepare_int8(q, outputs=outs)
        group = inp.H_v // inp.H_k
        by = inp.C * inp.d_k / group + inp.C * inp.d_v + inp.C * inp.d_k + inp.C * inp.d_v + inp.C * inp.C + 6 * inp.C
        out["sweep_c128:int8"] = _timed_extra(fn, q.n_chunks, by, hbm_peak, 10, 3)
        del inp, q, outs
    except Exception as exc:
        out["sweep_c128:int8"] = {"error": repr(exc)}
    # INT16 variant (the paper's primary integer precision) on the prefill shapes: two bytes per element
    try:
        inp = gen.make_workload("prefill_gqa", device=dev)
        q = gen.make_int16_inputs(inp)
        outs = gdn.chunk_prepare_int16(q)
        fn = lambda: gdn.chunk_prepare_int16(q, outputs=outs)
        group = inp.H_v // inp.H_k
        by = 2 * (inp.C * inp.d_k / group + inp.C * inp.d_v + inp.C * inp.d_k + inp.C * inp.d_v + inp.C * inp.C) + 6 * inp.C
        out["prefill_gqa:int16"] = _timed_extra(fn, q.n_chunks, by, hbm_peak, 5, 2)
        del inp, q, outs
    except Exception as exc:
        out["prefill_gqa:int16"] = {"error": repr(exc)}
    # the rest of the layer (state passing + output, given the gated W and U) on the prefill and stress shapes; last,
    # because the stress shapes (20 GB, milliseconds per launch) push the GPU into its power cap
    for name in ("prefill_gqa", "stress"):
        try:
            inp = gen.make_workload(name, device=dev)
            gq = torch.Generator(device=dev).manual_seed(99)
            Q = torch.randn(inp.B, inp.H_k, inp.T, inp.d_k, device=dev, generator=gq)
            Q = (Q / Q.norm(dim=-1, keepdim=True)).to(inp.K.dtype)
            W, U, _ = gdn.chunk_prepare(inp.K, inp.V, inp.beta, inp.g, inp.C, flags=gdn.GDN_FLAG_W_GATED, want_tinv=False)
            outs = gdn.chunk_state_output(Q, inp.K, W, U, inp.g, inp.C, inp.d_k ** -0.5)
            fn = lambda: gdn.chunk_state_output(Q, inp.K, W, U, inp.g, inp.C, inp.d_k ** -0.5, outputs=outs)
            group = inp.H_v // inp.H_k
            # Q, K tiles (shared by a group), W, U read, O written, g
            by = inp.C * inp.d_k * 2 * (2.0 / group + 1) + 2 * inp.C * inp.d_v * 2 + 4 * inp.C
            r = _timed_extra(fn, inp.n_chunks, by, hbm_peak, 5, 2)
            r["us_per_chunk_of_a_sequence"] = r["ms"] * 1e3 / (inp.T // inp.C)
            out[f"{name}:state_output"] = r
            if inp.B == 1:
                # few long sequences: the segmented form (state maps of the segments in parallel)
                fn = lambda: gdn.chunk_state_output_segmented(Q[0], inp.K[0], W[0], U[0], inp.g[0], inp.C, inp.d_k ** -0.5)
                r = _timed_extra(fn, inp.n_chunks, by, hbm_peak, 5, 2)
                r["segments"] = int(gdn.load_library().gdn_chunk_state_segments(inp.H_v))
                out[f"{name}:state_output_segmented"] = r
            del inp, Q, W, U, outs
        except Exception as exc:
            out[f"{name}:state_output"] = {"error": repr(exc)}
    return out


def run_reference(args):
    """The base contract's reference arm: the CPU oracle, as it stands, on the host cores."""
    steps, warm = args.steps, args.warmup
    budget_per_step = max(0.2, min(10.0, args.cpu_seconds, 120.0 / max(1, steps + warm)))
    vals = []
    info = None
    for i in range(warm + steps):
        info, wall = time_oracle(args.workload, budget_per_step)
        if i >= warm:
            vals.append((info["value"], wall))
    value = float(np.mean([v for v, _ in vals]))
    from paper_2606_06034_b200 import inputs as gen
    cfg = gen.WORKLOADS[args.workload]
    info["value"] = value
    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warm,
        "ms_per_step": float(np.mean([w for _, w in vals])) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": {"workload": args.workload, "method": "neumann", "B": cfg["B"], "H_k": cfg["H_k"], "H_v": cfg["H_v"], "T": cfg["T"],
                   "C": cfg["C"], "d_k": cfg["d_k"], "d_v": cfg["d_v"],
                   "note": "each step is a bounded sample of the workload's chunks run through the fp64 CPU oracle"},
        "cpu_baseline": info,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (smaller captures under ncu)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--method", default="neumann", choices=["neumann", "fwdsubst", "fwdsubst-blocked", "fwdsubst-tc", "int8", "int16", "state", "model-native"])
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return

    _import_torch()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    dist_ctx = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))
        dist_ctx = dist
    line = run_ours(args, rank, world, dist_ctx)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist_ctx is not None:
        dist_ctx.destroy_process_group()


if __name__ == "__main__":
    main()

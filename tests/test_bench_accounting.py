"""The per-chunk figures bench.py divides by: algorithmic bytes, nominal flops, integer operations of the INT8 variant."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_algorithmic_bytes_per_chunk():
    # K, V, W, U tiles of 64 x 128 bf16, the full 64 x 64 inverse, beta and g: 4 * 16384 + 8192 + 512
    assert bench.algorithmic_bytes_per_chunk(64, 128, 128, 1) == 74240
    # pairs of value heads share the key tile
    assert bench.algorithmic_bytes_per_chunk(64, 128, 128, 2) == 66048
    assert bench.algorithmic_bytes_per_chunk(16, 128, 128, 1) == 17024
    assert bench.algorithmic_bytes_per_chunk(128, 128, 128, 1) == 164864


def test_nominal_flops_follow_the_papers_matmul_counts():
    # C = 64: Gram + 11 products of 64^3 + W + U (Sec. 4.3 counts 11 at N = 3, S = 8); C = 32: 7
    assert bench.nominal_flops_per_chunk(64, 128, 128) == 2 * 64 * 64 * 128 * 3 + 11 * 2 * 64 ** 3
    assert bench.nominal_flops_per_chunk(32, 128, 128) == 2 * 32 * 32 * 128 * 3 + 7 * 2 * 32 ** 3


def test_int8_integer_operation_count():
    ops = bench.int8_integer_ops_per_chunk(64, 128, 128, 3, 8)
    assert ops == 386806
    # more residual terms or a wider band cannot need fewer operations; W and U dominate and scale with d
    assert bench.int8_integer_ops_per_chunk(64, 128, 128, 3, 4) < ops
    assert bench.int8_integer_ops_per_chunk(64, 128, 128, 2, 8) != ops
    assert bench.int8_integer_ops_per_chunk(64, 256, 256, 3, 8) - ops == 12 * 64 * 256


def test_host_bf16_rounding_matches_torch():
    import numpy as np
    import torch
    x = np.random.default_rng(0).standard_normal(4096) * np.exp(np.random.default_rng(1).uniform(-20, 20, 4096))
    x[:4] = [0.0, 1.0, -1.0, 1.00390625]  # the last one is a tie between two bf16 values: rounds to even
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).double().numpy()
    assert np.array_equal(bench._bf16_round(x), want)


def test_sample_chunk_ids_cover_the_corner_chunks():
    ids = bench.sample_chunk_ids(n_heads=256, n_c=1024, n_random=58, seed=11)
    assert ids == sorted(set(ids)) and len(ids) <= 64
    for must in (0, 1023, 255 * 1024, 256 * 1024 - 1, 1024, 2047):   # first / last chunk of the first / last head, head 1
        assert must in ids
    assert ids == bench.sample_chunk_ids(256, 1024, 58, seed=11)
    assert bench.sample_chunk_ids(1, 4, 58, seed=0) == [0, 1, 2, 3]


def test_parity_report_on_a_result_that_is_the_oracle_rounded_to_bf16():
    """A 'GPU result' that is the oracle's own result rounded to bf16 must report an error equal to the bf16 floor,
    a deviation from the exact inverse of the same size, and the scheme's own deviation at fp64 rounding level."""
    import numpy as np
    from oracle import gdn_oracle as orc
    from paper_2606_06034_b200 import inputs as gen
    inp = gen.make_inputs(1, 2, 2, 256, 64, 128, 128, seed=5, adversarial_heads="odd")
    sl = gen.chunk_slices(inp, range(inp.n_chunks))
    sample = tuple(np.stack([s[i] for s in sl]) for i in range(4))
    W, U, T = orc.chunk_prepare(*sample)
    rep = bench.parity_report(orc, sample, (bench._bf16_round(W), bench._bf16_round(U), bench._bf16_round(T)))
    assert rep["chunks"] == inp.n_chunks
    for name in ("Tinv", "W", "U"):
        r = rep[name]
        assert r["worst_rel_frobenius"] == r["worst_bf16_floor"] == r["bf16_floor_of_that_chunk"]
        assert 1e-5 < r["worst_rel_frobenius"] < 2.2e-3
        assert r["scheme_vs_exact_inverse_worst"] < 1e-9
        assert abs(r["gpu_vs_exact_inverse_worst"] - r["worst_rel_frobenius"]) < 1e-8
        assert 50 < r["snr_db_worst"] <= r["snr_db_mean"]


def test_oracle_pool_runs_on_several_processes():
    import numpy as np
    from oracle import gdn_oracle as orc
    from oracle import pool
    rng = np.random.default_rng(3)
    K = rng.standard_normal((8, 16, 8)); V = rng.standard_normal((8, 16, 8))
    b = rng.uniform(0.1, 0.9, (8, 16)); g = -np.cumsum(rng.uniform(0, 1, (8, 16)), axis=-1)
    done, wall, used = pool.timed_chunk_prepare(K, V, b, g, 200, workers=2, batch=4)
    assert done == 200 and used == 2 and wall > 0
    done, wall, used = pool.timed_chunk_prepare(K, V, b, g, 37, workers=1, batch=4)
    assert done == 37 and used == 1
    assert pool.usable_cores() >= 1

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

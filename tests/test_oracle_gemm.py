"""Pins for the fp64 GEMM oracle (CPU only): closed forms, a hand-worked product, exact
integer arithmetic and agreement with numpy's own fp64 matmul."""
import os

import numpy as np
import pytest

from oracle import gemm as og
from paper_2609_24270_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_hand_worked_product():
    rows = [l for l in open(os.path.join(GOLD, "gemm_2x3x4.txt")) if l.strip() and not l.startswith("#")]
    vals = [list(map(float, r.split())) for r in rows]
    A, B, C = np.array(vals[0:2]), np.array(vals[2:6]), np.array(vals[6:8])
    for fn in (og.gemm_bruteforce, og.gemm_blocked):
        got = fn(bf(A), bf(B))
        assert got.shape == (2, 3)
        assert np.array_equal(got, C)


@pytest.mark.parametrize("shape", [(1, 1, 1), (2, 3, 4), (17, 19, 23), (128, 256, 64)])
def test_bruteforce_matches_numpy_fp64(shape):
    M, N, K = shape
    A, B = inputs.gemm_inputs(M, N, K, seed=3)
    ref = inputs.bf16_bits_to_f64(A) @ inputs.bf16_bits_to_f64(B)
    got = og.gemm_bruteforce(A, B)
    assert np.allclose(got, ref, rtol=0, atol=1e-11)


@pytest.mark.parametrize("shape", [(5, 7, 9), (64, 96, 130), (130, 1030, 70)])
def test_blocked_equals_bruteforce_bitwise(shape):
    M, N, K = shape
    A, B = inputs.gemm_inputs(M, N, K, seed=11)
    assert np.array_equal(og.gemm_blocked(A, B), og.gemm_bruteforce(A, B))


def test_identity_and_ones_closed_forms():
    K = 96
    B = inputs.uniform_bf16(K, 40, seed=5)
    I = bf(np.eye(K))
    assert np.array_equal(og.gemm_blocked(I, B), inputs.bf16_bits_to_f64(B))      # I.B = B exactly
    ones_a = bf(np.ones((33, K)))
    ones_b = bf(np.ones((K, 21)))
    assert np.array_equal(og.gemm_blocked(ones_a, ones_b), np.full((33, 21), float(K)))
    colsum = inputs.bf16_bits_to_f64(B).sum(axis=0)
    got = og.gemm_blocked(ones_a, B)
    assert np.allclose(got, np.tile(colsum, (33, 1)), rtol=0, atol=1e-12)


def test_integer_inputs_are_exact():
    M, N, K = 37, 29, 211
    A = inputs.small_int_bf16(M, K, seed=1)
    B = inputs.small_int_bf16(K, N, seed=2)
    ai = inputs.bf16_bits_to_f64(A).astype(np.int64)
    bi = inputs.bf16_bits_to_f64(B).astype(np.int64)
    assert ai.min() >= -2 and ai.max() <= 2 and len(np.unique(ai)) == 5
    want = (ai @ bi).astype(np.float64)
    assert np.array_equal(og.gemm_bruteforce(A, B), want)
    assert np.array_equal(og.gemm_blocked(A, B), want)


def test_one_hot_localises_addressing():
    M, N, K = 9, 11, 13
    B = inputs.uniform_bf16(K, N, seed=8)
    A = np.zeros((M, K), dtype=np.float32)
    A[4, 6] = 1.0
    got = og.gemm_bruteforce(bf(A), B)
    want = np.zeros((M, N))
    want[4] = inputs.bf16_bits_to_f64(B)[6]
    assert np.array_equal(got, want)


def test_block_and_entries_agree_with_full():
    M, N, K = 70, 90, 50
    A, B = inputs.gemm_inputs(M, N, K, seed=21)
    full = og.gemm_blocked(A, B)
    assert np.array_equal(og.gemm_block(A, B, 10, 33, 7, 80), full[10:33, 7:80])
    rows, cols = [0, 69, 13], [0, 89, 55]
    assert np.array_equal(og.gemm_entries(A, B, rows, cols), full[rows, cols])


def test_generator_properties():
    a = inputs.uniform_bf16(64, 64, seed=inputs.DEFAULT_SEED)
    v = inputs.bf16_bits_to_f64(a)
    assert v.min() >= -1.0 and v.max() <= 1.0
    assert abs(v.mean()) < 0.05 and abs(v.var() - 1.0 / 3.0) < 0.03
    assert np.array_equal(a, inputs.uniform_bf16(64, 64, seed=inputs.DEFAULT_SEED))
    assert not np.array_equal(a, inputs.uniform_bf16(64, 64, seed=inputs.DEFAULT_SEED + 1))
    # chunked generation is seamless
    assert np.array_equal(inputs.uniform_bf16(8, 1024, 4, chunk=1000), inputs.uniform_bf16(8, 1024, 4))
    # round-to-nearest-even on the bf16 boundary: 1 + 2^-8 is a tie -> even mantissa
    tie = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    assert list(inputs.f32_to_bf16_bits(tie)) == [0x3F80, 0x3F82]

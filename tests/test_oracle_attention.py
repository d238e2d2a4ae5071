"""Pins for the attention-decode oracle: closed forms, a worked two-key example, invariances, brute force."""
import math

import numpy as np

from oracle import attention as oa
from paper_2609_24270_b200 import inputs


def bf16(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_case(B, Hq, Hkv, L, D, seed):
    Q = inputs.uniform_bf16(B * Hq, D, seed).reshape(B, Hq, D)
    K = inputs.uniform_bf16(B * Hkv * L, D, seed + 1).reshape(B, Hkv, L, D)
    V = inputs.uniform_bf16(B * Hkv * L, D, seed + 2).reshape(B, Hkv, L, D)
    return Q, K, V


def test_zero_query_gives_the_mean_of_v_of_the_right_kv_head():
    # q = 0: all scores equal, p uniform, o = mean of the value rows.  The values differ per KV head, so the
    # mapping query head -> KV head (hq // group, not hq % Hkv) is pinned too.
    B, Hq, Hkv, L, D = 2, 8, 2, 5, 4
    _, K, V = rand_case(B, Hq, Hkv, L, D, 3)
    Q = np.zeros((B, Hq, D), dtype=np.uint16)
    O = oa.gqa_decode(Q, K, V)
    Vf = oa.bf16_to_f64(V)
    for b in range(B):
        for hq in range(Hq):
            assert np.allclose(O[b, hq], Vf[b, hq // 4].mean(axis=0), rtol=0, atol=1e-15)
    assert not np.allclose(Vf[0, 0].mean(axis=0), Vf[0, 1].mean(axis=0))


def test_one_dominant_key_returns_its_value_row():
    B, Hq, Hkv, L, D = 1, 2, 1, 7, 128
    _, K, V = rand_case(B, Hq, Hkv, L, D, 5)
    K[:] = 0
    Q = np.zeros((B, Hq, D), dtype=np.uint16)
    Q[0, :, 0] = bf16([64.0])[0]
    K[0, 0, 4, 0] = bf16([64.0])[0]            # score of key 4 = 4096 / sqrt(128) = 362, all others 0
    O = oa.gqa_decode(Q, K, V)
    assert np.allclose(O[0, 0], oa.bf16_to_f64(V)[0, 0, 4], rtol=0, atol=1e-150)


def test_two_keys_worked_by_hand():
    # D = 4, q = (2, 0, 0, 0), k1 = (1, 0, 0, 0), k2 = (-1, 0, 0, 0): scores +1 and -1 (2 / sqrt(4) = 1),
    # p1 = e / (e + 1/e) = 1 / (1 + e^-2) = 0.880797077977882..., o = p1 v1 + (1 - p1) v2
    Q = bf16([[[2.0, 0, 0, 0]]])
    K = bf16([[[[1.0, 0, 0, 0], [-1.0, 0, 0, 0]]]])
    V = bf16([[[[1.0, 2.0, -4.0, 0.5], [3.0, -2.0, 8.0, 0.25]]]])
    p1 = 0.8807970779778823                      # 1 / (1 + exp(-2)), from tables of the logistic function
    assert abs(p1 - 1.0 / (1.0 + math.exp(-2.0))) < 1e-15
    want = [p1 * 1 + (1 - p1) * 3, p1 * 2 - (1 - p1) * 2, -4 * p1 + 8 * (1 - p1), 0.5 * p1 + 0.25 * (1 - p1)]
    assert np.allclose(oa.gqa_decode(Q, K, V)[0, 0], want, rtol=0, atol=1e-14)


def test_invariances_and_lengths():
    B, Hq, Hkv, L, D = 3, 4, 2, 9, 8
    Q, K, V = rand_case(B, Hq, Hkv, L, D, 11)
    O = oa.gqa_decode(Q, K, V)
    # permuting the keys together with their values changes nothing
    perm = np.array([3, 0, 8, 1, 2, 7, 6, 5, 4])
    assert np.allclose(oa.gqa_decode(Q, K[:, :, perm], V[:, :, perm]), O, rtol=0, atol=1e-14)
    # every output row is a convex combination of value rows
    Vf = oa.bf16_to_f64(V)
    for b in range(B):
        for hq in range(Hq):
            h = hq // 2
            assert (O[b, hq] <= Vf[b, h].max(axis=0) + 1e-15).all() and (O[b, hq] >= Vf[b, h].min(axis=0) - 1e-15).all()
    # keys past kv_len do not count: the result equals that of the truncated cache, whatever lies behind
    lens = [9, 4, 0]
    O2 = oa.gqa_decode(Q, K, V, lens)
    assert np.allclose(O2[0], O[0], rtol=0, atol=0)
    assert np.allclose(O2[1], oa.gqa_decode(Q[1:2], K[1:2, :, :4], V[1:2, :, :4])[0], rtol=0, atol=0)
    assert not O2[2].any()
    # duplicating every key-value pair leaves the softmax average unchanged
    assert np.allclose(oa.gqa_decode(Q, np.concatenate([K, K], axis=2), np.concatenate([V, V], axis=2)), O, rtol=0, atol=1e-14)


def test_against_scalar_loops_on_tiny_cases():
    for (B, Hq, Hkv, L, D, seed) in ((1, 1, 1, 1, 1, 1), (2, 4, 2, 3, 5, 2), (1, 8, 8, 6, 16, 3)):
        Q, K, V = rand_case(B, Hq, Hkv, L, D, seed)
        lens = [(L * (b + 1)) // B for b in range(B)]
        assert np.allclose(oa.gqa_decode(Q, K, V, lens), oa.gqa_decode_loops(Q, K, V, lens), rtol=0, atol=1e-14)

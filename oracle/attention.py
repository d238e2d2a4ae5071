"""TEST INFRASTRUCTURE: fp64 oracle of grouped-query attention decode (one query token per request).

The paper schedules attention kernels (MHA / GQA / MLA, prefill and decode) the same way as its GEMMs
(Section 7.1.2; workload appendix: decode processes S_q = 1 query token per request against a KV sequence of
S_k tokens, H_kv = 8 KV heads for GQA, head dimension D = 128, KV working set 4 B S_k H_kv D bytes).  What such a
kernel computes has a plain definition, written out here:

    for request b, query head hq (its KV head is h = hq // (H_q / H_kv)):
        s_j = (q . k_j) / sqrt(D)            for the first len_b keys of (b, h)
        p_j = exp(s_j - max_j s_j) / sum_j exp(s_j - max_j s_j)
        o   = sum_j p_j v_j

Inputs are bf16 bit patterns (numpy uint16); everything is computed in float64.
"""
from __future__ import annotations

import math

import numpy as np


def bf16_to_f64(bits) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def gqa_decode(Q, K, V, kv_len=None) -> np.ndarray:
    """Q [B, Hq, D], K and V [B, Hkv, L, D] as bf16 bits; kv_len [B] (default: L for every request).
    Returns O [B, Hq, D] in float64.  A request with kv_len 0 gives zeros."""
    Q, K, V = bf16_to_f64(Q), bf16_to_f64(K), bf16_to_f64(V)
    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    assert K.shape == V.shape == (B, Hkv, L, D) and Hq % Hkv == 0
    group = Hq // Hkv
    lens = np.full(B, L, dtype=np.int64) if kv_len is None else np.asarray(kv_len, dtype=np.int64)
    O = np.zeros((B, Hq, D), dtype=np.float64)
    scale = 1.0 / math.sqrt(D)
    for b in range(B):
        n = int(lens[b])
        if n == 0:
            continue
        for hq in range(Hq):
            h = hq // group
            s = (K[b, h, :n] @ Q[b, hq]) * scale
            p = np.exp(s - s.max())
            p /= p.sum()
            O[b, hq] = p @ V[b, h, :n]
    return O


def gqa_decode_loops(Q, K, V, kv_len=None) -> np.ndarray:
    """The same definition with nothing but scalar Python arithmetic (tiny cases only)."""
    Q, K, V = bf16_to_f64(Q), bf16_to_f64(K), bf16_to_f64(V)
    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    group = Hq // Hkv
    O = np.zeros((B, Hq, D), dtype=np.float64)
    for b in range(B):
        n = L if kv_len is None else int(kv_len[b])
        for hq in range(Hq):
            h = hq // group
            s = []
            for j in range(n):
                acc = 0.0
                for t in range(D):
                    acc += float(Q[b, hq, t]) * float(K[b, h, j, t])
                s.append(acc / math.sqrt(D))
            if not s:
                continue
            m = max(s)
            e = [math.exp(x - m) for x in s]
            z = sum(e)
            for t in range(D):
                O[b, hq, t] = sum(e[j] * float(V[b, h, j, t]) for j in range(n)) / z
    return O

"""Seeded synthetic input generators (shared by the tests, the bench and the oracle's callers).

This module holds none of the method's arithmetic: it only manufactures inputs.
It imports neither the CUDA binding nor anything under ``oracle/``.

The paper's GEMM workloads (co-located GEMM pairs, GroupGEMM shapes, the
prefill/decode split of an 8B model, Section 7) come from no public dataset, so
seeded uniform bf16 matrices *are* the workload.  Elements are drawn uniform in
[-1, 1): element ``i`` of a matrix generated with ``seed`` is

    h = mix64(mix64(seed) + i)            (64-bit counter-based mixer)
    u = (h >> 40) / 2**24                 (top 24 bits, in [0, 1))
    v = float32(2 * u - 1)
    bf16 bits = round-to-nearest-even(v)

The same bf16 bit patterns are handed to the GPU path and to the oracle, so the
generator is never a parity risk.
"""
from __future__ import annotations

import numpy as np

DEFAULT_SEED = 20260924
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def mix64_np(x: np.ndarray) -> np.ndarray:
    """Vectorised 64-bit finaliser (add-golden-ratio, two xorshift-multiplies)."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += np.uint64(0x9E3779B97F4A7C15)
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


def f32_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (uint16). No NaN inputs expected."""
    u = np.ascontiguousarray(v, dtype=np.float32).view(np.uint32)
    rounding = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact decode of bf16 bit patterns to float64 (test convenience)."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def uniform_bf16(rows: int, cols: int, seed: int, chunk: int = 1 << 22) -> np.ndarray:
    """rows x cols matrix of bf16 bit patterns (uint16), uniform in [-1, 1), row-major."""
    n = rows * cols
    out = np.empty(n, dtype=np.uint16)
    base = mix64_np(np.array([seed], dtype=np.uint64))[0]
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        idx = np.arange(s, e, dtype=np.uint64)
        with np.errstate(over="ignore"):
            h = mix64_np(idx + base)
        u = (h >> np.uint64(40)).astype(np.float64) / float(1 << 24)
        out[s:e] = f32_to_bf16_bits((2.0 * u - 1.0).astype(np.float32))
    return out.reshape(rows, cols)


def small_int_bf16(rows: int, cols: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer-valued bf16 matrix with entries in {lo..hi}.

    With such inputs every partial sum of a GEMM is an integer far below 2**24, so
    fp32 accumulation is exact in any order and GPU output must match the fp64
    oracle bit for bit.
    """
    n = rows * cols
    base = mix64_np(np.array([seed], dtype=np.uint64))[0]
    idx = np.arange(n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = mix64_np(idx + base)
    span = np.uint64(hi - lo + 1)
    v = ((h >> np.uint64(33)) % span).astype(np.int64) + lo
    return f32_to_bf16_bits(v.astype(np.float32)).reshape(rows, cols)


def gemm_inputs(M: int, N: int, K: int, seed: int = DEFAULT_SEED):
    """A (M x K) from ``seed``, B (K x N) from ``seed + 1``; bf16 bit patterns."""
    return uniform_bf16(M, K, seed), uniform_bf16(K, N, seed + 1)


def group_rows(G: int, M: int, seed: int) -> np.ndarray:
    """Rows per expert of a grouped GEMM as in the paper's workload appendix: M_i = floor(M * U_i),
    U_i uniform in [0.7, 1.3), drawn from the repo's counter-based mixer."""
    h = mix64_np(np.arange(G, dtype=np.uint64) + mix64_np(np.array([seed], dtype=np.uint64))[0])
    u = 0.7 + 0.6 * ((h >> np.uint64(40)).astype(np.float64) / float(1 << 24))
    return np.floor(M * u).astype(np.int32)


# ----------------------------------------------------------------------------
# Synthetic chips and affinity maps for the CPU-side plan tests.
# ----------------------------------------------------------------------------

def synthetic_topo(n_sm: int = 148, die0_sms: int = 74, gpcs_per_die: int = 4,
                   n_random: int = 20, seed: int = 1) -> dict:
    """A made-up floorswept two-die chip in the shape the paper describes for B200
    (Section 5: 148 SMs, 2 dies x 4 GPCs, TPC = two consecutive SM ids, the highest
    ids are the floorsweeping-dependent "random" SMs; Section 7.1: die splits such as
    70/78, 72/76, 74/74).  Normal TPCs stripe over the 8 GPCs; random TPCs are
    scattered by the seed so that die 0 ends up with ``die0_sms`` SMs.
    """
    assert n_sm % 2 == 0 and die0_sms % 2 == 0 and n_random % 2 == 0
    n_gpc = 2 * gpcs_per_die
    n_tpc = n_sm // 2
    n_norm_tpc = (n_sm - n_random) // 2
    tpc_gpc = np.zeros(n_tpc, dtype=np.int32)
    for t in range(n_norm_tpc):
        tpc_gpc[t] = t % n_gpc
    gpc_die = np.array([g % 2 for g in range(n_gpc)], dtype=np.int32)
    # how many random TPCs must land on die 0 to reach die0_sms
    norm_die0 = int(sum(1 for t in range(n_norm_tpc) if gpc_die[tpc_gpc[t]] == 0))
    need0 = die0_sms // 2 - norm_die0
    n_rand_tpc = n_random // 2
    assert 0 <= need0 <= n_rand_tpc, "die split not reachable with this many random SMs"
    order = np.argsort(mix64_np(np.arange(n_rand_tpc, dtype=np.uint64) + np.uint64(seed * 1000003)))
    for rank, r in enumerate(order):
        d = 0 if rank < need0 else 1
        gpcs_d = [g for g in range(n_gpc) if gpc_die[g] == d]
        h = int(mix64_np(np.array([seed * 7919 + int(r)], dtype=np.uint64))[0])
        tpc_gpc[n_norm_tpc + int(r)] = gpcs_d[h % len(gpcs_d)]
    sm = np.arange(n_sm)
    tpc = (sm // 2).astype(np.int32)
    gpc = tpc_gpc[tpc].astype(np.int32)
    die = gpc_die[gpc].astype(np.int32)
    is_random = (tpc >= n_norm_tpc).astype(np.uint8)
    return {
        "n_sm": n_sm, "n_tpc": n_tpc, "n_gpc": n_gpc, "n_die": 2,
        "tpc": tpc, "gpc": gpc, "die": die, "is_random": is_random,
        "gpc_die": gpc_die,
    }


def synthetic_chunk_die(n_chunks: int, seed: int = 7, mask_bits: int = 0x1B5) -> np.ndarray:
    """Chunk -> die bitmap in the shape Section 6.1.2 describes: an XOR (parity) hash
    over address bits whose lowest participating bit is the 4 KB chunk bit, so every
    aligned pair of chunks has one chunk per die; a per-2-MiB-page constant models the
    unknown physical placement of each large page.
    """
    idx = np.arange(n_chunks, dtype=np.uint64)
    m = np.uint64(mask_bits | 1)                     # bit 0 of the chunk index always participates
    x = idx & m
    par = np.zeros(n_chunks, dtype=np.uint8)
    for b in range(16):
        par ^= ((x >> np.uint64(b)) & np.uint64(1)).astype(np.uint8)
    page = idx >> np.uint64(9)                       # 512 chunks per 2 MiB page
    c = (mix64_np(page + np.uint64(seed)) & np.uint64(1)).astype(np.uint8)
    return (par ^ c).astype(np.uint8)

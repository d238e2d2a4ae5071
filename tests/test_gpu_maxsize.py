"""Largest shapes: operands and outputs beyond 2^32 bytes and 2^31 elements, a million-deep contraction, a
million-key request.  Integer-valued inputs keep every sum exact, so sampled outputs must equal the fp64 oracle
bit for bit and whole-matrix checksums must equal the closed form; nothing here is a tolerance test."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from oracle import gemm as og
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import device_topo, to_dev_bf16

pytestmark = pytest.mark.gpu


def device_small_ints(rows, cols, seed):
    """Seeded integers in {-2..2} as bf16, drawn on the device (too many for the host generator to be quick)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device="cuda")
    step = max(1, (1 << 28) // cols)
    for r in range(0, rows, step):
        n = min(step, rows - r)
        out[r:r + n] = torch.randint(-2, 3, (n, cols), generator=g, device="cuda", dtype=torch.int8).to(torch.bfloat16)
    return out


def bits_of(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("tile_m,tile_n", [(256, 256), (128, 256)])
def test_output_beyond_two_to_the_31_elements(tile_m, tile_n):
    """C has 65792 x 33024 = 2.17e9 fp32 entries (8.7 GB): row offsets pass 2^31 elements and 2^33 bytes."""
    M, N, K = 65792, 33024, 64
    assert M * N > 2 ** 31
    A, B = inputs.small_int_bf16(M, K, 71), inputs.small_int_bf16(K, N, 72)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=tile_m, tile_n=tile_n,
                                                                raster_group=4))
    plan.reset_record()
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    owner, count = plan.tile_record()
    assert (count == 1).all()
    # whole matrix: every entry written, and the sum of all entries equals (column sums of A) . (row sums of B)
    assert not bool(torch.isnan(dC).any())
    a64, b64 = inputs.bf16_bits_to_f64(A), inputs.bf16_bits_to_f64(B)
    assert float(dC.sum(dtype=torch.float64)) == float(a64.sum(axis=0) @ b64.sum(axis=1))
    # per-row sums (exact small integers) against the oracle's closed form for every row
    row_sum = dC.sum(dim=1, dtype=torch.float64).cpu().numpy()
    assert np.array_equal(row_sum, a64 @ b64.sum(axis=1))
    # sampled rows in full: the first and last tile, the rows around element 2^31, some anywhere
    edge = 2 ** 31 // N
    rows = np.unique(np.concatenate([np.arange(0, 4), np.arange(M - 260, M), np.arange(edge - 3, edge + 4),
                                     np.random.default_rng(3).integers(0, M, 64)]))
    got = dC[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    assert np.array_equal(got, og.gemm_blocked(A[rows], B))


@pytest.mark.parametrize("k_splits,in_memory", [(1, 0), (4, 1), (4, 0)])
def test_weights_beyond_four_gigabytes(k_splits, in_memory):
    """Decode-shaped GEMM over 1088 x 2098176 row-major weights (4.57 GB): byte offsets into B pass 2^32."""
    M, K, N = 16, 1088, (1 << 21) + 1024
    assert K * N * 2 > 2 ** 32
    dB = device_small_ints(K, N, 81)
    A = inputs.small_int_bf16(M, K, 82)
    dA = to_dev_bf16(A)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16, tile_n=128,
                                                                k_splits=k_splits, splitk_in_memory=in_memory))
    plan.reset_record()
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    owner, count = plan.tile_record()
    assert (count == 1).all()
    assert not bool(torch.isnan(dC).any())
    # column checksum over the whole output: sum over rows of C = (column sums of A) . B, computed per column block on the
    # device in fp64 from the same bits (a reduction of the inputs, none of the kernel's arithmetic)
    a_col = torch.from_numpy(inputs.bf16_bits_to_f64(A).sum(axis=0)).cuda()
    want = torch.empty(N, dtype=torch.float64, device="cuda")
    for c in range(0, N, 1 << 18):
        want[c:c + (1 << 18)] = a_col @ dB[:, c:c + (1 << 18)].to(torch.float64)
    assert torch.equal(dC.sum(dim=0, dtype=torch.float64), want)
    # sampled columns against the oracle: first and last tiles and some anywhere
    cols = np.unique(np.concatenate([np.arange(0, 130), np.arange(N - 260, N), np.random.default_rng(4).integers(0, N, 256)]))
    tc = torch.from_numpy(cols).cuda()
    got = dC[:, tc].cpu().numpy().astype(np.float64)
    assert np.array_equal(got, og.gemm_blocked(A, bits_of(dB[:, tc])))


def test_contraction_over_a_million():
    """K = 2^20 on the decode-shaped kernel (16384 k-slabs in 16 splits) and K = 2^19 on block pairs: slab counters and
    pipeline phases over many laps.  |sums| stay below 2^24, so fp32 accumulation is exact."""
    topo = device_topo()
    M, N, K = 16, 256, 1 << 20
    A, B = inputs.small_int_bf16(M, K, 91), inputs.small_int_bf16(K, N, 92)
    want = og.gemm_blocked(A, B)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    for ksp, in_mem in ((16, 0), (16, 1), (1, 0)):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16, tile_n=128,
                                                                    k_splits=ksp, splitk_in_memory=in_mem))
        ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), want)
    del dA, dB
    M, N, K = 512, 256, 1 << 19
    A, B = inputs.small_int_bf16(M, K, 93), inputs.small_int_bf16(K, N, 94)
    want = og.gemm_blocked(A, B)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    for tile_m, ksp in ((256, 1), (128, 1), (128, 4)):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=tile_m, tile_n=256,
                                                                    k_splits=ksp))
        ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), want)


def test_request_of_a_million_keys():
    """One request at the documented maximum of 2^20 keys: 1024 chunks per KV head, combined by the second kernel."""
    B, Hq, Hkv, L, D = 1, 8, 2, 1 << 20, 128
    Q = inputs.uniform_bf16(B * Hq, D, 101).reshape(B, Hq, D)
    K = inputs.uniform_bf16(B * Hkv * L, D, 102).reshape(B, Hkv, L, D)
    V = inputs.uniform_bf16(B * Hkv * L, D, 103).reshape(B, Hkv, L, D)
    topo = device_topo()
    n_chunks = L // 1024
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=Hq // Hkv, N=128 * B * Hkv * n_chunks, K=L,
                                                                tile_m=16, tile_n=128, k_splits=1))
    kv_bytes = 2 * B * Hkv * L * D * 2
    dst_bytes = kv_bytes + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dK, dV, dQ = to_dev_bf16(K.reshape(-1, D)), to_dev_bf16(V.reshape(-1, D)), to_dev_bf16(Q.reshape(-1, D))
    kv = ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L, plan, amap, dst.data_ptr(), dst_bytes, ag.KV_INTERLEAVED)
    dO = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    for kv_len in (None, [L - 77]):
        dlen = None if kv_len is None else torch.tensor(kv_len, dtype=torch.int32, device="cuda")
        ag.attention_decode(dQ.data_ptr(), kv, None if dlen is None else dlen.data_ptr(), dO.data_ptr(), B, Hq, plan)
        torch.cuda.synchronize()
        st = plan.last_status()
        assert st == ag.AG_OK, (ag.strerror(st), plan.last_status_where())
        got = dO.cpu().numpy().astype(np.float64)
        want = oa.gqa_decode(Q, K, V, kv_len=None if kv_len is None else np.array(kv_len))
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert np.isfinite(got).all() and rel <= 5e-5 and np.abs(got - want).max() <= 2e-4, rel
    with pytest.raises(ag.AgError):                          # one page more than the documented maximum
        ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L + 128, plan, amap, dst.data_ptr(), dst_bytes, ag.KV_INTERLEAVED)

"""Seeded random shapes and policies: the CUDA plan must equal the oracle's bytewise and the GEMM under it
must be bit-exact on integer-valued inputs (any summation order is exact there)."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from oracle import plan as op
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import device_topo, oracle_policy, run_gemm

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", range(24))
def test_random_case(case):
    rng = np.random.default_rng(1000 + case)
    topo = device_topo()
    topo_d = topo.as_dict()
    pairs = bool(rng.integers(0, 2))
    M = int(rng.integers(1, 1200))
    N = int(rng.integers(1, 200)) * 8
    K = int(rng.integers(1, 120)) * 8
    kind = int(rng.choice([ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT]))
    kw = dict(kind=kind, M=M, N=N, K=K, raster_group=int(rng.integers(1, 6)))
    if pairs:
        b = 2 * int(rng.integers(1, topo.n_sm // 2 + 1))
        kw.update(tile_m=256, tile_n=256, sm_select=int(rng.integers(0, 2)), pair_lists=1)
        if kind == ag.AG_OBLIVIOUS:
            kw["seed"] = 0                                  # lowest ids: whole TPCs
    else:
        b = int(rng.integers(1, topo.n_sm + 1))
        n_slab = -(-K // 64)
        ksp = int(rng.integers(1, min(3, n_slab) + 1))
        per = -(-n_slab // ksp)
        if (ksp - 1) * per >= n_slab:
            ksp = 1
        kw.update(tile_m=128, tile_n=int(rng.choice([64, 128, 256])), k_splits=ksp, static_assign=int(rng.integers(0, 2)),
                  seed=int(rng.integers(0, 4)) if kind == ag.AG_OBLIVIOUS else 0)
    plan = ag.sched_build(topo, None, b, ag.make_policy(**kw))
    want = op.export(op.build_plan(topo_d, None, b, oracle_policy(**kw)))
    assert plan.export().tobytes() == want.tobytes(), kw
    A, B = inputs.small_int_bf16(M, K, 7 + case), inputs.small_int_bf16(K, N, 77 + case)
    plan.reset_record()
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B)), kw
    _, count = plan.tile_record()
    assert (count == 1).all()


@pytest.mark.parametrize("case", range(24))
def test_random_affinity_plan(case):
    """Affinity plans over random chunk-to-die tables: random shapes, operands present or not, margins clipped or not,
    inverted or not, either quota rule, any budget - bytewise equal to the oracle's (the CUDA builder finds the full
    die's cut by a radix select, the oracle sorts)."""
    rng = np.random.default_rng(5000 + case)
    topo = inputs.synthetic_topo(die0_sms=int(rng.choice([70, 72, 74])), seed=case)
    M = int(rng.integers(1, 1100))
    N = int(rng.integers(1, 160)) * 8
    K = int(rng.integers(1, 130)) * 8
    tile_m, tile_n = int(rng.choice([16, 128])), int(rng.choice([64, 128, 256]))
    n_slab = -(-K // 64)
    ksp = int(rng.integers(1, min(4, n_slab) + 1))
    per = -(-n_slab // ksp)
    if (ksp - 1) * per >= n_slab:
        ksp = 1
    a_off, b_off, c_off = 0, M * K * 2, M * K * 2 + K * N * 2
    nbytes = c_off + M * N * 4
    n_chunks = -(-nbytes // 4096) + 1
    style = case % 3
    if style == 0:
        tbl = rng.integers(0, 2, size=n_chunks, dtype=np.uint8)            # noise: every margin differs
    elif style == 1:
        tbl = inputs.synthetic_chunk_die(n_chunks, seed=case).copy()        # XOR hash: many exact ties
        tbl[:: int(rng.integers(3, 9))] = int(rng.integers(0, 2))
    else:
        tbl = (np.arange(n_chunks) // int(rng.integers(1, 64)) % 2).astype(np.uint8)   # long runs: one die oversubscribed
    present = rng.integers(0, 2, size=3)
    if not present.any():
        present[int(rng.integers(0, 3))] = 1
    ops = {}
    if present[0]:
        ops["a"] = dict(offset=a_off, row_stride=K * 2, elem_bytes=2)
    if present[1]:
        ops["b"] = dict(offset=b_off, row_stride=N * 2, elem_bytes=2)
    if present[2]:
        ops["c"] = dict(offset=c_off, row_stride=N * 4, elem_bytes=4)
    kw = dict(kind=ag.AG_AFFINITY, M=M, N=N, K=K, tile_m=tile_m, tile_n=tile_n, k_splits=ksp, raster_group=int(rng.integers(1, 9)),
              invert_affinity=int(rng.integers(0, 2)), min_margin=int(rng.choice([0, 0, 512, 4096, 1 << 16])),
              die_quota=int(rng.integers(0, 2)), **ops)
    b = int(rng.integers(1, 149))
    plan = ag.sched_build(ag.TopoMap.from_dict(topo), ag.affinity_from_table(0, tbl), b, ag.make_policy(**kw))
    want = op.export(op.build_plan(topo, dict(chunk_bytes=4096, die_of_chunk=tbl), b, oracle_policy(**kw)))
    assert plan.export().tobytes() == want.tobytes(), (kw, b)


@pytest.mark.parametrize("case", range(24))
def test_random_decode_shaped_case(case):
    """The decode-shaped kernel over random shapes: 1 to 128 activation rows, row-major weights, die-local pages (groups or
    single pages) or pages in consecutive chunks, both split-K modes, any SM budget, launches overlapping or not; three
    calls queued back to back, exact on integer inputs."""
    rng = np.random.default_rng(9000 + case)
    topo = device_topo()
    M = int(rng.choice([1, 7, 16, 17, 32, 33, 64, 100, 128]))
    layout = int(rng.integers(0, 4))                          # 0 row-major, 1 die-local groups, 2 die-local single pages, 3 consecutive
    N = int(rng.integers(1, 40)) * (128 if layout else 8)
    K = int(rng.integers(1, 40)) * (64 if layout else 8)
    n_slab = -(-K // 64)
    ksp = int(rng.integers(1, min(6, n_slab) + 1))
    per = -(-n_slab // ksp)
    if (ksp - 1) * per >= n_slab:
        ksp = 1
    tile_m = 16 if M <= 16 else 32 if M <= 32 else 64 if M <= 64 else 128
    kw = dict(kind=int(rng.choice([ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT])), M=M, N=N, K=K, tile_m=tile_m, tile_n=128, k_splits=ksp,
              splitk_in_memory=int(rng.integers(0, 2)), overlap_launches=int(rng.integers(0, 3)), decode_shaped=1 if M > 64 else 0,
              sm_select=int(rng.integers(0, 2)), static_assign=1)
    b = int(rng.integers(1, topo.n_sm + 1))
    plan = ag.sched_build(topo, None, b, ag.make_policy(**kw))
    A, B = inputs.small_int_bf16(M, K, 300 + case), inputs.small_int_bf16(K, N, 400 + case)
    dA, dB = torch.from_numpy(A.view(np.int16).copy()).cuda(), torch.from_numpy(B.view(np.int16).copy()).cuda()
    dCs = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    packed = None
    if layout:
        n_pages = (N // 128) * (K // 16)
        dst_bytes = n_pages * 4096 * (1 if layout == 3 else 2) + (8 << 20)
        dst = ag.aligned_device_bytes(dst_bytes)
        amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
        packed = ag.pack_weights(dB.data_ptr(), K, N, plan, amap, dst.data_ptr(), dst_bytes, single_pages=layout == 2, consecutive=layout == 3)
    plan.reset_record()
    for dC in dCs:
        if packed is not None:
            ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan)
        else:
            ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK, (kw, b, layout, plan.last_status_where())
    want = og.gemm_blocked(A, B)
    for dC in dCs:
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), want), (kw, b, layout)
    _, count = plan.tile_record()
    assert (count == 3).all()

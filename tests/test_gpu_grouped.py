"""Grouped (MoE-shaped) decode GEMM against the fp64 oracle, expert by expert."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import check_close, device_topo, to_dev_bf16

pytestmark = pytest.mark.gpu


def make_problem(G, M, N, K, seed, integer):
    rows = inputs.group_rows(G, M, seed)
    total = int(rows.sum())
    gen = inputs.small_int_bf16 if integer else inputs.uniform_bf16
    A_all = gen(total, K, seed + 1)
    Bs = [gen(K, N, seed + 10 + g) for g in range(G)]
    return rows, A_all, Bs


def expert_refs(rows, A_all, Bs):
    out, off = [], 0
    for g, r in enumerate(rows):
        out.append(og.gemm_blocked(A_all[off:off + r], Bs[g]) if r else np.zeros((0, Bs[g].shape[1])))
        off += r
    return np.concatenate(out, axis=0)


def test_group_rows_follow_the_paper_recipe():
    r = inputs.group_rows(32, 20, seed=1)
    assert r.min() >= 14 and r.max() <= 25 and len(set(r.tolist())) > 3
    assert np.array_equal(r, inputs.group_rows(32, 20, seed=1))
    assert abs(inputs.group_rows(4096, 192, seed=2).mean() - 192) < 3


@pytest.mark.parametrize("G,M,N,K,ksp,in_mem", [(6, 20, 512, 512, 1, 0), (6, 20, 512, 1024, 4, 1), (32, 20, 256, 512, 2, 0),
                                                (5, 12, 384, 256, 2, 1), (6, 48, 512, 512, 2, 1), (4, 96, 256, 1024, 4, 0)])
def test_grouped_rowmajor_integer_exact(G, M, N, K, ksp, in_mem):
    rows, A_all, Bs = make_problem(G, M, N, K, seed=3, integer=True)
    topo = device_topo()
    tile_m = 16 if rows.max() <= 16 else 32 if rows.max() <= 32 else 64 if rows.max() <= 64 else 128   # up to 128 rows per expert
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=int(rows.max()), N=G * N, K=K,
                                                                tile_m=tile_m, tile_n=128, k_splits=ksp,
                                                                splitk_in_memory=in_mem, decode_shaped=1))
    dA = to_dev_bf16(A_all)
    dBs = [to_dev_bf16(b) for b in Bs]
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in dBs], N, K, tile_m)
    ref = expert_refs(rows, A_all, Bs)
    for _ in range(2):
        dC.fill_(float("nan"))
        ag.gemm_persistent_grouped(desc, None, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref)


def test_grouped_packed_weights_sit_on_the_experts_die_and_match_oracle():
    G, M, N, K, ksp = 8, 20, 1024, 1024, 4
    rows, A_all, Bs = make_problem(G, M, N, K, seed=5, integer=False)
    topo = device_topo()
    kw = dict(M=int(rows.max()), N=G * N, K=K, tile_m=32, tile_n=128, k_splits=ksp, splitk_in_memory=1)
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
    dst_bytes = 2 * G * K * N * 2 + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dBs = [to_dev_bf16(b) for b in Bs]
    packed = ag.pack_weights_grouped([b.data_ptr() for b in dBs], K, N, plan, amap, dst.data_ptr(), dst_bytes)
    # pages of an expert sit on the die whose queue holds the expert's units
    p = plan.parsed()
    unit_die = np.zeros(p["n_units"], dtype=np.uint8)
    unit_die[p["die_q"][int(p["die_q_off"][1]):]] = 1
    table, tbl = packed.page_table(), amap.export()
    ppt, tiles = K // 16, N // 128
    page_owner = np.repeat(unit_die, ppt // ksp)             # units are (tn, ks), pages of a unit are consecutive
    assert (tbl[table] == page_owner).mean() > 0.99
    # experts are kept together: at most one expert straddles the cut between the dies
    expert_dies = [set(unit_die[g * tiles * ksp:(g + 1) * tiles * ksp].tolist()) for g in range(G)]
    assert sum(1 for s in expert_dies if len(s) > 1) <= 1
    dA = to_dev_bf16(A_all)
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, None, N, K, 32)
    ag.gemm_persistent_grouped(desc, packed, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    check_close(dC.cpu().numpy(), expert_refs(rows, A_all, Bs))
    # a descriptor made without row-major weights cannot be used without packed ones
    assert ag.lib().gemm_persistent_grouped(desc.handle, None, plan.handle, None) == ag.AG_ERR_ARG


def test_grouped_handles_an_expert_without_rows():
    G, N, K = 4, 256, 256
    rows = np.array([9, 0, 16, 3], dtype=np.int32)
    A_all = inputs.small_int_bf16(int(rows.sum()), K, 1)
    Bs = [inputs.small_int_bf16(K, N, 2 + g) for g in range(G)]
    topo = device_topo()
    plan = ag.sched_build(topo, None, 16, ag.make_policy(kind=ag.AG_OBLIVIOUS, M=16, N=G * N, K=K, tile_m=16, tile_n=128))
    dA = to_dev_bf16(A_all)
    dBs = [to_dev_bf16(b) for b in Bs]
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in dBs], N, K, 16)
    ag.gemm_persistent_grouped(desc, None, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    assert np.array_equal(dC.cpu().numpy().astype(np.float64), expert_refs(rows, A_all, Bs))


@pytest.mark.parametrize("ksp,in_mem,budget,overlap", [(1, 0, None, 0), (4, 1, None, 0), (4, 0, 37, 0), (2, 1, 5, 0),
                                                       (4, 1, None, 2), (4, 1, 37, 2), (2, 0, 74, 1)])
def test_grouped_mostly_idle_experts(ksp, in_mem, budget, overlap):
    """A mixture-of-experts step in which most experts have no token: their units are ticked off without touching
    their weights (every unit still shows up once per launch in the record), the others are exact."""
    G, N, K = 16, 256, 512
    rows = np.zeros(G, dtype=np.int32)
    rows[[1, 6, 7, 13]] = [5, 16, 1, 11]
    A_all = inputs.small_int_bf16(int(rows.sum()), K, 71)
    Bs = [inputs.small_int_bf16(K, N, 72 + g) for g in range(G)]
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm if budget is None else budget,
                          ag.make_policy(kind=ag.AG_DIE_COMPACT, M=16, N=G * N, K=K, tile_m=16, tile_n=128, k_splits=ksp, splitk_in_memory=in_mem,
                                         overlap_launches=overlap))
    dA = to_dev_bf16(A_all)
    dBs = [to_dev_bf16(b) for b in Bs]
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in dBs], N, K, 16)
    plan.reset_record()
    for _ in range(3):
        ag.gemm_persistent_grouped(desc, None, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    assert np.array_equal(dC.cpu().numpy().astype(np.float64), expert_refs(rows, A_all, Bs))
    owner, count = plan.tile_record()
    assert (count == 3).all()


@pytest.mark.parametrize("G,M,N,K,integer", [(6, 192, 512, 256, True), (3, 700, 768, 512, True), (8, 192, 1024, 1024, False)])
def test_grouped_dense_block_pairs(G, M, N, K, integer):
    """Many rows per expert (the paper's M = 192 / 1024 settings, scaled down): block pairs with
    per-expert A, B and C views; units below an expert's last row are skipped."""
    rows, A_all, Bs = make_problem(G, M, N, K, seed=7, integer=integer)
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=int(rows.max()), N=G * N, K=K,
                                                                tile_m=256, tile_n=256, raster_group=1))
    dA = to_dev_bf16(A_all)
    dBs = [to_dev_bf16(b) for b in Bs]
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in dBs], N, K, 256)
    ref = expert_refs(rows, A_all, Bs)
    for _ in range(2):
        dC.fill_(float("nan"))
        ag.gemm_persistent_grouped(desc, None, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        C = dC.cpu().numpy()
        if integer:
            assert np.array_equal(C.astype(np.float64), ref)
        else:
            check_close(C, ref)


def test_grouped_dense_over_packed_weights():
    G, M, N, K = 4, 192, 512, 512
    rows, A_all, Bs = make_problem(G, M, N, K, seed=9, integer=True)
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=int(rows.max()), N=G * N, K=K,
                                                                tile_m=256, tile_n=256))
    dst_bytes = 2 * G * K * N * 2 + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dBs = [to_dev_bf16(b) for b in Bs]
    packed = ag.pack_weights_grouped([b.data_ptr() for b in dBs], K, N, plan, amap, dst.data_ptr(), dst_bytes)
    dA = to_dev_bf16(A_all)
    dC = torch.full((int(rows.sum()), N), float("nan"), dtype=torch.float32, device="cuda")
    desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, None, N, K, 256)
    ag.gemm_persistent_grouped(desc, packed, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    assert np.array_equal(dC.cpu().numpy().astype(np.float64), expert_refs(rows, A_all, Bs))

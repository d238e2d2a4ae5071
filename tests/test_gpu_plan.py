"""sched_build (CUDA plan builder) against the CPU oracle: plan images must be bytewise equal."""
import numpy as np
import pytest

from oracle import plan as op
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import oracle_policy

pytestmark = pytest.mark.gpu


def both(topo_d, amap_tbl, budget, **kw):
    topo = ag.TopoMap.from_dict(topo_d)
    amap = ag.affinity_from_table(0, amap_tbl) if amap_tbl is not None else None
    plan = ag.sched_build(topo, amap, budget, ag.make_policy(**kw))
    got = plan.export()
    okw = dict(kw)
    if "avoid" in okw:
        okw["avoid"] = tuple(okw["avoid"])
    o_amap = dict(chunk_bytes=4096, die_of_chunk=amap_tbl) if amap_tbl is not None else None
    want = op.export(op.build_plan(topo_d, o_amap, budget, oracle_policy(**okw)))
    return got, want, plan


@pytest.mark.parametrize("die0", [70, 72, 74])
@pytest.mark.parametrize("kind", [ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT])
@pytest.mark.parametrize("b", [1, 16, 37, 74, 111, 148])
def test_plan_matches_oracle_oblivious_and_compact(die0, kind, b):
    topo = inputs.synthetic_topo(die0_sms=die0, seed=die0)
    for shape, g, ksp in (((4096, 4096, 4096), 4, 1), ((1000, 1000, 1000), 1, 1), ((16, 8192, 8192), 1, 4)):
        M, N, K = shape
        got, want, _ = both(topo, None, b, kind=kind, M=M, N=N, K=K, raster_group=g, k_splits=ksp,
                            tile_m=128 if M > 16 else 16, tile_n=256 if M > 16 else 128)
        assert got.tobytes() == want.tobytes()


@pytest.mark.parametrize("seed", [1, 2, 17, 32])
@pytest.mark.parametrize("b", [16, 32, 48, 64, 74])
def test_seeded_random_subsets_match_oracle(seed, b):
    topo = inputs.synthetic_topo(die0_sms=72, seed=2)
    got, want, _ = both(topo, None, b, kind=ag.AG_OBLIVIOUS, seed=seed, M=4096, N=4096, K=4096)
    assert got.tobytes() == want.tobytes()


@pytest.mark.parametrize("b", [16, 48, 64, 74, 111])
def test_gpc_spread_selection_matches_oracle(b):
    topo = inputs.synthetic_topo(die0_sms=70, seed=8)
    for kind in (ag.AG_DIE_COMPACT,):
        got, want, _ = both(topo, None, b, kind=kind, M=4096, N=4096, K=4096, raster_group=8, sm_select=1)
        assert got.tobytes() == want.tobytes()


@pytest.mark.parametrize("b", [16, 37, 74, 111, 148])
def test_equal_die_quota_matches_oracle(b):
    """die_quota = 1 (equal shares for the dies that hold SMs): bytewise equal to the oracle."""
    for die0 in (70, 74):
        topo = inputs.synthetic_topo(die0_sms=die0, seed=die0 + 1)
        for kw in (dict(M=16, N=8192, K=8192, tile_m=16, tile_n=128, k_splits=8), dict(M=4, N=128 * 1000 + 128, K=512, tile_m=16, tile_n=128),
                   dict(M=4096, N=4096, K=4096, raster_group=4)):
            for sel in (0, 1):
                got, want, plan = both(topo, None, b, kind=ag.AG_DIE_COMPACT, die_quota=1, sm_select=sel, **kw)
                assert got.tobytes() == want.tobytes()
                p = plan.parsed()
                n_d = [int(x) for x in p["die_sm_count"]]
                if min(n_d) > 0:
                    q0 = int(p["die_q_off"][1])
                    assert abs(2 * q0 - int(p["n_units"])) <= 1


@pytest.mark.parametrize("c", [4, 8])
@pytest.mark.parametrize("b", [10, 32, 64, 72, 100, 140, 148])
def test_cluster_aware_sets_match_oracle(c, b):
    """Sets for kernels that launch clusters of c blocks: bytewise equal to the oracle, and the capacity the library
    reports is the oracle's."""
    for die0, seed in ((70, 3), (74, 6)):
        topo = inputs.synthetic_topo(die0_sms=die0, seed=seed)
        for sel in (0, 1):
            got, want, plan = both(topo, None, b, kind=ag.AG_DIE_COMPACT, M=4096, N=4096, K=4096, raster_group=4,
                                   sm_select=sel, cluster_size=c)
            assert got.tobytes() == want.tobytes()
            S = [int(x) for x in plan.parsed()["sm_list"]]
            assert plan.cluster_capacity(ag.TopoMap.from_dict(topo), c) == op.cluster_capacity(topo, S, c)
    # the hand-worked toy chip: one random TPC, a GPC of five TPCs
    toy = dict(n_sm=24, n_tpc=12, n_gpc=3, n_die=2, tpc=np.array([s // 2 for s in range(24)]),
               gpc=np.array([0] * 10 + [1] * 8 + [2] * 6), die=np.array([0] * 18 + [1] * 6),
               is_random=np.array([0] * 22 + [1, 1]), gpc_die=[0, 0, 1], die_sm_count=[18, 6], gpc_sm_count=[10, 8, 6])
    if b <= 24:
        got, want, plan = both(toy, None, b, kind=ag.AG_DIE_COMPACT, M=512, N=512, K=64, cluster_size=c)
        assert got.tobytes() == want.tobytes()
        if (c, b) == (4, 10):
            assert [int(x) for x in plan.parsed()["sm_list"]] == [0, 1, 2, 3, 4, 5, 10, 11, 12, 13]


def test_avoid_mask_and_unplaced_sms():
    topo = inputs.synthetic_topo(die0_sms=74, seed=4)
    topo["gpc"] = topo["gpc"].copy()
    topo["gpc"][topo["is_random"] == 1] = -1                  # random SMs not yet placed
    avoid = [s for s in range(148) if topo["die"][s] == 1][:38]
    for kind in (ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT):
        got, want, _ = both(topo, None, 74, kind=kind, M=8192, N=4096, K=4096, avoid=avoid, raster_group=2)
        assert got.tobytes() == want.tobytes()
    with pytest.raises(ag.AgError):
        both(topo, None, 111, kind=ag.AG_DIE_COMPACT, M=8192, N=4096, K=4096, avoid=avoid)


def test_full_size_config_plans_match():
    """The 8192^3 case with 128x256 tiles on all SMs (2048 units)."""
    topo = inputs.synthetic_topo(die0_sms=70, seed=11)
    for kind in (ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT):
        for g in (1, 8):
            got, want, _ = both(topo, None, 148, kind=kind, M=8192, N=8192, K=8192, raster_group=g)
            assert got.tobytes() == want.tobytes()


@pytest.mark.parametrize("invert,min_margin", [(0, 0), (1, 0), (0, 20000), (0, 1 << 40)])
def test_affinity_plan_matches_oracle_rowmajor(invert, min_margin):
    topo = inputs.synthetic_topo(die0_sms=72, seed=6)
    M = N = K = 1024
    a_off, b_off, c_off = 0, M * K * 2, M * K * 2 + K * N * 2
    nbytes = c_off + M * N * 4
    tbl = inputs.synthetic_chunk_die(nbytes // 4096, seed=3)
    # break the perfect pair balance so that margins are not all zero
    tbl = tbl.copy()
    tbl[::7] = 0
    kw = dict(kind=ag.AG_AFFINITY, M=M, N=N, K=K, tile_m=128, tile_n=128, invert_affinity=invert, raster_group=2,
              min_margin=min_margin,
              a=dict(offset=a_off, row_stride=K * 2, elem_bytes=2),
              b=dict(offset=b_off, row_stride=N * 2, elem_bytes=2),
              c=dict(offset=c_off, row_stride=N * 4, elem_bytes=4))
    got, want, plan = both(topo, tbl, 148, **kw)
    assert got.tobytes() == want.tobytes()
    if min_margin >= 1 << 40:                               # every margin is a tie: the die_compact bands
        dc = op.export(op.build_plan(topo, None, 148, oracle_policy(kind=op.DIE_COMPACT, M=M, N=N, K=K, tile_m=128,
                                                                    tile_n=128, raster_group=2)))
        assert np.array_equal(got[2:], dc[2:])
    # margins, unit by unit
    pol = oracle_policy(**kw)
    amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    R = op.raster_order(8, 8, 1, 2)
    m = plan.margins()
    for i in (0, 1, 17, 63):
        l0, l1 = op.unit_local_bytes(pol, amap, R[i])
        assert m[i] == l0 - l1


@pytest.mark.parametrize("invert", [0, 1])
def test_affinity_plan_with_100k_units_and_tied_margins_matches_oracle(invert):
    """More units than a sort-free builder used to take (65536), with only five distinct margin values, so the cut
    between the units a full die keeps and those it passes on falls inside a run of equal keys."""
    topo = inputs.synthetic_topo(die0_sms=70, seed=4)
    U = 100_000
    M, N, K = 4, 128 * U, 64
    nbytes = M * N * 4
    tbl = inputs.synthetic_chunk_die(nbytes // 4096, seed=11).copy()
    tbl[::3] = 0                                             # die 0 is preferred by more units than its quota
    kw = dict(kind=ag.AG_AFFINITY, M=M, N=N, K=K, tile_m=16, tile_n=128, invert_affinity=invert, raster_group=1,
              c=dict(offset=0, row_stride=N * 4, elem_bytes=4))
    got, want, plan = both(topo, tbl, 148, **kw)
    assert got.tobytes() == want.tobytes()
    m = np.abs(plan.margins())
    assert len(np.unique(m)) <= 5 and (m > 0).sum() > U // 4


def test_affinity_full_size_sampled_margins_and_invariants():
    """8192^3 / 2048 units: the oracle scores a sample of units; the rest is checked by invariants."""
    topo = inputs.synthetic_topo(die0_sms=70, seed=12)
    M = N = K = 8192
    a_off, b_off, c_off = 0, M * K * 2, 2 * M * K * 2
    nbytes = c_off + M * N * 4
    tbl = inputs.synthetic_chunk_die(nbytes // 4096, seed=9).copy()
    tbl[::5] = 1
    kw = dict(kind=ag.AG_AFFINITY, M=M, N=N, K=K, raster_group=8,
              a=dict(offset=a_off, row_stride=K * 2, elem_bytes=2),
              b=dict(offset=b_off, row_stride=N * 2, elem_bytes=2),
              c=dict(offset=c_off, row_stride=N * 4, elem_bytes=4))
    plan = ag.sched_build(ag.TopoMap.from_dict(topo), ag.affinity_from_table(0, tbl), 148, ag.make_policy(**kw))
    p = plan.parsed()
    assert sorted(p["die_q"]) == list(range(2048)) and sorted(p["sm_q"]) == list(range(2048))
    assert list(p["die_q_off"]) == [0, op.quotas(2048, [70, 78], 148)[0], 2048]
    pol = oracle_policy(**kw)
    amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    R = op.raster_order(64, 32, 1, 8)
    m = plan.margins()
    for i in (0, 777, 2047):
        l0, l1 = op.unit_local_bytes(pol, amap, R[i])
        assert m[i] == l0 - l1


def test_paged_weights_affinity_recovers_packing_plan():
    topo = inputs.synthetic_topo(die0_sms=70, seed=9)
    kw = dict(M=16, N=2048, K=1024, tile_m=16, tile_n=128, k_splits=2)
    plan_d = op.build_plan(topo, None, 148, op.default_policy(kind=op.DIE_COMPACT, **kw))
    unit_die = [0] * plan_d["n_units"]
    for d in (0, 1):
        for u in plan_d["die_q"][d]:
            unit_die[u] = d
    n_log = 16 * 64
    tbl = inputs.synthetic_chunk_die(2 * n_log, seed=5)
    table = op.build_page_table(op.page_die_from_plan(plan_d, 1024), dict(chunk_bytes=4096, die_of_chunk=tbl))
    bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=table)
    for inv in (0, 1):
        got, want, _ = both(topo, tbl, 148, kind=ag.AG_AFFINITY, invert_affinity=inv, b=bop, **kw)
        assert got.tobytes() == want.tobytes()


def test_bad_arguments():
    topo = ag.TopoMap.from_dict(inputs.synthetic_topo())
    for kw in (dict(M=0, N=8, K=8), dict(M=128, N=128, K=128, k_splits=3), dict(M=128, N=128, K=128, kind=ag.AG_AFFINITY)):
        with pytest.raises(ag.AgError) as e:
            ag.sched_build(topo, None, 8, ag.make_policy(**kw))
        assert e.value.status == ag.AG_ERR_ARG
    with pytest.raises(ag.AgError):
        ag.sched_build(topo, None, 149, ag.make_policy(M=128, N=128, K=128))


def test_hash_fit_recovers_a_synthetic_xor_mask():
    """Section 6.1.2 on a made-up layout: die = parity(chunk index in page & mask) ^ per-page constant."""
    for mask in (0x1EF, 0x1B5, 0x001):
        tbl = inputs.synthetic_chunk_die(8192, seed=3, mask_bits=mask)
        amap = ag.affinity_from_table(0, tbl)
        got, violations = amap.fit_hash()
        assert got == (mask | 1) and violations == 0
    noisy = inputs.synthetic_chunk_die(8192, seed=3, mask_bits=0x1EF).copy()
    noisy[::97] ^= 1
    got, violations = ag.affinity_from_table(0, noisy).fit_hash()
    assert got == 0x1EF and 0 < violations <= 8192 // 97 + 1


@pytest.mark.parametrize("kind", [ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT])
@pytest.mark.parametrize("b", [16, 48, 74, 148])
def test_pair_lists_match_oracle(kind, b):
    topo = inputs.synthetic_topo(die0_sms=70, seed=13)
    for sel in (0, 1):
        got, want, _ = both(topo, None, b, kind=kind, M=4096, N=4096, K=4096, tile_m=256, tile_n=256, raster_group=4,
                            sm_select=sel, pair_lists=1)
        assert got.tobytes() == want.tobytes()
    with pytest.raises(ag.AgError):
        ag.sched_build(ag.TopoMap.from_dict(topo), None, 37, ag.make_policy(kind=ag.AG_OBLIVIOUS, seed=3, M=4096, N=4096,
                                                                            K=4096, tile_m=256, tile_n=256, pair_lists=1))

"""Pins for the CPU plan builder: hand-derived tiny plans, invariants the paper's scheduling
principles imply, the printed remap formula, and published mixer vectors."""
import os

import numpy as np
import pytest

from oracle import plan as op
from paper_2609_24270_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TOY = dict(n_sm=4, n_tpc=2, n_gpc=2, n_die=2, tpc=[0, 0, 1, 1], gpc=[0, 0, 1, 1],
           die=[0, 0, 1, 1], is_random=[0, 0, 0, 0], gpc_die=[0, 1])


def golden():
    out = {}
    for line in open(os.path.join(GOLD, "plan_tiny.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, q0, q1, smq = [f.strip() for f in line.split("|")]
        out[name] = ([int(x) for x in q0.split()], [int(x) for x in q1.split()],
                     [[int(x) for x in s.split()] for s in smq.split(";")])
    return out


def toy_amap_case_d():
    doc = np.zeros(512, dtype=np.uint8)
    for r in range(256):
        tm = r // 128
        for tn in (0, 1):
            u = tm * 2 + tn
            if u == 0:
                d = 1
            elif u == 1:
                d = 0 if (r % 128) < 96 else 1
            elif u == 2:
                d = 0
            else:
                d = 0 if (r % 128) < 64 else 1
            doc[2 * r + tn] = d
    return dict(chunk_bytes=1024, die_of_chunk=doc)


def test_hand_derived_tiny_plans():
    g = golden()
    base = dict(M=256, N=512, K=64)
    cases = {
        "obl_b3": (op.default_policy(kind=op.OBLIVIOUS, **base), None, 3),
        "dc_b3": (op.default_policy(kind=op.DIE_COMPACT, **base), None, 3),
        "dc_g2_k2_b4": (op.default_policy(kind=op.DIE_COMPACT, M=256, N=512, K=128, k_splits=2,
                                          raster_group=2), None, 4),
        "aff_b4": (op.default_policy(kind=op.AFFINITY, c=op.operand(0, 2048, 4), **base),
                   toy_amap_case_d(), 4),
        "aff_inv_b4": (op.default_policy(kind=op.AFFINITY, invert_affinity=1,
                                         c=op.operand(0, 2048, 4), **base), toy_amap_case_d(), 4),
    }
    for name, (pol, amap, b) in cases.items():
        p = op.build_plan(TOY, amap, b, pol)
        assert (p["die_q"][0], p["die_q"][1], p["sm_q"]) == g[name], name


def test_case_d_margins_by_brute_force_byte_count():
    """local_d(u) against a per-byte count over the whole C tile."""
    amap = toy_amap_case_d()
    pol = op.default_policy(kind=op.AFFINITY, M=256, N=512, K=64, c=op.operand(0, 2048, 4))
    want_margin = {0: -131072, 1: 65536, 2: 131072, 3: 0}
    for u in range(4):
        tm, tn = u // 2, u % 2
        cnt = [0, 0]
        for r in range(tm * 128, tm * 128 + 128):
            for byte in range(r * 2048 + tn * 1024, r * 2048 + tn * 1024 + 1024):
                cnt[int(amap["die_of_chunk"][byte // 1024])] += 1
        assert op.unit_local_bytes(pol, amap, u) == cnt
        assert cnt[0] - cnt[1] == want_margin[u]


def test_interval_counting_unaligned():
    doc = np.array([0, 1, 1, 0, 1], dtype=np.uint8)
    amap = dict(chunk_bytes=100, die_of_chunk=doc)
    # [50, 430): 50 of chunk0(d0), 100 c1(d1), 100 c2(d1), 100 c3(d0), 30 c4(d1)
    assert op._bytes_per_die_interval(amap, 50, 430) == [150, 230]
    assert op._bytes_per_die_interval(amap, 120, 120) == [0, 0]


def test_raster_orders():
    assert op.raster_order(2, 3, 1, 1) == [0, 1, 2, 3, 4, 5]
    assert op.raster_order(3, 2, 1, 2) == [0, 2, 1, 3, 4, 5]
    assert sorted(op.raster_order(5, 7, 3, 4)) == list(range(105))


def test_quota_proportional_to_die_sm_count():
    # the 70/78 split the paper reports for some B200 chips (Section 7.1)
    assert op.quotas(2048, [70, 78], 148) == [969, 1079]
    assert op.quotas(2048, [74, 74], 148) == [1024, 1024]
    assert op.quotas(10, [0, 5], 5) == [0, 10]
    for n_u in (1, 7, 512, 2047):
        for n0 in (1, 16, 37, 70):
            q = op.quotas(n_u, [n0, 148 - n0], 148)
            assert sum(q) == n_u
            assert abs(q[0] / n_u - n0 / 148) <= 1.0 / n_u + 1e-12


def test_equal_die_quota_splits_by_dies_not_by_sms():
    """die_quota = 1: hand values on a two-die toy chip (3 + 5 SMs, 10 units in one row of tiles)."""
    topo = dict(n_sm=8, n_tpc=4, n_gpc=2, n_die=2, tpc=np.array([0, 0, 1, 1, 2, 2, 3, 3]), gpc=np.array([0] * 4 + [1] * 4),
                die=np.array([0, 0, 0, 1, 1, 1, 1, 1]), is_random=np.zeros(8, dtype=np.int32), gpc_die=[0, 1],
                die_sm_count=[3, 5], gpc_sm_count=[4, 4])
    base = dict(kind=op.DIE_COMPACT, M=16, N=1280, K=64, tile_m=16, tile_n=128)
    prop = op.build_plan(topo, None, 8, op.default_policy(**base))
    # proportional: floor(10 * 3 / 8) = 3 and floor(10 * 5 / 8) = 6, the unit left over goes to the larger remainder
    # (30 mod 8 = 6 against 50 mod 8 = 2): die 0
    assert [len(q) for q in prop["die_q"]] == [4, 6]
    equal = op.build_plan(topo, None, 8, op.default_policy(die_quota=1, **base))
    assert [len(q) for q in equal["die_q"]] == [5, 5]
    assert equal["die_q"] == [[0, 1, 2, 3, 4], [5, 6, 7, 8, 9]]          # contiguous bands in raster order
    # entry i of a die's queue goes to the SM of rank i mod n_d: die 0's three SMs hold 2, 2, 1 units
    assert [equal["sm_q"][i] for i in range(3)] == [[0, 3], [1, 4], [2]]
    # a set with all its SMs on one die keeps everything there
    one = op.build_plan(topo, None, 4, op.default_policy(die_quota=1, preferred_die=1, **base))
    assert [len(q) for q in one["die_q"]] == [0, 10]
    # odd unit count: the unit left over goes to the lower die (equal remainders)
    odd = op.build_plan(topo, None, 8, op.default_policy(die_quota=1, **dict(base, N=1408)))
    assert [len(q) for q in odd["die_q"]] == [6, 5]


def test_mixer_published_vectors():
    # splitmix64 seeded with 0: published first three outputs
    assert op.mix64(0) == 0xE220A8397B1DCDAF
    assert op.mix64(0x9E3779B97F4A7C15) == 0x6E789E6AA1B965F4
    assert op.mix64((2 * 0x9E3779B97F4A7C15) & ((1 << 64) - 1)) == 0x06C45D188009454F
    # the vectorised generator-side copy agrees with the scalar one
    xs = np.array([0, 1, 12345, 2 ** 63 + 5], dtype=np.uint64)
    assert [int(v) for v in inputs.mix64_np(xs)] == [op.mix64(int(x)) for x in xs]


def seeded_golden():
    out = {}
    for line in open(os.path.join(GOLD, "seeded_subset.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = [f.strip() for f in line.split("|")]
        out[k] = v
    return out


def test_seeded_subset_worked_example():
    """The Fisher-Yates subset for a 6-SM chip and seed 5 against the swaps written out in the golden file."""
    g = seeded_golden()
    toy6 = dict(n_sm=6, n_tpc=3, n_gpc=1, n_die=2, tpc=[0, 0, 1, 1, 2, 2], gpc=[0] * 6, die=[0, 0, 0, 1, 1, 1],
                is_random=[0] * 6, gpc_die=[0])
    seed = int(g["seed"])
    # the listed mixer outputs are the pinned mixer's (published-vector test above) ...
    assert op.mix64(seed) == int(g["base"], 16)
    r = {int(k): int(v, 16) for k, v in (f.split(":") for f in g["r"].split())}
    j = {int(k): int(v) for k, v in (f.split(":") for f in g["j"].split())}
    for i in range(5, 0, -1):
        assert op.mix64((int(g["base"], 16) + i) & ((1 << 64) - 1)) == r[i]
        assert r[i] % (i + 1) == j[i]
    # ... the swaps of the file, replayed, give its final order ...
    arr = list(range(6))
    for i in range(5, 0, -1):
        arr[i], arr[j[i]] = arr[j[i]], arr[i]
    assert arr == [int(x) for x in g["final"].split()]
    # ... and select_sms returns the first b of it, sorted
    for b in (2, 3, 4):
        pol = op.default_policy(kind=op.OBLIVIOUS, seed=seed, M=1, N=1, K=1)
        assert op.select_sms(toy6, b, pol) == [int(x) for x in g[f"b{b}"].split()] == sorted(arr[:b])
    # with SM 1 taken by another plan the candidate list is [0 2 3 4 5]: i runs 4..1 over five entries;
    # r_4 mod 5 = 2, r_3 mod 4 = 0, r_2 mod 3 = 1, r_1 mod 2 = 0 ->
    #   [0 2 3 4 5] -> swap(4,2) [0 2 5 4 3] -> swap(3,0) [4 2 5 0 3] -> swap(2,1) [4 5 2 0 3] -> swap(1,0) [5 4 2 0 3]
    pol = op.default_policy(kind=op.OBLIVIOUS, seed=seed, M=1, N=1, K=1, avoid=[1])
    assert op.select_sms(toy6, 3, pol) == [2, 4, 5]


def test_k_range_when_splits_do_not_divide_the_slabs():
    """Five k-slabs of 64: two splits take 3 + 2 slabs, three splits 2 + 2 + 1 (the first splits take the
    longer runs); a ragged K clips the last slab."""
    pol = op.default_policy(M=1, N=1, K=320, k_unit=64, k_splits=2)
    assert [op.k_range(pol, ks) for ks in range(2)] == [(0, 192), (192, 320)]
    pol = op.default_policy(M=1, N=1, K=320, k_unit=64, k_splits=3)
    assert [op.k_range(pol, ks) for ks in range(3)] == [(0, 128), (128, 256), (256, 320)]
    pol = op.default_policy(M=1, N=1, K=300, k_unit=64, k_splits=2)      # ceil(300 / 64) = 5 slabs, the last holds 44
    assert [op.k_range(pol, ks) for ks in range(2)] == [(0, 192), (192, 300)]
    pol = op.default_policy(M=1, N=1, K=320, k_unit=64, k_splits=4)      # 2 + 2 + 1 + 0: the last split is empty
    assert [op.k_range(pol, ks) for ks in range(4)] == [(0, 128), (128, 256), (256, 320), (320, 320)]
    pol = op.default_policy(M=1, N=1, K=8192, k_unit=64, k_splits=16)
    assert op.k_range(pol, 5) == (5 * 512, 6 * 512)


def test_rowmajor_b_panel_bytes_by_hand_and_by_brute_force():
    """local_d(u) for a row-major B operand: rows = the unit's k range, columns = the unit's tile columns."""
    # B is 128 x 512 bf16 (row stride 1024 B), chunks of 512 B: row k holds chunk 2k (columns 0..255) and
    # chunk 2k+1 (columns 256..511).  Chunks of the left half sit on die 0 for k < 96, else die 1; the right
    # half sits on die 1.  tile_n = 256, two k-splits of one 64-slab each.
    doc = np.zeros(256, dtype=np.uint8)
    for k in range(128):
        doc[2 * k] = 0 if k < 96 else 1
        doc[2 * k + 1] = 1
    amap = dict(chunk_bytes=512, die_of_chunk=doc)
    pol = op.default_policy(kind=op.AFFINITY, M=128, N=512, K=128, tile_m=128, tile_n=256, k_splits=2,
                            b=op.operand(0, 1024, 2))
    # unit id = (tm * 2 + tn) * 2 + ks
    assert op.unit_local_bytes(pol, amap, 0) == [64 * 512, 0]            # tn 0, k 0..63: all on die 0
    assert op.unit_local_bytes(pol, amap, 1) == [32 * 512, 32 * 512]     # tn 0, k 64..127: 32 rows each
    assert op.unit_local_bytes(pol, amap, 2) == [0, 64 * 512]            # tn 1
    assert op.unit_local_bytes(pol, amap, 3) == [0, 64 * 512]
    # an irregular map, an offset that is not chunk aligned, a ragged N: count byte by byte
    rng = np.random.default_rng(3)
    doc = rng.integers(0, 2, size=700).astype(np.uint8)
    amap = dict(chunk_bytes=256, die_of_chunk=doc)
    K, N, off, stride = 192, 328, 136, 672
    pol = op.default_policy(kind=op.AFFINITY, M=64, N=N, K=K, tile_m=64, tile_n=128, k_splits=2, k_unit=64,
                            b=op.operand(off, stride, 2))
    tiles_n = 3
    for u in range(tiles_n * 2):
        ks, tn = u % 2, u // 2
        k0, k1 = op.k_range(pol, ks)
        cnt = [0, 0]
        for k in range(k0, k1):
            for n in range(tn * 128, min(N, tn * 128 + 128)):
                for byte in (0, 1):
                    cnt[int(doc[(off + k * stride + n * 2 + byte) // 256])] += 1
        assert op.unit_local_bytes(pol, amap, u) == cnt
        assert sum(cnt) == (k1 - k0) * (min(N, tn * 128 + 128) - tn * 128) * 2


def check_invariants(topo, plan, pol, b, avoid=()):
    S = plan["sm_list"]
    assert len(S) == b and S == sorted(set(S)) and not (set(S) & set(avoid))
    assert all(0 <= s < topo["n_sm"] for s in S)
    assert [int(topo["die"][s]) for s in S] == plan["sm_die"]
    assert sum(plan["die_sm_count"]) == b
    n_u = plan["n_units"]
    assert sorted(plan["die_q"][0] + plan["die_q"][1]) == list(range(n_u))
    assert sorted(u for l in plan["sm_q"] for u in l) == list(range(n_u))
    for slot, lst in enumerate(plan["sm_q"]):
        if pol["kind"] != op.OBLIVIOUS:
            d = plan["sm_die"][slot]
            assert set(lst) <= set(plan["die_q"][d])
    if pol["kind"] != op.OBLIVIOUS:
        assert [len(q) for q in plan["die_q"]] == plan["quotas"]
    for s, slot in enumerate(plan["smid_to_slot"]):
        assert (slot >= 0) == (s in S)
        if slot >= 0:
            assert S[slot] == s
    lens = [len(l) for l in plan["sm_q"]]
    if pol["kind"] == op.OBLIVIOUS:
        assert max(lens) - min(lens) <= 1


@pytest.mark.parametrize("die0", [70, 72, 74])
@pytest.mark.parametrize("kind", [op.OBLIVIOUS, op.DIE_COMPACT])
@pytest.mark.parametrize("b", [16, 37, 74, 148])
def test_invariants_on_synthetic_b200(die0, kind, b):
    topo = inputs.synthetic_topo(die0_sms=die0, seed=die0)
    assert int((topo["die"] == 0).sum()) == die0 and topo["n_sm"] == 148
    pol = op.default_policy(kind=kind, M=4096, N=4096, K=4096, raster_group=4)
    plan = op.build_plan(topo, None, b, pol)
    check_invariants(topo, plan, pol, b)
    exp = op.export(plan)
    assert exp.dtype == np.int32 and exp[0] == op.PLAN_MAGIC
    assert len(exp) == 16 + 3 * b + 2 + 3 + plan["n_units"] + b + 1 + plan["n_units"] + 148


def test_seeded_subsets_and_avoid_mask():
    topo = inputs.synthetic_topo()
    pol1 = op.default_policy(kind=op.OBLIVIOUS, seed=1, M=4096, N=4096, K=4096)
    pol2 = op.default_policy(kind=op.OBLIVIOUS, seed=2, M=4096, N=4096, K=4096)
    s1, s1b, s2 = op.select_sms(topo, 32, pol1), op.select_sms(topo, 32, pol1), op.select_sms(topo, 32, pol2)
    assert s1 == s1b and s1 != s2 and len(set(s1)) == 32
    # every SM is drawn about equally often over many seeds (Fisher-Yates is unbiased)
    hits = np.zeros(148)
    for seed in range(1, 401):
        for s in op.select_sms(topo, 37, op.default_policy(kind=op.OBLIVIOUS, seed=seed, M=1, N=1, K=1)):
            hits[s] += 1
    assert hits.min() > 60 and hits.max() < 140           # mean 100
    avoid = list(range(0, 148, 2))
    pol = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096, avoid=avoid)
    plan = op.build_plan(topo, None, 40, pol)
    check_invariants(topo, plan, pol, 40, avoid)
    with pytest.raises(ValueError):
        op.select_sms(topo, 75, pol)


def test_die_compact_is_compact_and_gpc_balanced():
    topo = inputs.synthetic_topo(die0_sms=70, seed=3)     # die 1 is the larger (78)
    pol = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096)
    S = op.select_sms(topo, 32, pol)
    assert all(topo["die"][s] == 1 for s in S)            # fits in the primary (larger) die
    per_gpc = np.bincount([topo["gpc"][s] for s in S], minlength=8)
    used = per_gpc[per_gpc > 0]
    assert len(used) == 4 and used.max() - used.min() <= 2        # whole TPCs dealt round-robin
    assert all((s ^ 1) in S for s in S)                   # whole TPCs
    S = op.select_sms(topo, 100, pol)
    assert sum(1 for s in S if topo["die"][s] == 1) == 78  # primary die exhausted first
    pol0 = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096, preferred_die=0)
    assert all(topo["die"][s] == 0 for s in op.select_sms(topo, 32, pol0))


def test_pair_lists_deal_units_to_tpcs():
    toy8 = dict(n_sm=8, n_tpc=4, n_gpc=2, n_die=2, tpc=[0, 0, 1, 1, 2, 2, 3, 3], gpc=[0, 0, 0, 0, 1, 1, 1, 1],
                die=[0, 0, 0, 0, 1, 1, 1, 1], is_random=[0] * 8, gpc_die=[0, 1])
    # hand-derived: 10 units (2 x 5 tiles of 256 x 256), oblivious, 4 TPCs: entries 0..3 -> lower SMs 0,2,4,6;
    # 4..7 -> upper SMs 1,3,5,7; 8,9 -> lower SMs 0,2
    pol = op.default_policy(kind=op.OBLIVIOUS, M=512, N=1280, K=64, tile_m=256, tile_n=256, pair_lists=1)
    plan = op.build_plan(toy8, None, 8, pol)
    assert plan["sm_q"] == [[0, 8], [4], [1, 9], [5], [2], [6], [3], [7]]
    check_invariants(toy8, plan, pol, 8)
    # die_compact, 37 TPCs in one die of a synthetic chip: 256 units -> TPC totals 7 or 6 (ranks dealing: 8 and 6)
    topo = inputs.synthetic_topo(die0_sms=74, seed=5)
    for pair_lists, worst in ((1, 7), (0, 8)):
        pol = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096, tile_m=256, tile_n=256, raster_group=4,
                                pair_lists=pair_lists)
        plan = op.build_plan(topo, None, 74, pol)
        check_invariants(topo, plan, pol, 74)
        per_tpc = [len(plan["sm_q"][2 * j]) + len(plan["sm_q"][2 * j + 1]) for j in range(37)]
        assert max(per_tpc) == worst and sum(per_tpc) == 256
        if pair_lists:   # the two lists of a TPC, taken in alternation (lower first), are the die queue entries j, j+P, ...
            q = plan["die_q"][plan["sm_die"][0]]
            j = 5
            lo, hi = plan["sm_q"][2 * j], plan["sm_q"][2 * j + 1]
            merged = [x for pair in zip(lo, hi + [None]) for x in pair if x is not None]
            assert merged == q[j::37]
    # half a TPC in the set: refused
    with pytest.raises(ValueError):
        op.build_plan(topo, None, 37, op.default_policy(kind=op.OBLIVIOUS, seed=3, M=4096, N=4096, K=4096, tile_m=256,
                                                        tile_n=256, pair_lists=1))


def test_gpc_spread_selection_minimises_sms_per_gpc():
    topo = inputs.synthetic_topo(die0_sms=70, seed=3)
    for b in (16, 48, 64, 100):
        pol = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096, sm_select=1)
        S = op.select_sms(topo, b, pol)
        assert len(S) == b and all((s ^ 1) in S for s in S)            # whole TPCs
        per_gpc = np.bincount([topo["gpc"][s] for s in S], minlength=8)
        sizes = np.bincount(topo["gpc"], minlength=8)
        cap = -(-b // 16) * 2                                         # ceil(b / 8 GPCs) rounded up to a TPC
        assert all(per_gpc[g] <= max(cap, 2) or per_gpc[g] == sizes[g] for g in range(8))
        assert per_gpc.max() - per_gpc[per_gpc < sizes].min() <= 2
        plan = op.build_plan(topo, None, b, pol)
        check_invariants(topo, plan, pol, b)
    # the die-compact set of the same budget sits in four GPCs only
    S0 = op.select_sms(topo, 64, op.default_policy(kind=op.DIE_COMPACT, M=1, N=1, K=1))
    assert len({topo["gpc"][s] for s in S0}) == 4


def test_equal_dies_split_c_in_halves():
    topo = inputs.synthetic_topo(die0_sms=74)
    # one raster group over all 64 tile rows: two contiguous bands of the raster (tn outer): die 0
    # owns the left half of C's columns, die 1 the right half
    pol = op.default_policy(kind=op.DIE_COMPACT, M=8192, N=8192, K=8192, raster_group=64)
    plan = op.build_plan(topo, None, 148, pol)
    assert sorted(plan["die_q"][0]) == [tm * 32 + tn for tm in range(64) for tn in range(16)]
    # groups of 8 tile rows: every group is cut the same way, so the dies advance together
    pol = op.default_policy(kind=op.DIE_COMPACT, M=8192, N=8192, K=8192, raster_group=8)
    plan = op.build_plan(topo, None, 148, pol)
    assert sorted(plan["die_q"][0]) == [tm * 32 + tn for tm in range(64) for tn in range(16)]
    assert plan["die_q"][0][:8] == [tm * 32 for tm in range(8)]
    # unequal dies (70/78): the cut follows floor(x * q0 / n_u) and the quotas still hold exactly
    topo = inputs.synthetic_topo(die0_sms=70, seed=2)
    plan = op.build_plan(topo, None, 148, pol)
    assert [len(q) for q in plan["die_q"]] == op.quotas(2048, [70, 78], 148)
    per_group0 = [sum(1 for u in plan["die_q"][0] if u // 32 // 8 == g) for g in range(8)]
    assert max(per_group0) - min(per_group0) <= 1


def test_min_margin_turns_weak_preferences_into_ties():
    amap = toy_amap_case_d()
    base = dict(M=256, N=512, K=64, c=op.operand(0, 2048, 4))
    # margins are -131072, +65536, +131072, 0: with a floor of 100000 unit 1 becomes a tie and
    # falls back to the die_compact rule (second unit of its tile row -> die 1); unit 3, also a
    # tie for die 1, then finds die 1 full and goes to die 0
    p1 = op.build_plan(TOY, amap, 4, op.default_policy(kind=op.AFFINITY, min_margin=100000, **base))
    assert p1["die_q"] == [[2, 3], [0, 1]]
    # with a floor above every margin the plan is the die_compact one
    p2 = op.build_plan(TOY, amap, 4, op.default_policy(kind=op.AFFINITY, min_margin=1 << 30, **base))
    p3 = op.build_plan(TOY, None, 4, op.default_policy(kind=op.DIE_COMPACT, M=256, N=512, K=64))
    assert p2["die_q"] == p3["die_q"] == [[0, 2], [1, 3]] and p2["sm_q"] == p3["sm_q"]


def test_all_ties_affinity_equals_die_compact():
    topo = inputs.synthetic_topo(die0_sms=72)
    # A rows are 8 KB = one aligned chunk pair (dies 0,1): every margin is exactly 0
    kw = dict(M=1024, N=1024, K=4096, tile_m=128, tile_n=256)
    pa = op.default_policy(kind=op.AFFINITY, a=op.operand(0, 8192, 2), **kw)
    pd = op.default_policy(kind=op.DIE_COMPACT, **kw)
    amap = dict(chunk_bytes=4096, die_of_chunk=(np.arange(4096) & 1).astype(np.uint8))
    assert op.unit_local_bytes(pa, amap, 5) == [128 * 4096, 128 * 4096]
    e_a = op.export(op.build_plan(topo, amap, 148, pa))
    e_d = op.export(op.build_plan(topo, None, 148, pd))
    assert e_a[1] == op.AFFINITY and e_d[1] == op.DIE_COMPACT
    assert np.array_equal(e_a[2:], e_d[2:])               # identical apart from the kind word


def test_packing_by_plan_is_recovered_by_affinity():
    """Pack the weight pages of each unit onto the die a die_compact plan gave the unit;
    the affinity policy must then rebuild that plan, and invert_affinity its mirror."""
    topo = inputs.synthetic_topo(die0_sms=70, seed=9)
    kw = dict(M=16, N=2048, K=1024, tile_m=16, tile_n=128, k_splits=2)
    pd = op.default_policy(kind=op.DIE_COMPACT, **kw)
    plan_d = op.build_plan(topo, None, 148, pd)
    n_tiles = 16
    ppt = 1024 // 16                                       # pages per n-tile
    pages_per_unit = ppt // 2
    unit_die = [0] * plan_d["n_units"]
    for d in (0, 1):
        for u in plan_d["die_q"][d]:
            unit_die[u] = d
    n_log = n_tiles * ppt
    amap = dict(chunk_bytes=4096, die_of_chunk=inputs.synthetic_chunk_die(2 * n_log, seed=5))
    doc = amap["die_of_chunk"]
    assert all(doc[2 * j] != doc[2 * j + 1] for j in range(n_log))      # pair rule of Section 7.1.1
    page_die = op.page_die_from_plan(plan_d, 1024)
    assert page_die == [d for d in unit_die for _ in range(pages_per_unit)]
    table = op.build_page_table(page_die, amap)
    assert len(set(table)) == len(table) and max(table) < 2 * max(page_die.count(0), page_die.count(1))
    assert all(int(doc[table[u * pages_per_unit + p]]) == unit_die[u]
               for u in range(plan_d["n_units"]) for p in range(pages_per_unit))
    bop = op.operand(0, 0, 2, layout=op.LAYOUT_PAGED, page_table=table)
    pa = op.default_policy(kind=op.AFFINITY, b=bop, **kw)
    plan_a = op.build_plan(topo, amap, 148, pa)
    assert plan_a["die_q"] == plan_d["die_q"] and plan_a["sm_q"] == plan_d["sm_q"]
    pi = op.default_policy(kind=op.AFFINITY, invert_affinity=1, b=bop, **kw)
    plan_i = op.build_plan(topo, amap, 148, pi)
    # the mirror: as many units as quotas allow sit on the *other* die
    on_wrong = sum(1 for d in (0, 1) for u in plan_i["die_q"][d] if unit_die[u] != d)
    assert on_wrong == 2 * min(plan_d["quotas"])
    check_invariants(topo, plan_i, pi, 148)


def test_page_owner_for_dense_plans_is_the_majority_die_of_the_column():
    topo = inputs.synthetic_topo(die0_sms=70, seed=4)
    kw = dict(M=2048, N=2048, K=256, tile_m=256, tile_n=256, raster_group=4)
    plan = op.build_plan(topo, None, 148, op.default_policy(kind=op.DIE_COMPACT, **kw))
    pd = op.page_die_from_plan(plan, 256)
    ppt, ppc = 16, 2
    assert len(pd) == 8 * ppc * ppt
    unit_die = {u: d for d in (0, 1) for u in plan["die_q"][d]}
    for tn in range(8):
        votes = [sum(1 for tm in range(8) if unit_die[tm * 8 + tn] == d) for d in (0, 1)]
        want = 0 if votes[0] >= votes[1] else 1
        assert set(pd[tn * ppc * ppt:(tn + 1) * ppc * ppt]) == {want}
    # die 0 (70 of 148 SMs) owns the left columns, die 1 the right ones
    owners = [pd[tn * ppc * ppt] for tn in range(8)]
    assert owners == sorted(owners) and owners[0] == 0 and owners[-1] == 1
    # an affinity plan over such a packing keeps every unit of a column on the column's die
    n_pages = len(pd)
    amap = dict(chunk_bytes=4096, die_of_chunk=inputs.synthetic_chunk_die(2 * n_pages, seed=6))
    table = op.build_page_table(pd, amap)
    bop = op.operand(0, 0, 2, layout=op.LAYOUT_PAGED, page_table=table)
    pa = op.build_plan(topo, amap, 148, op.default_policy(kind=op.AFFINITY, b=bop, **kw))
    die_a = {u: d for d in (0, 1) for u in pa["die_q"][d]}
    agree = sum(1 for u in range(64) if die_a[u] == owners[u % 8])
    assert agree >= 56                                      # quotas may move a few units of the cut column


def test_page_table_views_share_pairs_and_survive_broken_pairs():
    doc = np.array([0, 1, 1, 0, 1, 1, 0, 0, 1, 0], dtype=np.uint8)      # pairs 2 and 3 break the pair rule
    amap = dict(chunk_bytes=4096, die_of_chunk=doc)
    table = op.build_page_table([0, 1, 1, 0, 0, 1, 1, 0], amap)
    # view 0 pages -> pairs 0,1,2,3 ; view 1 pages -> pairs 0,1,2,3
    assert table == [0, 1, 2, 3, 5, 4, 7, 6]
    assert len(set(table)) == 8


def test_packed_page_layout_by_hand():
    K, N = 32, 128
    B = np.arange(K * N, dtype=np.uint16).reshape(K, N)                 # B[k][n] = k*128 + n
    img = op.pack_weights(B, [3, 1], n_chunks=4)
    assert not img[0].any() and not img[2].any()
    page0 = img[3]                                                       # k16 = 0
    # element (n, k) at halfword (n//8)*128 + (k//8)*64 + (n%8)*8 + (k%8)
    for n, k in ((0, 0), (1, 0), (0, 1), (7, 7), (8, 0), (0, 8), (127, 15), (77, 13)):
        assert page0[(n // 8) * 128 + (k // 8) * 64 + (n % 8) * 8 + (k % 8)] == k * 128 + n
    assert img[1][(5 // 8) * 128 + (9 // 8) * 64 + 5 * 8 + 1] == (16 + 9) * 128 + 5   # k16 = 1


def test_quad_groups_follow_the_xor_hash():
    # a hash over chunk-index bits 0-3 and 5-8 (bit 4 free), as measured on B200
    tbl = inputs.synthetic_chunk_die(4096, seed=11, mask_bits=0x1EF)
    amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    groups = op.quad_groups(amap, free_bit=4)
    assert len(groups[0]) + len(groups[1]) == 4096 // 4          # every chunk is in exactly one group
    seen = set()
    for d in (0, 1):
        assert groups[d] == sorted(groups[d])
        for q in groups[d]:
            a = 3 if q % 4 == 0 else 1
            members = [q, q + a, q + 16, q + 16 + a]
            assert all(tbl[c] == d for c in members) and not (seen & set(members))
            seen |= set(members)
    assert len(seen) == 4096
    # a hash that also uses bit 4 breaks the groups: none survives (flipping bit 4 changes the die)
    bad = inputs.synthetic_chunk_die(4096, seed=11, mask_bits=0x1FF)
    assert op.quad_groups(dict(chunk_bytes=4096, die_of_chunk=bad), 4) == [[], []]
    # noise in one chunk removes exactly its group
    noisy = tbl.copy()
    noisy[37] ^= 1
    g2 = op.quad_groups(dict(chunk_bytes=4096, die_of_chunk=noisy), 4)
    assert len(g2[0]) + len(g2[1]) == 1023
    # page table: runs of four pages -> one group each, on the owner's die, pages in the order q, q+a, q+F, q+F+a
    page_die = [0] * 8 + [1] * 4 + [0] * 4
    table = op.build_page_table_quads(page_die, amap, 4)
    assert len(set(table)) == 16 and all(tbl[c] == d for c, d in zip(table, page_die))
    q = table[0]
    a = 3 if q % 4 == 0 else 1
    assert table[:4] == [q, q + a, q + 16, q + 16 + a] and table[0] == groups[0][0] and table[4] == groups[0][1]
    assert table[8] == groups[1][0] and table[12] == groups[0][2]


def test_page_table_matches_printed_remap_formula():
    """Eq. 1 (appendix on address remapping): page_phys = 2j + [parity((page_start + 2j) & MASK) xor P]
    when a chunk's die is parity((page_start + chunk) & MASK) and bit 0 is in MASK."""
    MASK, start = 0b1011_0110_1, 0x5A2C0                   # even start page, bit 0 in the mask
    par = lambda x: bin(x).count("1") & 1
    n_log = 4096
    doc = np.array([par((start + c) & MASK) for c in range(2 * n_log)], dtype=np.uint8)
    amap = dict(chunk_bytes=4096, die_of_chunk=doc)
    for P in (0, 1):
        table = op.build_page_table([P] * n_log, amap)
        want = [2 * j + (par((start + 2 * j) & MASK) ^ P) for j in range(n_log)]
        assert table == want


def test_closed_form_remap_equals_the_printed_formula_and_the_table():
    """Eq. 1 in closed form from a fitted 9-bit mask and one bit per 2 MiB page, against the printed formula with a
    16-bit MASK and a physical start page, and against the table built from the measured bits."""
    MASK, start = 0b0110_1001_1011_0110_1, 0x7A4C6        # bits above 8 end up in the per-page constants
    n_log = 6000                                            # 12000 chunks: 24 pages of 2 MiB
    doc = np.array([op._parity((start + c) & MASK) for c in range(2 * n_log)], dtype=np.uint8)
    amap = dict(chunk_bytes=4096, die_of_chunk=doc)
    first = start % 512                                     # the buffer's base inside its 2 MiB page (even)
    mask9 = MASK & 0x1FF
    c_bits, bad = op.fit_page_constants(amap, mask9, first)
    assert bad == 0 and len(set(c_bits)) == 2               # both constants occur: the high bits do matter
    for P in (0, 1):
        table = op.build_page_table([P] * n_log, amap)
        for j in list(range(0, 600)) + [n_log - 1, 2047, 2048, 4095, 4096]:
            want = 2 * j + (op._parity((start + 2 * j) & MASK) ^ P)          # the formula as printed
            assert op.page_from_hash(j, P, mask9, c_bits, first) == want == table[j]
            assert doc[want] == P
    # a wrong mask is caught by the fit
    assert op.fit_page_constants(amap, mask9 ^ 0b100, first)[1] > 1000


@pytest.mark.parametrize("first", [0, 4, 20, 508])
def test_closed_form_quad_groups_equal_the_enumeration(first):
    """r-th group of a die from the hash alone against the enumeration over the measured map."""
    mask, f = 0x1EF, 4                                      # bits 0-3 and 5-8 in the hash, bit 4 free (as on B200)
    n = 3000
    idx = np.arange(first, first + n)
    par = np.array([op._parity(int(i) & mask) for i in idx], dtype=np.uint8)
    c = (inputs.mix64_np((idx >> 9).astype(np.uint64) + np.uint64(3)) & np.uint64(1)).astype(np.uint8)
    doc = par ^ c
    amap = dict(chunk_bytes=4096, die_of_chunk=doc)
    c_bits, bad = op.fit_page_constants(amap, mask, first)
    assert bad == 0
    groups = op.quad_groups(amap, f, first)
    for d in (0, 1):
        assert len(groups[d]) > 300
        # the enumeration may stop a few groups early at the end of the buffer; compare all that it lists
        for r, q in enumerate(groups[d]):
            q2, a = op.quad_group_from_hash(r, d, mask, c_bits, f, first)
            assert q2 == q and a == (3 if ((first + q) & 3) == 0 else 1)
            assert all(doc[x] == d for x in (q, q + a, q + 16, q + 16 + a))
    # page table from the closed form = page table from the enumeration
    page_die = [0] * 8 + [1] * 8 + [0] * 4
    table = op.build_page_table_quads(page_die, amap, f, first)
    nxt, want = [0, 0], []
    for r4 in range(len(page_die) // 4):
        d = page_die[4 * r4]
        q, a = op.quad_group_from_hash(nxt[d], d, mask, c_bits, f, first)
        nxt[d] += 1
        want += [q, q + a, q + 16, q + 16 + a]
    assert table == want


TOY24 = dict(n_sm=24, n_tpc=12, n_gpc=3, n_die=2, tpc=[s // 2 for s in range(24)],
             gpc=[0] * 10 + [1] * 8 + [2] * 4 + [2, 2], die=[0] * 18 + [1] * 6,
             is_random=[0] * 22 + [1, 1], gpc_die=[0, 0, 1])


def test_cluster_aware_sets_by_hand():
    """A 24-SM toy chip: GPC 0 has five TPCs (SMs 0-9), GPC 1 four (10-17), GPC 2 two (18-21) plus one random TPC
    (22, 23) that never hosts clusters larger than 2.  Die 0 = GPCs 0 and 1."""
    base = dict(kind=op.DIE_COMPACT, M=1, N=1, K=1)
    # budget 12, clusters of 4.  Die 0 first: GPC 0 blocks [0-3] [4-7] (8, 9 left aside), GPC 1 blocks [10-13] [14-17];
    # dealt round-robin: [0-3], [10-13], [4-7] -> 12 SMs, three clusters of four.
    S4 = op.select_sms(TOY24, 12, op.default_policy(cluster_size=4, **base))
    assert S4 == [0, 1, 2, 3, 4, 5, 6, 7, 10, 11, 12, 13]
    assert op.cluster_capacity(TOY24, S4, 4) == 3
    # the TPC-wise rule takes three TPCs from either GPC: six SMs each, room for only one cluster of four per GPC
    S1 = op.select_sms(TOY24, 12, op.default_policy(**base))
    assert S1 == [0, 1, 2, 3, 4, 5, 10, 11, 12, 13, 14, 15]
    assert op.cluster_capacity(TOY24, S1, 4) == 2
    # budget 20, clusters of 8: blocks [0-7] and [10-17]; GPC 2 (four normal SMs) has no block of eight; the budget is
    # filled with the normal SMs left aside, die 0 first (8, 9), then die 1 (18, 19)
    S8 = op.select_sms(TOY24, 20, op.default_policy(cluster_size=8, **base))
    assert S8 == list(range(20))
    assert op.cluster_capacity(TOY24, S8, 8) == 2
    # random SMs come last: budget 23 leaves out SM 23, budget 22 takes no random SM at all
    assert op.select_sms(TOY24, 22, op.default_policy(cluster_size=4, **base)) == list(range(22))
    assert op.select_sms(TOY24, 23, op.default_policy(cluster_size=4, **base)) == list(range(23))
    # a budget that is no multiple of the cluster size: two whole blocks ([0-3], [10-13]; a third does not fit), then
    # the lowest normal SMs not yet taken (4, 5)
    S10 = op.select_sms(TOY24, 10, op.default_policy(cluster_size=4, **base))
    assert S10 == [0, 1, 2, 3, 4, 5, 10, 11, 12, 13] and op.cluster_capacity(TOY24, S10, 4) == 2
    # Section 7.3's arithmetic: twelve SMs of one GPC form three clusters of four but one cluster of eight
    one_gpc = dict(TOY24, gpc=[0] * 24, is_random=[0] * 24)
    assert op.cluster_capacity(one_gpc, list(range(12)), 4) == 3
    assert op.cluster_capacity(one_gpc, list(range(12)), 8) == 1
    # GPC spread with clusters of 4: blocks dealt over the GPCs of both dies: [0-3], [10-13], [18-21]
    Ss = op.select_sms(TOY24, 12, op.default_policy(cluster_size=4, sm_select=1, **base))
    assert Ss == [0, 1, 2, 3, 10, 11, 12, 13, 18, 19, 20, 21]


def test_cluster_aware_sets_on_synthetic_b200():
    topo = inputs.synthetic_topo(die0_sms=70, seed=3)
    n_random = int(sum(topo["is_random"]))
    assert n_random > 0
    for c in (4, 8):
        for b in (32, 64, 72, 100, 148):
            for sel in (0, 1):
                pol = op.default_policy(kind=op.DIE_COMPACT, M=4096, N=4096, K=4096, cluster_size=c, sm_select=sel)
                S = op.select_sms(topo, b, pol)
                assert len(S) == b == len(set(S))
                cap = op.cluster_capacity(topo, S, c)
                best = op.cluster_capacity(topo, list(range(148)), c)
                assert cap == min(b // c, best) or (sel == 0 and cap >= min(b // c, best) - 1)
                # never worse than the TPC-wise set of the same budget, and random SMs only when nothing else is left
                S0 = op.select_sms(topo, b, op.default_policy(kind=op.DIE_COMPACT, M=1, N=1, K=1, sm_select=sel))
                assert cap >= op.cluster_capacity(topo, S0, c)
                if b <= 148 - n_random:
                    assert not any(topo["is_random"][s] for s in S)
                plan = op.build_plan(topo, None, b, pol)
                check_invariants(topo, plan, pol, b)


@pytest.mark.parametrize("seed,invert", [(1, 0), (2, 0), (3, 1), (4, 1)])
def test_affinity_greedy_pass_keeps_a_full_dies_first_takers(seed, invert):
    """What the greedy pass must amount to: until a die is full every unit gets the die it prefers, afterwards everything
    goes to the other one; the quotas add up to the unit count, so at most one die has more takers than quota, and it
    keeps exactly its first takers in the order (|margin| descending, raster index ascending)."""
    topo = inputs.synthetic_topo(die0_sms=70, seed=seed)
    M, N, K = 16, 128 * 300, 64
    rng = np.random.default_rng(seed)
    tbl = rng.integers(0, 2, size=M * N * 4 // 4096, dtype=np.uint8)
    tbl[rng.random(tbl.size) < 0.3] = 0                      # more bytes on die 0 than its quota of units
    amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    pol = op.default_policy(kind=op.AFFINITY, M=M, N=N, K=K, tile_m=16, tile_n=128, raster_group=1, invert_affinity=invert,
                            c=op.operand(0, N * 4, 4))
    plan = op.build_plan(topo, amap, 148, pol)
    n_u, q = plan["n_units"], plan["quotas"]
    R = op.raster_order(1, 300, 1, 1)
    die_of = {u: d for d in (0, 1) for u in plan["die_q"][d]}
    takers = {0: [], 1: []}
    for i, u in enumerate(R):
        l0, l1 = op.unit_local_bytes(pol, amap, u)
        m = (l1 - l0) if invert else (l0 - l1)
        pref = 0 if m > 0 else 1 if m < 0 else op.band_die(i, n_u, q[0], 300)
        takers[pref].append((-abs(m), i, u))
    over = [d for d in (0, 1) if len(takers[d]) > q[d]]
    assert len(over) == 1                                    # the case is built so that one die is oversubscribed
    d = over[0]
    kept = [u for _, _, u in sorted(takers[d])[:q[d]]]
    assert sorted(plan["die_q"][d]) == sorted(kept)
    assert all(die_of[u] == 1 - d for _, _, u in takers[1 - d])

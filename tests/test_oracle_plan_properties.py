"""Property-based checks of the CPU plan builder: for any chip, budget and policy the invariants that
the paper's scheduling principles imply must hold (every unit exactly once, lists stay on their die,
quotas proportional to the SM counts)."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import plan as op
from paper_2609_24270_b200 import inputs
from tests.test_oracle_plan import check_invariants


@settings(max_examples=120, deadline=None)
@given(die0=st.sampled_from([66, 70, 72, 74, 78]), seed=st.integers(1, 50), kind=st.sampled_from([op.OBLIVIOUS, op.DIE_COMPACT]),
       b=st.integers(1, 148), tiles=st.tuples(st.integers(1, 9), st.integers(1, 9)), ksp=st.integers(1, 3),
       g=st.integers(1, 5), sub_seed=st.integers(0, 5), sel=st.integers(0, 1), unplaced=st.booleans())
def test_plan_invariants_hold_for_any_policy(die0, seed, kind, b, tiles, ksp, g, sub_seed, sel, unplaced):
    topo = inputs.synthetic_topo(die0_sms=die0, seed=seed)
    if unplaced:
        topo["gpc"] = topo["gpc"].copy()
        topo["gpc"][topo["is_random"] == 1] = -1
    pol = op.default_policy(kind=kind, seed=sub_seed if kind == op.OBLIVIOUS else 0, M=tiles[0] * 128, N=tiles[1] * 256,
                            K=64 * ksp * 2, k_splits=ksp, raster_group=g, sm_select=sel)
    plan = op.build_plan(topo, None, b, pol)
    check_invariants(topo, plan, pol, b)
    n_u = tiles[0] * tiles[1] * ksp
    assert plan["n_units"] == n_u
    if kind == op.DIE_COMPACT:
        n_d = plan["die_sm_count"]
        assert [len(q) for q in plan["die_q"]] == op.quotas(n_u, n_d, b)
        for d in (0, 1):
            if n_d[d]:
                lens = [len(plan["sm_q"][s]) for s in range(b) if plan["sm_die"][s] == d]
                assert max(lens) - min(lens) <= 1
        # each die's queue is in raster order
        pos = {u: i for i, u in enumerate(op.raster_order(tiles[0], tiles[1], ksp, g))}
        for q in plan["die_q"]:
            assert [pos[u] for u in q] == sorted(pos[u] for u in q)
    exp = op.export(plan)
    assert len(exp) == 16 + 3 * b + 5 + n_u + b + 1 + n_u + 148


@settings(max_examples=60, deadline=None)
@given(die0=st.sampled_from([70, 74]), seed=st.integers(1, 20), pairs=st.integers(1, 74), units=st.tuples(st.integers(1, 12), st.integers(1, 12)),
       kind=st.sampled_from([op.OBLIVIOUS, op.DIE_COMPACT]), sel=st.integers(0, 1))
def test_pair_lists_are_balanced_per_tpc(die0, seed, pairs, units, kind, sel):
    topo = inputs.synthetic_topo(die0_sms=die0, seed=seed)
    b = 2 * pairs
    pol = op.default_policy(kind=kind, M=units[0] * 256, N=units[1] * 256, K=128, tile_m=256, tile_n=256, raster_group=2,
                            sm_select=sel, pair_lists=1)
    plan = op.build_plan(topo, None, b, pol)
    check_invariants(topo, plan, pol, b)
    groups = [list(range(b))] if kind == op.OBLIVIOUS else [[s for s in range(b) if plan["sm_die"][s] == d] for d in (0, 1)]
    for slots in groups:
        if not slots:
            continue
        per_tpc = [len(plan["sm_q"][slots[2 * j]]) + len(plan["sm_q"][slots[2 * j + 1]]) for j in range(len(slots) // 2)]
        assert max(per_tpc) - min(per_tpc) <= 1
        for j in range(len(slots) // 2):
            lo, hi = len(plan["sm_q"][slots[2 * j]]), len(plan["sm_q"][slots[2 * j + 1]])
            assert 0 <= lo - hi <= 1                      # the lower SM goes first

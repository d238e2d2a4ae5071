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

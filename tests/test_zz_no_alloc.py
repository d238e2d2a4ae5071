"""The allocation-free entry point.  Its callers are processes that cannot obtain device memory at
the moment they need the GEMM: a server whose own pool already holds every free byte of the GPU (cudaMalloc
fails there), a request loop that must not call an allocator, code running after a framework's "no more
allocations" point.  For them the split-K workspace is a fixed array inside the library.  Checked here
against the ordinary entry point and against the fp64 oracle on the same inputs, twice in a row (the
workspace is shared and keeps old contents), and the second call is checked to take no device memory."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs

pytestmark = pytest.mark.gpu


def test_noalloc_matches_regular_entry_point_and_oracle_twice():
    M, N, K, ksp = 16, 2048, 2048, 4
    topo = ag.topo_discover(ag.AG_TOPO_CENSUS | ag.AG_TOPO_LATENCY)
    A, B = inputs.gemm_inputs(M, N, K, seed=5)
    A2, B2 = inputs.gemm_inputs(M, N, K, seed=9)
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16,
                                                                tile_n=128, k_splits=ksp))
    stream = torch.cuda.current_stream().cuda_stream
    for call, (a_bits, b_bits) in enumerate(((A, B), (A2, B2))):     # two calls in a row, different data
        dA = torch.from_numpy(a_bits.view(np.int16).copy()).cuda()
        dB = torch.from_numpy(b_bits.view(np.int16).copy()).cuda()
        c_ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        c_new = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), c_ref.data_ptr(), M, N, K, plan, stream)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        free_before = torch.cuda.mem_get_info()[0]
        launches_before = ag.kernel_launch_count()
        ag.gemm_persistent_noalloc(dA.data_ptr(), dB.data_ptr(), c_new.data_ptr(), M, N, K, plan, stream)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        # two kernels of the library (the GEMM and the adding-up of the k-split slices), nothing else
        assert ag.kernel_launch_count() == launches_before + 2
        if call == 1:
            # the first call on a device may make the driver place the library's kernels and the workspace;
            # from the second call on the free device memory must not move
            assert torch.cuda.mem_get_info()[0] == free_before
        ref = c_ref.cpu().numpy().astype(np.float64)
        got = c_new.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        # same tolerance as the GEMM parity tests: relative Frobenius <= 1e-4, max abs <= 1e-2
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-4
        assert np.abs(got - ref).max() <= 1e-2
        want = og.gemm_blocked(a_bits, b_bits)                          # fp64 oracle
        assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-4
        assert np.abs(got - want).max() <= 1e-2


def test_noalloc_refuses_problems_beyond_the_builtin_workspace():
    topo = ag.topo_discover(ag.AG_TOPO_CENSUS | ag.AG_TOPO_LATENCY)
    M, N, K, ksp = 32, 8192, 4096, 16                         # 32 * 8192 * 16 * 4 B = 16 MiB > 8 MiB
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=32,
                                                                tile_n=128, k_splits=ksp))
    t = torch.zeros(K * N, dtype=torch.int16, device="cuda")
    c = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    st = ag.lib().gemm_persistent_noalloc(t.data_ptr(), t.data_ptr(), c.data_ptr(), M, N, K, plan.handle, None)
    assert st == ag.AG_ERR_ARG
    dense = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(M=256, N=256, K=256))
    st = ag.lib().gemm_persistent_noalloc(t.data_ptr(), t.data_ptr(), c.data_ptr(), 256, 256, 256, dense.handle, None)
    assert st == ag.AG_ERR_ARG


def test_launches_are_refused_while_the_stream_is_capturing():
    """A launch carries a per-launch epoch in its kernel parameters, which a replayed graph would repeat: every
    gemm_persistent* call on a capturing stream returns AG_ERR_ARG and records nothing."""
    M, N, K = 16, 1024, 512
    topo = ag.topo_discover(ag.AG_TOPO_CENSUS | ag.AG_TOPO_LATENCY)
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16,
                                                                tile_n=128, k_splits=2))
    dense = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(M=256, N=256, K=256))
    a = torch.zeros(256 * 512, dtype=torch.int16, device="cuda")
    b = torch.zeros(K * N, dtype=torch.int16, device="cuda")
    c = torch.zeros(256 * N, dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    launches = ag.kernel_launch_count()
    with torch.cuda.stream(s):
        g.capture_begin()
        try:
            st1 = ag.lib().gemm_persistent_noalloc(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, plan.handle, s.cuda_stream)
            st2 = ag.lib().gemm_persistent(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, plan.handle, s.cuda_stream)
            st3 = ag.lib().gemm_persistent(a.data_ptr(), b.data_ptr(), c.data_ptr(), 256, 256, 256, dense.handle, s.cuda_stream)
        finally:
            g.capture_end()
    assert st1 == st2 == st3 == ag.AG_ERR_ARG
    assert ag.kernel_launch_count() == launches
    torch.cuda.synchronize()
    # the same calls outside capture still work
    ag.gemm_persistent_noalloc(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, plan, 0)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK

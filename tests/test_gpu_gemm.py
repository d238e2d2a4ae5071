"""gemm_persistent through the C ABI against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import check_close, device_topo, run_gemm, to_dev_bf16

pytestmark = pytest.mark.gpu


def plan_for(M, N, K, b=None, **kw):
    topo = device_topo()
    b = topo.n_sm if b is None else b
    return ag.sched_build(topo, None, b, ag.make_policy(M=M, N=N, K=K, **kw))


@pytest.mark.parametrize("shape", [(128, 256, 64), (128, 256, 256), (256, 512, 128), (1024, 1024, 1024)])
def test_integer_inputs_bit_exact(shape):
    """Entries in {-2..2}: every partial sum is a small integer, so fp32 accumulation is exact in
    any order and the result must equal the oracle bit for bit.  Pins tile indexing, swizzles,
    k-slab order and epilogue addressing."""
    M, N, K = shape
    A = inputs.small_int_bf16(M, K, seed=1)
    B = inputs.small_int_bf16(K, N, seed=2)
    plan = plan_for(M, N, K)
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))


def test_one_hot_localises_addressing():
    M, N, K = 256, 512, 192
    B = inputs.uniform_bf16(K, N, seed=8)
    A = np.zeros((M, K), dtype=np.float32)
    A[130, 77] = 1.0
    A[5, 191] = 2.0
    Ab = inputs.f32_to_bf16_bits(A)
    C = run_gemm(Ab, B, plan_for(M, N, K))
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(Ab, B))


@pytest.mark.parametrize("shape", [(1024, 1024, 1024), (1000, 1000, 1000), (333, 776, 520), (1, 8, 8), (129, 264, 72),
                                   (2048, 2304, 1536)])
def test_uniform_inputs_within_tolerance(shape):
    M, N, K = shape
    A, B = inputs.gemm_inputs(M, N, K)
    C = run_gemm(A, B, plan_for(M, N, K, kind=ag.AG_DIE_COMPACT, raster_group=2))
    check_close(C, og.gemm_blocked(A, B))


@pytest.mark.parametrize("tile_n", [64, 128, 256])
@pytest.mark.parametrize("k_splits", [1, 4])
def test_tile_widths_and_split_k(tile_n, k_splits):
    M, N, K = 512, 768, 1024
    A, B = inputs.gemm_inputs(M, N, K, seed=77)
    C = run_gemm(A, B, plan_for(M, N, K, tile_n=tile_n, k_splits=k_splits))
    check_close(C, og.gemm_blocked(A, B))
    Ai, Bi = inputs.small_int_bf16(M, K, 3), inputs.small_int_bf16(K, N, 4)
    Ci = run_gemm(Ai, Bi, plan_for(M, N, K, tile_n=tile_n, k_splits=k_splits))
    assert np.array_equal(Ci.astype(np.float64), og.gemm_blocked(Ai, Bi))


@pytest.mark.parametrize("kind", [ag.AG_OBLIVIOUS, ag.AG_DIE_COMPACT])
@pytest.mark.parametrize("b", [1, 16, 37, 74, 148])
@pytest.mark.parametrize("static", [1, 0])
def test_sm_budgets_policies_and_dynamic_queues(kind, b, static):
    M, N, K = 1024, 1536, 512
    A, B = inputs.small_int_bf16(M, K, 5), inputs.small_int_bf16(K, N, 6)
    plan = plan_for(M, N, K, b=b, kind=kind, static_assign=static, seed=0)
    plan.reset_record()
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    owner, count = plan.tile_record()
    assert (count == 1).all()                               # every unit ran exactly once
    p = plan.parsed()
    assert set(owner) <= set(p["sm_list"])                  # only planned SMs did any work
    if static:
        want = np.empty(p["n_units"], dtype=np.int32)
        for slot in range(b):
            want[p["sm_q"][p["sm_q_off"][slot]:p["sm_q_off"][slot + 1]]] = p["sm_list"][slot]
        assert np.array_equal(owner, want)                  # the SM the plan names ran the unit


def test_random_subset_and_repeat_launches():
    M, N, K = 1024, 1024, 256
    A, B = inputs.small_int_bf16(M, K, 9), inputs.small_int_bf16(K, N, 10)
    want = og.gemm_blocked(A, B)
    plan = plan_for(M, N, K, b=32, seed=5)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    for _ in range(5):                                      # epochs: claim flags reset themselves
        dC.fill_(float("nan"))
        ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), want)


def test_non_default_stream():
    M, N, K = 512, 512, 512
    A, B = inputs.gemm_inputs(M, N, K, seed=4)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        C = run_gemm(A, B, plan_for(M, N, K), stream=s)
    check_close(C, og.gemm_blocked(A, B))


def test_rejects_mismatched_shapes_and_alignment():
    plan = plan_for(256, 256, 256)
    t = torch.zeros(1 << 20, dtype=torch.int16, device="cuda")
    c = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    L = ag.lib()
    assert L.gemm_persistent(t.data_ptr(), t.data_ptr(), c.data_ptr(), 256, 256, 128, plan.handle, None) == ag.AG_ERR_ARG
    assert L.gemm_persistent(t.data_ptr() + 2, t.data_ptr(), c.data_ptr(), 256, 256, 256, plan.handle, None) == ag.AG_ERR_ARG
    with pytest.raises(ag.AgError):
        p2 = plan_for(256, 252, 256)
        ag.gemm_persistent(t.data_ptr(), t.data_ptr(), c.data_ptr(), 256, 252, 256, p2)


def test_full_size_one_block_tiles_sampled_against_oracle():
    """8192^3 with one 128 x 256 tile per block (the kernel used for arbitrary SM sets); the
    headline configuration with block pairs is covered in test_gpu_fullsize.py."""
    M = N = K = 8192
    A, B = inputs.gemm_inputs(M, N, K)
    plan = plan_for(M, N, K, kind=ag.AG_DIE_COMPACT, raster_group=16)
    plan.reset_record()
    C = run_gemm(A, B, plan)
    rng = np.random.default_rng(0)
    rows, cols = rng.integers(0, M, 200), rng.integers(0, N, 200)
    rows[:4], cols[:4] = [0, M - 1, 0, M - 1], [0, 0, N - 1, N - 1]
    ref = og.gemm_entries(A, B, rows, cols)
    got = C[rows, cols].astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-2
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-4
    blk = og.gemm_block(A, B, 8064, 8192, 7936, 8192)       # the last tile
    check_close(C[8064:8192, 7936:8192], blk)
    owner, count = plan.tile_record()
    assert (count == 1).all()


@pytest.mark.parametrize("shape", [(256, 256, 64), (512, 768, 256), (1024, 1024, 1024), (1000, 776, 520), (2048, 2304, 1536)])
def test_two_cta_units_integer_exact(shape):
    """256 x 256 units computed by pairs of thread blocks (full-chip plans)."""
    M, N, K = shape
    A, B = inputs.small_int_bf16(M, K, 21), inputs.small_int_bf16(K, N, 22)
    plan = plan_for(M, N, K, tile_m=256, tile_n=256, kind=ag.AG_DIE_COMPACT, raster_group=2)
    plan.reset_record()
    for _ in range(2):
        C = run_gemm(A, B, plan)
        assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    owner, count = plan.tile_record()
    assert (count == 2).all() and set(owner) <= set(plan.parsed()["sm_list"])


def test_two_cta_units_uniform_and_rejections():
    M, N, K = 1024, 1536, 2048
    A, B = inputs.gemm_inputs(M, N, K, seed=13)
    C = run_gemm(A, B, plan_for(M, N, K, tile_m=256, tile_n=256))
    check_close(C, og.gemm_blocked(A, B))
    topo = device_topo()
    with pytest.raises(ag.AgError):                         # a random subset is not made of whole TPCs: no pair lists ...
        ag.sched_build(topo, None, 37, ag.make_policy(M=M, N=N, K=K, tile_m=256, tile_n=256, seed=3))
    odd = ag.sched_build(topo, None, 37, ag.make_policy(M=M, N=N, K=K, tile_m=256, tile_n=256, seed=3, pair_lists=0))
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    st = ag.lib().gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, odd.handle, None)
    assert st == ag.AG_ERR_ARG                              # ... and no block pairs either


@pytest.mark.parametrize("b,sm_select", [(16, 0), (64, 0), (74, 0), (64, 1), (100, 1)])
def test_two_cta_units_on_sub_budgets_of_whole_tpcs(b, sm_select):
    """Die-compact and GPC-spread sets hold whole TPCs, so block pairs can run on them."""
    M, N, K = 1024, 1536, 512
    A, B = inputs.small_int_bf16(M, K, 31), inputs.small_int_bf16(K, N, 32)
    plan = plan_for(M, N, K, b=b, tile_m=256, tile_n=256, kind=ag.AG_DIE_COMPACT, sm_select=sm_select, raster_group=2)
    plan.reset_record()
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    owner, count = plan.tile_record()
    assert (count == 1).all() and set(owner) <= set(plan.parsed()["sm_list"])


def test_bounded_wait_gives_up_and_leaves_the_device_usable():
    """Every device-side wait of the library has a limit; here one is made to run out on purpose
    (a barrier that nothing signals, 2 ms limit): the kernel returns AG_ERR_TIMEOUT, nothing hangs."""
    st, waited = ag.wait_probe(2_000_000)
    assert st == ag.AG_ERR_TIMEOUT
    assert 2_000_000 <= waited < 200_000_000
    assert ag.lib().ag_wait_probe(0, None) == ag.AG_ERR_ARG
    A, B = inputs.small_int_bf16(256, 64, 1), inputs.small_int_bf16(64, 256, 2)
    C = run_gemm(A, B, plan_for(256, 256, 64))               # the context still works
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))


def packed_dense_setup(M, N, K, raster_group=2, integer=True, seed=51):
    topo = device_topo()
    if integer:
        A, B = inputs.small_int_bf16(M, K, seed), inputs.small_int_bf16(K, N, seed + 1)
    else:
        A, B = inputs.gemm_inputs(M, N, K, seed=seed)
    kw = dict(M=M, N=N, K=K, tile_m=256, tile_n=256, raster_group=raster_group, pair_lists=1)
    plan_d = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
    dst_bytes = 2 * K * ((N + 255) // 256 * 256) * 2 + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dB = to_dev_bf16(B)
    packed = ag.pack_weights(dB.data_ptr(), K, N, plan_d, amap, dst.data_ptr(), dst_bytes)
    return topo, A, B, kw, plan_d, dst, amap, packed


@pytest.mark.parametrize("shape", [(256, 256, 64), (1024, 1024, 512), (1000, 776, 192), (2048, 2304, 1536)])
def test_block_pairs_over_die_packed_b_integer_exact(shape):
    M, N, K = shape
    topo, A, B, kw, plan_d, dst, amap, packed = packed_dense_setup(M, N, K)
    dA = to_dev_bf16(A)
    ref = og.gemm_blocked(A, B)
    for _ in range(2):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan_d)
        torch.cuda.synchronize()
        assert plan_d.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref)


def test_die_packed_b_pages_and_affinity_plan_match_oracle():
    from oracle import plan as op
    M, N, K = 2048, 2048, 256
    topo, A, B, kw, plan_d, dst, amap, packed = packed_dense_setup(M, N, K, raster_group=4, integer=False)
    tbl = amap.export()
    o_plan = op.build_plan(topo.as_dict(), None, topo.n_sm, op.default_policy(kind=op.DIE_COMPACT, **kw))
    page_die = op.page_die_from_plan(o_plan, K)
    f = packed.group_free_bit()
    o_amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    want_table = (op.build_page_table(page_die, o_amap) if f < 0 else
                  op.build_page_table_quads(page_die, o_amap, f, first=(dst.data_ptr() // 4096) % 512))
    got_table = packed.page_table()
    assert np.array_equal(got_table, np.array(want_table, dtype=np.int32))
    n_chunks = int(got_table.max()) + 1
    got_img = dst[: n_chunks * 4096].cpu().numpy().view(np.uint16).reshape(n_chunks, 2048)
    assert np.array_equal(got_img, op.pack_weights(B, want_table, n_chunks))
    # affinity over the packed B panels: bytewise equal to the oracle's plan, and the GEMM under it is right
    bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=got_table)
    plan_a = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, b=bop, **kw))
    o_aff = op.build_plan(topo.as_dict(), dict(chunk_bytes=4096, die_of_chunk=tbl), topo.n_sm,
                          op.default_policy(kind=op.AFFINITY, b=op.operand(0, 0, 2, op.LAYOUT_PAGED, want_table), **kw))
    assert plan_a.export().tobytes() == op.export(o_aff).tobytes()
    dA = to_dev_bf16(A)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan_a)
    torch.cuda.synchronize()
    assert plan_a.last_status() == ag.AG_OK
    check_close(dC.cpu().numpy(), og.gemm_blocked(A, B))


@pytest.mark.parametrize("blocks", [100, 37, 1])
@pytest.mark.parametrize("static", [1, 0])
def test_fewer_blocks_than_planned_sms_still_complete_the_plan(blocks, static):
    """Planned SMs that get no thread block: their lists are taken over (static) or the queues are
    drained by the blocks that exist (dynamic).  Every unit still runs exactly once."""
    M, N, K = 1024, 1536, 256
    A, B = inputs.small_int_bf16(M, K, 41), inputs.small_int_bf16(K, N, 42)
    plan = plan_for(M, N, K, kind=ag.AG_DIE_COMPACT, static_assign=static, tile_n=128)
    plan.set_grid(blocks)
    plan.reset_record()
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    owner, count = plan.tile_record()
    assert (count == 1).all() and len(set(owner)) <= blocks
    if static:
        p = plan.parsed()
        with_work = sum(1 for s in range(p["b"]) if p["sm_q_off"][s + 1] > p["sm_q_off"][s])
        assert plan.adopted() >= min(with_work, p["b"]) - blocks   # at least the lists nobody was there for
    pair = plan_for(M, N, K, tile_m=256, tile_n=256)
    with pytest.raises(ag.AgError):
        pair.set_grid(64)
        run_gemm(A, B, pair)


@pytest.mark.parametrize("tile_m", [128, 256])
def test_unit_timeline(tile_m):
    M, N, K = 2048, 2048, 1024
    A, B = inputs.small_int_bf16(M, K, 61), inputs.small_int_bf16(K, N, 62)
    plan = plan_for(M, N, K, tile_m=tile_m, tile_n=256, kind=ag.AG_DIE_COMPACT)
    with pytest.raises(ag.AgError):
        plan.unit_times()                                   # tracing is off by default
    plan.trace(True)
    C = run_gemm(A, B, plan)
    assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    t0, t1 = plan.unit_times()
    assert (t0 > 0).all() and (t1 > t0).all()
    span_us = (int(t1.max()) - int(t0.min())) / 1e3
    assert 1.0 < span_us < 5000.0
    # the units of one SM's list run one after the other
    p = plan.parsed()
    lst = p["sm_q"][p["sm_q_off"][0]:p["sm_q_off"][1]]
    if tile_m == 128 and len(lst) > 1:
        assert all(t1[lst[i]] <= t1[lst[i + 1]] for i in range(len(lst) - 1))
    plan.trace(False)


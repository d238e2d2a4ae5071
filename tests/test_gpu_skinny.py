"""Decode-shaped GEMM (M <= 32): row-major and die-packed weights against the fp64 oracle, the
packing against the oracle's page table and page layout."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from oracle import plan as op
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import check_close, device_topo, oracle_policy, to_dev_bf16

pytestmark = pytest.mark.gpu


def run_rowmajor(A, B, plan):
    M, K = A.shape
    N = B.shape[1]
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    return dC.cpu().numpy()


@pytest.mark.parametrize("M,tile_m", [(16, 16), (32, 32), (5, 16), (20, 32), (1, 16)])
@pytest.mark.parametrize("k_splits", [1, 4])
def test_rowmajor_weights_integer_exact(M, tile_m, k_splits):
    N, K = 1024, 1024
    A, B = inputs.small_int_bf16(M, K, 11), inputs.small_int_bf16(K, N, 12)
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=tile_m,
                                                                tile_n=128, k_splits=k_splits))
    plan.reset_record()
    for _ in range(2):                                      # second launch: nothing is left over from the first
        C = run_rowmajor(A, B, plan)
        assert np.array_equal(C.astype(np.float64), og.gemm_blocked(A, B))
    owner, count = plan.tile_record()
    assert (count == 2).all()


@pytest.mark.parametrize("shape", [(16, 8192, 8192, 16), (32, 4096, 4096, 8), (16, 1000, 520, 2), (7, 264, 72, 1),
                                   (16, 384, 1280, 1), (32, 256, 1344, 2)])
@pytest.mark.parametrize("in_memory", [0, 1])
def test_rowmajor_weights_uniform(shape, in_memory):
    M, N, K, ksp = shape
    A, B = inputs.gemm_inputs(M, N, K, seed=31)
    topo = device_topo()
    for b in (37, topo.n_sm):
        plan = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, splitk_in_memory=in_memory,
                                                            tile_m=16 if M <= 16 else 32, tile_n=128, k_splits=ksp))
        for _ in range(2):
            check_close(run_rowmajor(A, B, plan), og.gemm_blocked(A, B))


@pytest.mark.parametrize("M,tile_m", [(64, 64), (48, 64), (128, 128), (100, 128), (33, 64)])
@pytest.mark.parametrize("k_splits,in_memory", [(1, 0), (4, 0), (4, 1)])
def test_up_to_128_activation_rows_integer_exact(M, tile_m, k_splits, in_memory):
    """64 and 128 activation rows on the MMA's N side (one MMA-issuing thread, four weight stages): bit-exact on integer
    inputs, row-major and die-packed weights, full chip and 37 SMs; 128 rows need policy.decode_shaped."""
    N, K = 1024, 1024
    A, B = inputs.small_int_bf16(M, K, 21), inputs.small_int_bf16(K, N, 22)
    want = og.gemm_blocked(A, B)
    topo = device_topo()
    for b in (topo.n_sm, 37):
        plan = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=tile_m, tile_n=128,
                                                            k_splits=k_splits, splitk_in_memory=in_memory, decode_shaped=1))
        for _ in range(2):
            assert np.array_equal(run_rowmajor(A, B, plan).astype(np.float64), want)
    dst_bytes = 2 * K * N * 2 + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    packed = ag.pack_weights(dB.data_ptr(), K, N, plan, amap, dst.data_ptr(), dst_bytes)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    assert np.array_equal(dC.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("shape", [(64, 8192, 8192, 4), (128, 4096, 4096, 8), (96, 1000, 520, 2), (128, 384, 1344, 1)])
def test_up_to_128_activation_rows_uniform(shape):
    M, N, K, ksp = shape
    A, B = inputs.gemm_inputs(M, N, K, seed=41)
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, splitk_in_memory=1, decode_shaped=1,
                                                                tile_m=64 if M <= 64 else 128, tile_n=128, k_splits=ksp, overlap_launches=1))
    for _ in range(3):
        check_close(run_rowmajor(A, B, plan), og.gemm_blocked(A, B))


def test_workspace_split_k_is_bit_reproducible():
    """splitk_in_memory = 0: the k-split slices are added in ascending split order, so the bits of C do not depend on
    which SMs ran which unit, nor on the order in which the units finished: the same C, bit for bit, from the full
    chip and from 37 SMs, from die-compact and oblivious plans, with and without overlapping launches and from one call
    to the next."""
    M, N, K, ksp = 16, 2048, 4096, 8
    A, B = inputs.gemm_inputs(M, N, K, seed=77)
    topo = device_topo()
    outs = []
    for b, kind, overlap in ((topo.n_sm, ag.AG_DIE_COMPACT, 0), (topo.n_sm, ag.AG_DIE_COMPACT, 1), (37, ag.AG_DIE_COMPACT, 0),
                             (topo.n_sm, ag.AG_OBLIVIOUS, 0), (53, ag.AG_OBLIVIOUS, 0)):
        plan = ag.sched_build(topo, None, b, ag.make_policy(kind=kind, M=M, N=N, K=K, tile_m=16, tile_n=128, k_splits=ksp,
                                                            seed=3 if kind == ag.AG_OBLIVIOUS else 0, overlap_launches=overlap))
        for _ in range(3):
            outs.append(run_rowmajor(A, B, plan))
    check_close(outs[0], og.gemm_blocked(A, B))
    for o in outs[1:]:
        assert o.tobytes() == outs[0].tobytes()


def test_overlapping_launches_in_a_dependent_chain():
    """overlap_launches = 1 in the situation it is meant for: the activations of every call are made from the result
    of the call before (here by a cast on the same stream).  Weights are permutation matrices, so the end of the chain
    is the input with its columns permuted - exactly."""
    M, N, K, ksp = 16, 2048, 2048, 4
    topo = device_topo()
    rng = np.random.default_rng(5)
    perms = [rng.permutation(N) for _ in range(6)]
    Ws = []
    for pm in perms:
        W = np.zeros((K, N), dtype=np.float32)
        W[np.arange(K), pm] = 1.0                       # (A W)[:, pm[k]] = A[:, k]
        Ws.append(to_dev_bf16(inputs.f32_to_bf16_bits(W)))
    A0 = rng.integers(-8, 9, size=(M, K)).astype(np.float32)
    x = torch.from_numpy(A0).cuda().to(torch.bfloat16)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    plans = [ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16, tile_n=128,
                                                          k_splits=ksp, splitk_in_memory=1, overlap_launches=1))
             for b in (topo.n_sm, 37, 74)]
    want = A0
    for rep in range(3):
        plan = plans[rep]
        for W, pm in zip(Ws, perms):
            ag.gemm_persistent(x.data_ptr(), W.data_ptr(), dC.data_ptr(), M, N, K, plan, torch.cuda.current_stream().cuda_stream)
            x = dC.to(torch.bfloat16)                    # the next call's activations, written by the launch right before it
            nxt = np.zeros_like(want)
            nxt[:, pm] = want
            want = nxt
    torch.cuda.synchronize()
    assert all(pl.last_status() == ag.AG_OK for pl in plans)
    assert np.array_equal(x.float().cpu().numpy(), want)


@pytest.mark.parametrize("in_memory,overlap", [(0, 1), (1, 1), (1, 2)])
def test_overlapping_launches_integer_exact(in_memory, overlap):
    """overlap_launches: a launch lets the next one start while it is still finishing.  Nine launches are queued
    without any synchronisation in between, over three weight matrices and three outputs; every output must be
    exact (integer-valued inputs), and every unit must have run once per launch."""
    M, N, K, ksp = 16, 2048, 4096, 8
    topo = device_topo()
    A = inputs.small_int_bf16(M, K, 61)
    Bs = [inputs.small_int_bf16(K, N, 62 + i) for i in range(3)]
    dA = to_dev_bf16(A)
    dBs = [to_dev_bf16(b) for b in Bs]
    dCs = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    for b, sel in ((topo.n_sm, 0), (74, 0), (37, 1), (20, 0)):
        # (on part of the chip the next launch's first blocks wait on the unplanned SMs until this launch's blocks have
        # left the planned ones)
        plan = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16, tile_n=128, sm_select=sel,
                                                            k_splits=ksp, splitk_in_memory=in_memory, overlap_launches=overlap))
        plan.reset_record()
        for i in range(9):
            ag.gemm_persistent(dA.data_ptr(), dBs[i % 3].data_ptr(), dCs[i % 3].data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        for i in range(3):
            assert np.array_equal(dCs[i].cpu().numpy().astype(np.float64), og.gemm_blocked(A, Bs[i]))
        owner, count = plan.tile_record()
        assert (count == 9).all()
        assert set(owner.tolist()) <= set(plan.parsed()["sm_list"].tolist())     # only planned SMs ran units


def test_in_memory_splitk_integer_exact_packed_and_rowmajor():
    M, N, K, ksp = 16, 2048, 2048, 8
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(M, N, K, ksp, integer=True)
    plan_m = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, splitk_in_memory=1, **kw))
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    ref = og.gemm_blocked(A, B)
    for _ in range(2):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan_m)
        torch.cuda.synchronize()
        assert plan_m.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref)
        assert np.array_equal(run_rowmajor(A, B, plan_m).astype(np.float64), ref)


def oracle_page_table(packed, page_die, tbl, dst_ptr):
    """The oracle's page table for the layout the library chose (single pages or groups of four)."""
    f = packed.group_free_bit()
    amap = dict(chunk_bytes=4096, die_of_chunk=tbl)
    if f < 0:
        return op.build_page_table(page_die, amap)
    return op.build_page_table_quads(page_die, amap, f, first=(dst_ptr // 4096) % 512)


def packed_setup(M, N, K, ksp, b=None, seed=41, integer=False, single_pages=False, consecutive=False):
    topo = device_topo()
    b = topo.n_sm if b is None else b
    if integer:
        A, B = inputs.small_int_bf16(M, K, seed), inputs.small_int_bf16(K, N, seed + 1)
    else:
        A, B = inputs.gemm_inputs(M, N, K, seed=seed)
    kw = dict(M=M, N=N, K=K, tile_m=16 if M <= 16 else 32, tile_n=128, k_splits=ksp)
    plan_d = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
    dst_bytes = 2 * K * N * 2 + (8 << 20)                    # two views, head-room for an uneven die split
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dB = to_dev_bf16(B)
    packed = ag.pack_weights(dB.data_ptr(), K, N, plan_d, amap, dst.data_ptr(), dst_bytes, single_pages=single_pages,
                             consecutive=consecutive)
    return topo, A, B, kw, plan_d, dst, amap, packed


@pytest.mark.parametrize("single_pages", [False, True])
def test_packing_matches_oracle_table_and_layout(single_pages):
    M, N, K, ksp = 16, 1024, 512, 2
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(M, N, K, ksp, single_pages=single_pages)
    assert (packed.group_free_bit() < 0) if single_pages else True
    tbl = amap.export()
    o_plan = op.build_plan(topo.as_dict(), None, topo.n_sm, op.default_policy(kind=op.DIE_COMPACT, **kw))
    assert plan_d.export().tobytes() == op.export(o_plan).tobytes()
    page_die = op.page_die_from_plan(o_plan, K)
    want_table = oracle_page_table(packed, page_die, tbl, dst.data_ptr())
    got_table = packed.page_table()
    assert np.array_equal(got_table, np.array(want_table, dtype=np.int32))
    assert len(set(got_table.tolist())) == got_table.size
    # every page sits on the die of its unit wherever the pair rule holds
    on_die = tbl[got_table] == np.array(page_die)
    assert on_die.mean() > 0.99
    n_chunks = int(got_table.max()) + 1
    want_img = op.pack_weights(B, want_table, n_chunks)
    got_img = dst[: n_chunks * 4096].cpu().numpy().view(np.uint16).reshape(n_chunks, 2048)
    assert np.array_equal(got_img, want_img)


@pytest.mark.parametrize("M,N,K,ksp,b", [(16, 1024, 1024, 1, None), (16, 2048, 2048, 4, None), (32, 1024, 512, 2, None), (9, 1096, 256, 1, None),
                                        (16, 2048, 4096 + 64, 3, 37), (64, 1024, 1024, 2, None), (128, 1024, 512, 1, 74)])
def test_packed_weights_in_consecutive_chunks(M, N, K, ksp, b):
    """The placement that ignores the dies: logical page p in chunk p (the page image is the oracle's for the identity
    table), a stage fetched with one plain copy; the GEMM over it is exact on integer inputs."""
    topo = device_topo()
    A, B = inputs.small_int_bf16(M, K, 77), inputs.small_int_bf16(K, N, 78)
    kw = dict(M=M, N=N, K=K, tile_m=16 if M <= 16 else 32 if M <= 32 else 64 if M <= 64 else 128, tile_n=128, k_splits=ksp,
              decode_shaped=1 if M > 64 else 0)
    plan = ag.sched_build(topo, None, b or topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
    n_pages = ((N + 127) // 128) * (K // 16)
    dst_bytes = n_pages * 4096
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    packed = ag.pack_weights(to_dev_bf16(B).data_ptr(), K, N, plan, amap, dst.data_ptr(), dst_bytes, consecutive=True)
    assert packed.group_free_bit() < 0 and not packed.closed_form()["enabled"]
    table = packed.page_table()
    assert np.array_equal(table, np.arange(n_pages, dtype=np.int32))
    if N % 128 == 0:
        want_img = op.pack_weights(B, table.tolist(), n_pages)
        assert np.array_equal(dst.cpu().numpy().view(np.uint16).reshape(n_pages, 2048), want_img)
    dA = to_dev_bf16(A)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), og.gemm_blocked(A, B))


@pytest.mark.parametrize("M,N,K,ksp", [(16, 1024, 1024, 1), (16, 2048, 2048, 4), (32, 1024, 512, 2), (9, 1096, 256, 1)])
@pytest.mark.parametrize("single_pages", [False, True])
def test_packed_gemm_integer_exact(M, N, K, ksp, single_pages):
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(M, N, K, ksp, integer=True, single_pages=single_pages)
    dA = to_dev_bf16(A)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan_d)
        torch.cuda.synchronize()
        assert plan_d.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), og.gemm_blocked(A, B))


def test_packed_gemm_full_size_affinity_and_inverted_plans():
    """M=16, N=K=8192 (the decode-shaped configuration): local and deliberately remote assignment
    compute the same C; the affinity policy over the page table rebuilds the packing plan."""
    M, N, K, ksp = 16, 8192, 8192, 16
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(M, N, K, ksp)
    table = packed.page_table()
    bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=table)
    plan_a = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, b=bop, **kw))
    plan_i = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, invert_affinity=1, b=bop, **kw))
    pa, pd, pi = plan_a.parsed(), plan_d.parsed(), plan_i.parsed()
    assert np.array_equal(pa["die_q"], pd["die_q"]) and np.array_equal(pa["sm_q"], pd["sm_q"])
    assert not np.array_equal(pi["die_q"], pd["die_q"])
    ref = og.gemm_blocked(A, B)
    dA = to_dev_bf16(A)
    for plan in (plan_d, plan_a, plan_i):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent_packed(dA.data_ptr(), packed, dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        check_close(dC.cpu().numpy(), ref)


@pytest.mark.parametrize("mask_bits,want_free_bit", [(0x1EF, 4), (0x1FF, -1)])
def test_closed_form_remap_on_a_synthetic_hash(mask_bits, want_free_bit):
    """Eq. 1 in closed form: with a map that is an exact XOR hash (handed in as a table), the kernel computes page
    addresses from the fitted mask and the per-page bits; the page table and C equal the table-driven path's."""
    M, N, K, ksp = 16, 1024, 2560, 4                          # 40 k-slabs: units of 10 slabs (5 stages)
    topo = device_topo()
    A, B = inputs.small_int_bf16(M, K, 71), inputs.small_int_bf16(K, N, 72)
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    kw = dict(M=M, N=N, K=K, tile_m=16, tile_n=128, k_splits=ksp)
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
    dst_bytes = 2 * K * N * 2 + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    assert dst.data_ptr() % (2 << 20) == 0
    doc = inputs.synthetic_chunk_die(dst_bytes // 4096, seed=13, mask_bits=mask_bits)
    amap = ag.affinity_from_table(dst.data_ptr(), doc)
    packs = {}
    for tables_only in (False, True):
        dst.zero_()
        packs[tables_only] = ag.pack_weights(dB.data_ptr(), K, N, plan, amap, dst.data_ptr(), dst_bytes, tables_only=tables_only)
        cf = packs[tables_only].closed_form()
        assert packs[tables_only].group_free_bit() == want_free_bit
        assert cf["enabled"] == (not tables_only)
        if cf["enabled"]:
            assert cf["mask"] == (mask_bits | 1) and cf["closed_bytes"] * 4 <= cf["table_bytes"]
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent_packed(dA.data_ptr(), packs[tables_only], dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), og.gemm_blocked(A, B))
    assert np.array_equal(packs[False].page_table(), packs[True].page_table())
    # the table is the oracle's: closed form on the oracle side too
    o_plan = op.build_plan(topo.as_dict(), None, topo.n_sm, oracle_policy(kind=op.DIE_COMPACT, **kw))
    page_die = op.page_die_from_plan(o_plan, K)
    o_amap = dict(chunk_bytes=4096, die_of_chunk=doc)
    want = (op.build_page_table_quads(page_die, o_amap, want_free_bit) if want_free_bit >= 0
            else op.build_page_table(page_die, o_amap))
    assert packs[False].page_table().tolist() == want


def test_closed_form_remap_on_the_measured_map():
    """On the chip's own map the closed form is used only if every table entry could be recomputed from the fitted
    hash; either way the result is the same as with tables."""
    M, N, K, ksp = 16, 2048, 2048, 4
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(M, N, K, ksp, integer=True)
    dA = to_dev_bf16(A)
    dB = to_dev_bf16(B)
    table0 = packed.page_table().copy()
    packed_t = ag.pack_weights(dB.data_ptr(), K, N, plan_d, amap, dst.data_ptr(), dst.numel(), tables_only=True)
    assert not packed_t.closed_form()["enabled"]
    assert np.array_equal(packed_t.page_table(), table0)
    for pk in (packed, packed_t):
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ag.gemm_persistent_packed(dA.data_ptr(), pk, dC.data_ptr(), M, N, K, plan_d)
        torch.cuda.synchronize()
        assert plan_d.last_status() == ag.AG_OK
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), og.gemm_blocked(A, B))
    print("closed form on the measured map:", packed.closed_form())


def test_packed_rejects_foreign_map_and_shapes():
    topo, A, B, kw, plan_d, dst, amap, packed = packed_setup(16, 512, 256, 1)
    other = ag.aligned_device_bytes(1 << 20)
    h = ag.C.c_void_p()
    st = ag.lib().ag_pack_weights(to_dev_bf16(B).data_ptr(), 256, 512, plan_d.handle, amap.handle, other.data_ptr(),
                                  other.numel(), ag.C.byref(h))
    assert st == ag.AG_ERR_STALE_AMAP
    dA = to_dev_bf16(A)
    dC = torch.zeros((16, 512), dtype=torch.float32, device="cuda")
    assert ag.lib().gemm_persistent_packed(dA.data_ptr(), packed.handle, dC.data_ptr(), 16, 512, 128, plan_d.handle,
                                           None) == ag.AG_ERR_ARG

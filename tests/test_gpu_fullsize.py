"""Parity at the full sizes of the workload configurations, in the launch configurations that
bench.py and experiments.py time.  The oracle computes sampled entries one by one and one full
block; exactly-once execution is checked from the plan's record."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import check_close, device_topo, to_dev_bf16

pytestmark = pytest.mark.gpu


def sampled_check(C, A, B, n=160, seed=0, block=None):
    M, N = C.shape
    rng = np.random.default_rng(seed)
    rows, cols = rng.integers(0, M, n), rng.integers(0, N, n)
    rows[:4], cols[:4] = [0, M - 1, 0, M - 1], [0, 0, N - 1, N - 1]
    ref = og.gemm_entries(A, B, rows, cols)
    got = C[rows, cols].astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-2
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-4
    if block is not None:
        r0, r1, c0, c1 = block
        check_close(C[r0:r1, c0:c1], og.gemm_block(A, B, r0, r1, c0, c1))


def test_headline_configuration_block_pairs_affinity_plan():
    """8192^3, 256 x 256 units of block pairs, affinity policy over a probed buffer, raster group 8."""
    M = N = K = 8192
    A, B = inputs.gemm_inputs(M, N, K)
    topo = device_topo()
    a_bytes, b_bytes, c_bytes = M * K * 2, K * N * 2, M * N * 4
    buf = torch.empty(a_bytes + b_bytes + c_bytes, dtype=torch.uint8, device="cuda")
    dA = buf[:a_bytes].view(torch.int16).view(M, K)
    dB = buf[a_bytes:a_bytes + b_bytes].view(torch.int16).view(K, N)
    dC = buf[a_bytes + b_bytes:].view(torch.float32).view(M, N)
    dA.copy_(torch.from_numpy(A.view(np.int16)))
    dB.copy_(torch.from_numpy(B.view(np.int16)))
    dC.fill_(float("nan"))
    amap = ag.affinity_probe(buf.data_ptr(), buf.numel(), topo)
    assert torch.equal(dA.cpu(), torch.from_numpy(A.view(np.int16)))     # the probe left the operands intact
    ops = dict(a=dict(offset=0, row_stride=K * 2, elem_bytes=2), b=dict(offset=a_bytes, row_stride=N * 2, elem_bytes=2),
               c=dict(offset=a_bytes + b_bytes, row_stride=N * 4, elem_bytes=4))
    min_margin = (256 * K * 2 + 256 * K * 2 + 256 * 256 * 4) // 8
    plan = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, M=M, N=N, K=K, tile_m=256, tile_n=256,
                                                                raster_group=8, min_margin=min_margin, **ops))
    plan.reset_record()
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    C = dC.cpu().numpy()
    assert np.isfinite(C).all()
    sampled_check(C, A, B, block=(7936, 8192, 7936, 8192))
    owner, count = plan.tile_record()
    assert (count == 1).all() and len(count) == 1024


@pytest.mark.parametrize("mode", ["random_subset_one_block", "die_compact_pairs", "gpc_spread_pairs"])
def test_sm_budget_configuration_4096(mode):
    M = N = K = 4096
    A, B = inputs.gemm_inputs(M, N, K)
    topo = device_topo()
    if mode == "random_subset_one_block":
        pol = ag.make_policy(kind=ag.AG_OBLIVIOUS, seed=7, M=M, N=N, K=K, raster_group=8)
    else:
        pol = ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=256, tile_n=256, raster_group=4,
                             sm_select=1 if mode == "gpc_spread_pairs" else 0)
    plan = ag.sched_build(topo, None, 64, pol)
    plan.reset_record()
    dA, dB = to_dev_bf16(A), to_dev_bf16(B)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    sampled_check(dC.cpu().numpy(), A, B, n=96, block=(3840, 4096, 0, 256))
    owner, count = plan.tile_record()
    assert (count == 1).all() and set(owner) <= set(plan.parsed()["sm_list"])


@pytest.mark.parametrize("partition", ["die_split", "oblivious"])
def test_two_stream_configuration_runs_both_gemms_correctly(partition):
    """Prefill 8192 x 4096 x 4096 and decode 32 x 4096 x 4096 at the same time on disjoint SM sets."""
    Mp, Md, N, K = 8192, 32, 4096, 4096
    Ap, Bp = inputs.gemm_inputs(Mp, N, K)
    Ad, Bd = inputs.uniform_bf16(Md, K, 77), inputs.uniform_bf16(K, N, 100)
    topo = device_topo()
    kind = ag.AG_DIE_COMPACT if partition == "die_split" else ag.AG_OBLIVIOUS
    plan_p = ag.sched_build(topo, None, 74, ag.make_policy(kind=kind, preferred_die=0, M=Mp, N=N, K=K, tile_m=256,
                                                           tile_n=256, raster_group=4))
    taken = [int(s) for s in plan_p.parsed()["sm_list"]]
    plan_d = ag.sched_build(topo, None, 74, ag.make_policy(kind=kind, avoid=taken, M=Md, N=N, K=K, tile_m=32, tile_n=128,
                                                           k_splits=8, splitk_in_memory=1))
    assert not set(taken) & set(int(s) for s in plan_d.parsed()["sm_list"])
    dAp, dBp, dAd, dBd = to_dev_bf16(Ap), to_dev_bf16(Bp), to_dev_bf16(Ad), to_dev_bf16(Bd)
    dCp = torch.full((Mp, N), float("nan"), dtype=torch.float32, device="cuda")
    dCd = torch.full((Md, N), float("nan"), dtype=torch.float32, device="cuda")
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for i in range(3):
        ag.gemm_persistent(dAp.data_ptr(), dBp.data_ptr(), dCp.data_ptr(), Mp, N, K, plan_p, s1.cuda_stream)
        for _ in range(8):
            ag.gemm_persistent(dAd.data_ptr(), dBd.data_ptr(), dCd.data_ptr(), Md, N, K, plan_d, s2.cuda_stream)
    torch.cuda.synchronize()
    assert plan_p.last_status() == ag.AG_OK and plan_d.last_status() == ag.AG_OK
    sampled_check(dCp.cpu().numpy(), Ap, Bp, n=96, block=(0, 256, 3840, 4096))
    check_close(dCd.cpu().numpy(), og.gemm_blocked(Ad, Bd))
    owner_p, _ = plan_p.tile_record()
    owner_d, _ = plan_d.tile_record()
    assert set(owner_p) <= set(taken) and not set(owner_d) & set(taken)     # each GEMM stayed on its own SMs


@pytest.mark.parametrize("k_splits,in_memory,overlap,budget,spread,consecutive",
                         [(16, 1, 2, 0, 0, 0), (16, 0, 2, 0, 0, 0), (16, 1, 1, 0, 0, 0), (4, 1, 2, 0, 0, 0), (4, 0, 2, 0, 0, 0), (4, 1, 1, 0, 0, 0),
                          (4, 1, 2, 74, 1, 0), (4, 1, 2, 37, 1, 0), (4, 1, 2, 74, 0, 0), (4, 0, 1, 37, 0, 0),
                          (16, 1, 2, 0, 0, 1), (4, 1, 2, 0, 0, 1), (4, 1, 2, 74, 0, 1)])
def test_decode_configuration_queued_back_to_back(k_splits, in_memory, overlap, budget, spread, consecutive):
    """M = 16, N = K = 8192 with die-local packed weights (or the same pages in consecutive chunks), as timed - on all SMs
    and on 74 and 37 of them (whole TPCs over both dies, or one die): calls queued without a synchronisation in between, rotating over four weight matrices,
    launches overlapping.  Every call writes a C of its own here, and every one of them is compared with the oracle in
    full (a race between overlapping launches would show in some)."""
    from tests.gpu_util import check_close as close
    M, N, K, n_buf, n_calls = 16, 8192, 8192, 4, 12
    topo = device_topo()
    A = inputs.uniform_bf16(M, K, inputs.DEFAULT_SEED)
    Bs = [inputs.uniform_bf16(K, N, inputs.DEFAULT_SEED + 1 + i) for i in range(n_buf)]
    dA, dBs = to_dev_bf16(A), [to_dev_bf16(b) for b in Bs]
    plan = ag.sched_build(topo, None, budget or topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=16, tile_n=128, sm_select=spread,
                                                                          k_splits=k_splits, splitk_in_memory=in_memory, overlap_launches=overlap))
    dst_bytes = 2 * K * N * 2 + (8 << 20)
    dsts = [ag.aligned_device_bytes(dst_bytes) for _ in range(n_buf)]
    packs = []
    for i in range(n_buf):
        amap = ag.affinity_probe(dsts[i].data_ptr(), dst_bytes, topo)
        packs.append(ag.pack_weights(dBs[i].data_ptr(), K, N, plan, amap, dsts[i].data_ptr(), dst_bytes, consecutive=bool(consecutive)))
    dCs = [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n_calls)]
    torch.cuda.synchronize()
    plan.reset_record()
    for c in range(n_calls):
        ag.gemm_persistent_packed(dA.data_ptr(), packs[c % n_buf], dCs[c].data_ptr(), M, N, K, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK
    owner, count = plan.tile_record()
    assert (count == n_calls).all()
    assert set(owner.tolist()) <= set(plan.parsed()["sm_list"].tolist())
    want = [og.gemm_blocked(A, b) for b in Bs]
    for c in range(n_calls):
        close(dCs[c].cpu().numpy(), want[c % n_buf])
    if not in_memory:                                       # the workspace mode adds in a fixed order: same weights, same bits
        assert torch.equal(dCs[0], dCs[n_buf]) and torch.equal(dCs[1], dCs[n_buf + 1])


@pytest.mark.parametrize("placement", ["local", "interleaved"])
def test_attention_configuration_queued_back_to_back(placement):
    """Batch 128, 32 query heads on 8 KV heads, 512 keys, all SMs, launches overlapping, as timed: six calls queued
    without a synchronisation, each with queries and outputs of its own; all of them against the oracle."""
    from oracle import attention as oa
    B, Hq, Hkv, L, D, n_calls = 128, 32, 8, 512, 128, 6
    topo = device_topo()
    K = inputs.uniform_bf16(B * Hkv * L, D, inputs.DEFAULT_SEED + 41).reshape(B, Hkv, L, D)
    V = inputs.uniform_bf16(B * Hkv * L, D, inputs.DEFAULT_SEED + 42).reshape(B, Hkv, L, D)
    Qs = [inputs.uniform_bf16(B * Hq, D, inputs.DEFAULT_SEED + 40 + 7 * c).reshape(B, Hq, D) for c in range(n_calls)]
    dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16).copy()).cuda()
    dK, dV, dQs = dev(K), dev(V), [dev(q) for q in Qs]
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=Hq // Hkv, N=128 * B * Hkv, K=L, tile_m=16,
                                                                tile_n=128, k_splits=1, overlap_launches=1))
    kv_bytes = 2 * B * Hkv * L * D * 2
    dst_bytes = 2 * kv_bytes + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    kv = ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L, plan, amap, dst.data_ptr(), dst_bytes,
                    ag.KV_LOCAL if placement == "local" else ag.KV_INTERLEAVED)
    dOs = [torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n_calls)]
    torch.cuda.synchronize()
    plan.reset_record()
    for c in range(n_calls):
        ag.attention_decode(dQs[c].data_ptr(), kv, None, dOs[c].data_ptr(), B, Hq, plan)
    torch.cuda.synchronize()
    assert plan.last_status() == ag.AG_OK, plan.last_status_where()
    owner, count = plan.tile_record()
    assert (count == n_calls).all()
    for c in range(n_calls):
        got = dOs[c].cpu().numpy().astype(np.float64)
        want = oa.gqa_decode(Qs[c], K, V)
        assert np.isfinite(got).all()
        assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 5e-5 and np.abs(got - want).max() <= 2e-4

"""Attention decode with die-local KV pages against the fp64 oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs
from tests.gpu_util import device_topo

pytestmark = pytest.mark.gpu

# Tolerance: scores are exact bf16 products accumulated in fp32 (relative 2^-24 per add), the exponential is the
# hardware's exp2 (2 ulp), the probabilities enter the second product with 16 significant bits, outputs are
# accumulated in fp32: a few 1e-6 relative in all; the bound asserted leaves a factor of ten.
REL_FRO, MAX_ABS = 5e-5, 2e-4


def make_case(B, Hq, Hkv, L, seed, q_scale=1.0):
    D = 128
    Q = inputs.uniform_bf16(B * Hq, D, seed).reshape(B, Hq, D)
    if q_scale != 1.0:
        qf = oa.bf16_to_f64(Q) * q_scale
        Q = inputs.f32_to_bf16_bits(qf.astype(np.float32)).reshape(B, Hq, D)
    K = inputs.uniform_bf16(B * Hkv * L, D, seed + 1).reshape(B, Hkv, L, D)
    V = inputs.uniform_bf16(B * Hkv * L, D, seed + 2).reshape(B, Hkv, L, D)
    return Q, K, V


def dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16).copy()).cuda()


def run_attention(Q, K, V, placement, kv_len=None, budget=None, overlap=0):
    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    topo = device_topo()
    b = topo.n_sm if budget is None else budget
    n_chunks = (L + 1023) // 1024                    # requests over 1024 keys: one unit per chunk of 1024 keys
    plan = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=Hq // Hkv, N=128 * B * Hkv * n_chunks, K=L, tile_m=16,
                                                        tile_n=128, k_splits=1, overlap_launches=overlap))
    kv_bytes = 2 * B * Hkv * L * D * 2
    dst_bytes = (2 * kv_bytes if placement != ag.KV_INTERLEAVED else kv_bytes) + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    dK, dV, dQ = dev(K), dev(V), dev(Q)
    kv = ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L, plan, amap, dst.data_ptr(), dst_bytes, placement)
    dO = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    dlen = None if kv_len is None else torch.tensor(kv_len, dtype=torch.int32, device="cuda")
    plan.reset_record()
    for _ in range(2):
        ag.attention_decode(dQ.data_ptr(), kv, None if dlen is None else dlen.data_ptr(), dO.data_ptr(), B, Hq, plan)
    torch.cuda.synchronize()
    st = plan.last_status()
    assert st == ag.AG_OK, (ag.strerror(st), plan.last_status_where())
    owner, count = plan.tile_record()
    assert (count == 2).all()
    return dO.cpu().numpy().astype(np.float64), kv.info(), dst


def check(got, want):
    assert np.isfinite(got).all()
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    mx = np.abs(got - want).max()
    assert rel <= REL_FRO and mx <= MAX_ABS, (rel, mx)


@pytest.mark.parametrize("placement", [ag.KV_LOCAL, ag.KV_REMOTE, ag.KV_INTERLEAVED])
@pytest.mark.parametrize("shape", [(4, 8, 2, 256), (3, 16, 2, 128), (9, 4, 4, 384)])
def test_small_cases_against_the_oracle(placement, shape):
    B, Hq, Hkv, L = shape
    for q_scale in (1.0, 12.0):                      # soft and peaked score distributions
        Q, K, V = make_case(B, Hq, Hkv, L, seed=100 + B, q_scale=q_scale)
        got, info, _ = run_attention(Q, K, V, placement)
        check(got, oa.gqa_decode(Q, K, V))
        if placement == ag.KV_LOCAL:
            assert info["local_fraction"] == 1.0 and info["group_free_bit"] >= 2


def test_ragged_lengths_and_closed_forms():
    B, Hq, Hkv, L = 6, 8, 2, 512
    Q, K, V = make_case(B, Hq, Hkv, L, seed=7)
    lens = [512, 130, 0, 1, 256, 383]
    got, _, _ = run_attention(Q, K, V, ag.KV_LOCAL, kv_len=lens)
    check(got, oa.gqa_decode(Q, K, V, lens))
    assert not got[2].any()
    # zero queries: every output row is the mean of the value rows of its KV head
    Q0 = np.zeros_like(Q)
    got, _, _ = run_attention(Q0, K, V, ag.KV_INTERLEAVED)
    Vf = oa.bf16_to_f64(V)
    for b in range(B):
        for hq in range(Hq):
            assert np.abs(got[b, hq] - Vf[b, hq // 4].mean(axis=0)).max() <= 1e-5


@pytest.mark.parametrize("placement", [ag.KV_LOCAL, ag.KV_INTERLEAVED])
@pytest.mark.parametrize("shape", [(2, 8, 2, 2048), (3, 4, 4, 1280), (2, 16, 2, 4096)])
def test_long_requests_in_chunks(placement, shape):
    """More than 1024 keys: chunks of 1024 keys run as units of their own and a second kernel puts them together."""
    B, Hq, Hkv, L = shape
    Q, K, V = make_case(B, Hq, Hkv, L, seed=300 + L, q_scale=6.0)
    got, _, _ = run_attention(Q, K, V, placement)
    check(got, oa.gqa_decode(Q, K, V))
    got, _, _ = run_attention(Q, K, V, placement, overlap=1)     # the second launch begins while the first one finishes
    check(got, oa.gqa_decode(Q, K, V))
    got, _, _ = run_attention(Q, K, V, placement, budget=37, overlap=1)   # the same on part of the chip
    check(got, oa.gqa_decode(Q, K, V))
    # ragged: lengths that end inside a chunk, at a chunk boundary, in the first chunk, and zero
    lens = [L - 1, 1025, 0][:B] if B == 3 else [1024, L - 127][:B]
    got, _, _ = run_attention(Q, K, V, placement, kv_len=lens)
    check(got, oa.gqa_decode(Q, K, V, lens))
    if 0 in lens:
        assert not got[lens.index(0)].any()


def test_serving_shape_on_sm_budgets():
    """Batch 128, 512 keys, 8 KV heads, 32 query heads (the decode side of the paper's serving split): 1024 units."""
    B, Hq, Hkv, L = 128, 32, 8, 512
    Q, K, V = make_case(B, Hq, Hkv, L, seed=21)
    want = oa.gqa_decode(Q, K, V)
    # the last one with overlapping launches (the second launch begins while the first one finishes)
    for placement, budget, overlap in ((ag.KV_LOCAL, None, 0), (ag.KV_REMOTE, None, 0), (ag.KV_LOCAL, 74, 0), (ag.KV_LOCAL, None, 1),
                                       (ag.KV_LOCAL, 74, 1), (ag.KV_INTERLEAVED, 37, 1)):
        got, _, _ = run_attention(Q, K, V, placement, budget=budget, overlap=overlap)
        check(got, want)


def test_appended_tokens_land_where_packing_would_put_them():
    """A decode loop: pack a cache that holds the first keys of every request, append the next tokens one step at a
    time (request b is at its own position), attend after every step; every step must agree with the oracle on the
    keys written so far, and the appended cache must equal a cache packed from the full K and V byte for byte."""
    B, Hq, Hkv, L = 5, 8, 2, 384
    Q, K, V = make_case(B, Hq, Hkv, L, seed=55)
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=Hq // Hkv, N=128 * B * Hkv, K=L, tile_m=16,
                                                               tile_n=128, k_splits=1))
    kv_bytes = 2 * B * Hkv * L * 128 * 2
    dst_bytes = 2 * kv_bytes + (8 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    start = np.array([0, 5, 127, 200, 380], dtype=np.int32)          # keys that every request already has
    K0, V0 = K.copy(), V.copy()
    for b in range(B):
        K0[b, :, start[b]:] = 0
        V0[b, :, start[b]:] = 0
    dK0, dV0, dQ = dev(K0), dev(V0), dev(Q)
    kv = ag.kv_pack(dK0.data_ptr(), dV0.data_ptr(), B, Hkv, L, plan, amap, dst.data_ptr(), dst_bytes, ag.KV_LOCAL)
    dO = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    lens = start.copy()
    for step in range(4):
        pos = np.where(lens < L, lens, -1).astype(np.int32)            # a full request takes no more tokens
        k_new = np.stack([K[b, :, min(lens[b], L - 1)] for b in range(B)])   # [B][H_kv][128]
        v_new = np.stack([V[b, :, min(lens[b], L - 1)] for b in range(B)])
        d_pos, d_k, d_v = torch.from_numpy(pos).cuda(), dev(k_new), dev(v_new)
        kv.append(d_k.data_ptr(), d_v.data_ptr(), d_pos.data_ptr())
        lens = np.minimum(lens + 1, L).astype(np.int32)
        d_len = torch.from_numpy(lens).cuda()
        ag.attention_decode(dQ.data_ptr(), kv, d_len.data_ptr(), dO.data_ptr(), B, Hq, plan)
        torch.cuda.synchronize()
        assert plan.last_status() == ag.AG_OK
        check(dO.cpu().numpy().astype(np.float64), oa.gqa_decode(Q, K, V, [int(x) for x in lens]))
    appended = dst.cpu().numpy().copy()
    # the same cache packed in one go from K and V with everything past the final lengths zeroed
    K1, V1 = K.copy(), V.copy()
    for b in range(B):
        K1[b, :, lens[b]:] = 0
        V1[b, :, lens[b]:] = 0
    dst.zero_()
    dK1, dV1 = dev(K1), dev(V1)
    kv2 = ag.kv_pack(dK1.data_ptr(), dV1.data_ptr(), B, Hkv, L, plan, amap, dst.data_ptr(), dst_bytes, ag.KV_LOCAL)
    torch.cuda.synchronize()
    assert np.array_equal(appended, dst.cpu().numpy())
    del kv2


@pytest.mark.parametrize("lens", [[1024, 0], [0, 1024, 0, 700], [0, 0, 0, 1], [640, 0, 0, 1024]])
def test_units_without_keys_between_long_units_on_one_sm(lens):
    """One SM runs every unit in turn.  A unit with more key tiles than the ring of probability tiles holds needs its
    value products issued while its softmax is still going on; they are issued when the next ring entry arrives, also
    when that entry is a unit without keys (this case once ended in a bounded wait running out)."""
    B, Hq, Hkv, L = len(lens), 4, 1, 1024
    Q, K, V = make_case(B, Hq, Hkv, L, seed=404)
    for budget in (1, 2):
        got, _, _ = run_attention(Q, K, V, ag.KV_INTERLEAVED, kv_len=lens, budget=budget)
        check(got, oa.gqa_decode(Q, K, V, lens))


@pytest.mark.parametrize("seed", range(10))
def test_seeded_random_shapes(seed):
    """Random batch, head counts, lengths (also beyond one chunk), SM budgets, placements and ragged kv_len."""
    rng = np.random.default_rng(1000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8]))
    B = int(rng.integers(1, 12))
    L = 128 * int(rng.choice([1, 2, 3, 5, 8, 9, 16, 20]))
    topo = device_topo()
    budget = int(rng.choice([topo.n_sm, 74, 37, 11]))
    placement = int(rng.choice([ag.KV_LOCAL, ag.KV_REMOTE, ag.KV_INTERLEAVED]))
    Q, K, V = make_case(B, Hkv * G, Hkv, L, seed=2000 + seed, q_scale=float(rng.choice([1.0, 4.0, 16.0])))
    lens = None if seed % 3 == 0 else [int(x) for x in rng.integers(0, L + 1, size=B)]
    got, _, _ = run_attention(Q, K, V, placement, kv_len=lens, budget=budget)
    check(got, oa.gqa_decode(Q, K, V, lens))


def test_bad_arguments():
    topo = device_topo()
    plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=4, N=128 * 8, K=256, tile_m=16,
                                                                tile_n=128, k_splits=1))
    dst = ag.aligned_device_bytes(16 << 20)
    amap = ag.affinity_probe(dst.data_ptr(), dst.numel(), topo)
    k = torch.zeros(8 * 256 * 128, dtype=torch.int16, device="cuda")
    h = ag.C.c_void_p()
    L_ = ag.lib()
    # L not a multiple of 128, too long, wrong unit count, wrong head dimension
    for (B, H, Lk, D) in ((4, 2, 200, 128), (4, 2, 2048, 128), (4, 4, 256, 128), (4, 2, 256, 64)):   # (2048 keys need a plan of 16 units)
        st = L_.ag_kv_pack(k.data_ptr(), k.data_ptr(), B, H, Lk, D, plan.handle, amap.handle, dst.data_ptr(), dst.numel(), 0, ag.C.byref(h))
        assert st == ag.AG_ERR_ARG

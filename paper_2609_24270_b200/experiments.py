"""Measurements for the workload configurations other than the headline one (which bench.py times).

    python -m paper_2609_24270_b200.experiments --config 3 [--out results.jsonl]
    python -m paper_2609_24270_b200.experiments --config 4
    python -m paper_2609_24270_b200.experiments --config 5
    python -m paper_2609_24270_b200.experiments --config raster      # raster-group sweep at 8192^3
    python -m paper_2609_24270_b200.experiments --config groupgemm         # MoE-shaped grouped GEMM, ~20 rows per expert
    python -m paper_2609_24270_b200.experiments --config groupgemm_dense   # same, 192 / 1024 rows per expert
    python -m paper_2609_24270_b200.experiments --config gpc_bandwidth     # L2 bandwidth of k SMs: one GPC vs spread
    python -m paper_2609_24270_b200.experiments --config latency           # latency histograms from one SM per die
    python -m paper_2609_24270_b200.experiments --config cluster_sets      # cluster eligibility of equal-size SM sets
    python -m paper_2609_24270_b200.experiments --config attention         # decode attention, KV pages local / remote / interleaved
    python -m paper_2609_24270_b200.experiments --config attention_sweep   # the paper's decode sweep: MHA / GQA, batch 1-64, keys from 512
    python -m paper_2609_24270_b200.experiments --config 5_attention       # prefill GEMM and decode attention on disjoint SM partitions

Every line printed is one JSON record.  Timing: CUDA events on the launching stream, warm-up
launches first, median of the timed launches.  torch is used for device memory, streams and events.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

from . import binding as ag
from . import inputs


def emit(rec, fh):
    line = json.dumps(rec)
    print(line, flush=True)
    if fh:
        fh.write(line + "\n")
        fh.flush()


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda()


def time_launches(fn, warmup=3, iters=10, stream=None, batches=3):
    """Per-launch times in ms: `batches` batches of `iters` back-to-back launches, each batch bracketed by one
    event pair (an event pair around every single launch would add several microseconds to each)."""
    stream = stream or torch.cuda.current_stream()
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    out = []
    for _ in range(batches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(iters):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) / iters)
    return out


def sm_set_summary(topo, plan):
    p = plan.parsed()
    sms = [int(s) for s in p["sm_list"]]
    die = [int(d) for d in p["die_sm_count"]]
    gpcs = np.bincount([topo.gpc[s] for s in sms if topo.gpc[s] >= 0], minlength=max(topo.n_gpc, 1))
    return dict(die_sm_count=die, gpc_sm_count=[int(x) for x in gpcs])


# ---------------------------------------------------------------------------------------------
def config3(fh, topo, budgets=(16, 32, 48, 64, 74), n_subsets=32):
    """M=N=K=4096 on SM budgets; 32 seeded random subsets and the die_compact subset per budget."""
    M = N = K = 4096
    A, B = inputs.gemm_inputs(M, N, K)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    flops = 2.0 * M * N * K
    for b in budgets:
        res = {}
        plans = {f"random_{s}": ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, seed=s, M=M, N=N, K=K,
                                                                            raster_group=4))
                 for s in range(1, n_subsets + 1)}
        plans["lowest_ids"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, M=M, N=N, K=K, raster_group=4))
        plans["die_compact"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K,
                                                                            raster_group=4))
        plans["gpc_spread"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K,
                                                                           raster_group=4, sm_select=1))
        # whole-TPC sets can also run block pairs (256 x 256 units); random subsets cannot
        for name, sel in (("die_compact_pairs", 0), ("gpc_spread_pairs", 1)):
            if b % 2 == 0:
                plans[name] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=M, N=N, K=K, tile_m=256,
                                                                           tile_n=256, raster_group=4, sm_select=sel))
        # two passes over all subsets so that clock drift is shared
        acc = {n: [] for n in plans}
        for _ in range(2):
            for n, plan in plans.items():
                acc[n] += time_launches(lambda: ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan),
                                        warmup=2, iters=5)
        for n in plans:
            res[n] = flops / (float(np.median(acc[n])) * 1e-3) / 1e12
            assert plans[n].last_status() == ag.AG_OK
        rnd = [res[f"random_{s}"] for s in range(1, n_subsets + 1)]
        rank = 1 + sum(1 for v in rnd if v > res["die_compact"])
        rank_spread = 1 + sum(1 for v in rnd if v > res["gpc_spread"])
        emit(dict(config=3, workload="dense GEMM 4096^3 bf16, 128x256 tiles", sm_budget=b,
                  random_subsets_tflops=dict(min=min(rnd), max=max(rnd), median=float(np.median(rnd)),
                                             spread_max_over_min=max(rnd) / min(rnd)),
                  lowest_ids_tflops=res["lowest_ids"], die_compact_tflops=res["die_compact"],
                  die_compact_rank_among_33=rank, die_compact_set=sm_set_summary(topo, plans["die_compact"]),
                  gpc_spread_tflops=res["gpc_spread"], gpc_spread_rank_among_33=rank_spread,
                  gpc_spread_set=sm_set_summary(topo, plans["gpc_spread"]),
                  die_compact_pairs_tflops=res.get("die_compact_pairs"), gpc_spread_pairs_tflops=res.get("gpc_spread_pairs"),
                  peak_scaled_tflops=2250.0 * b / topo.n_sm, all_tflops=rnd), fh)


# ---------------------------------------------------------------------------------------------
def config4(fh, topo, budgets=(37, 74, 148), n_buffers=4, overlap=2, k_splits=(16, 4)):
    """M=16, N=K=8192 decode-shaped GEMM, weights die-packed; die-local vs remote assignment; 16 and 4 k-splits.
    The calls are independent (same activations, rotating weights): overlap_launches = 2."""
    for ksp in k_splits:
        _config4(fh, topo, budgets, n_buffers, overlap, ksp)


def _config4(fh, topo, budgets, n_buffers, overlap, ksp):
    M, N, K = 16, 8192, 8192
    A = inputs.uniform_bf16(M, K, inputs.DEFAULT_SEED)
    dA = dev_bf16(A)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    algo_bytes = K * N * 2 + M * K * 2 + M * N * 4
    kw = dict(M=M, N=N, K=K, tile_m=16, tile_n=128, k_splits=ksp, splitk_in_memory=1, overlap_launches=overlap)
    Bs = [dev_bf16(inputs.uniform_bf16(K, N, inputs.DEFAULT_SEED + 1 + i)) for i in range(n_buffers)]
    dst_bytes = 2 * K * N * 2 + (8 << 20)
    for b in budgets:
        plan_local = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
        # the same budget taken as whole TPCs from the GPCs of both dies: each die then streams its own half of the
        # weights from its own memory, and the set uses the memory of both dies
        plan_spread = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, sm_select=1, **kw))
        dsts, packs, packs_single, packs_spread, packs_tables, packs_consec = [], [], [], [], [], []
        for i in range(n_buffers):                      # rotate buffers so that no launch finds its weights in L2
            dst2 = ag.aligned_device_bytes(dst_bytes)
            amap2 = ag.affinity_probe(dst2.data_ptr(), dst_bytes, topo)
            packs_spread.append((ag.pack_weights(Bs[i].data_ptr(), K, N, plan_spread, amap2, dst2.data_ptr(), dst_bytes), amap2))
            dsts.append(dst2)
            dst = ag.aligned_device_bytes(dst_bytes)
            amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
            packs.append((ag.pack_weights(Bs[i].data_ptr(), K, N, plan_local, amap, dst.data_ptr(), dst_bytes), amap))
            dsts.append(dst)
            dst3 = ag.aligned_device_bytes(dst_bytes)   # same layout, page addresses from tables
            amap3 = ag.affinity_probe(dst3.data_ptr(), dst_bytes, topo)
            packs_tables.append((ag.pack_weights(Bs[i].data_ptr(), K, N, plan_local, amap3, dst3.data_ptr(), dst_bytes,
                                                 tables_only=True), amap3))
            dsts.append(dst3)
            dstc = ag.aligned_device_bytes(K * N * 2)     # the same pages in consecutive chunks (dies ignored)
            amapc = ag.affinity_probe(dstc.data_ptr(), K * N * 2, topo)
            packs_consec.append((ag.pack_weights(Bs[i].data_ptr(), K, N, plan_local, amapc, dstc.data_ptr(), K * N * 2, consecutive=True), amapc))
            dsts.append(dstc)
            dst1 = ag.aligned_device_bytes(dst_bytes)   # same, one page per copy (for comparison)
            amap1 = ag.affinity_probe(dst1.data_ptr(), dst_bytes, topo)
            packs_single.append((ag.pack_weights(Bs[i].data_ptr(), K, N, plan_local, amap1, dst1.data_ptr(), dst_bytes,
                                                 single_pages=True), amap1))
            dsts.append(dst1)
        table = packs[0][0].page_table()
        page_owner = np.repeat(_unit_die(plan_local), K // 16 // ksp)      # pages of a unit are consecutive
        on_die = float((packs[0][1].export()[table] == page_owner).mean())
        bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=table)
        local_set = plan_local.parsed()["sm_list"]
        n0 = int(plan_local.parsed()["die_sm_count"][0])
        if b < topo.n_sm and (n0 == 0 or n0 == b):
            # all SMs on one die: the remote case runs the same units from SMs of the other die
            other = 1 - (0 if n0 == b else 1)
            plan_remote = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, preferred_die=other, **kw))
        else:
            plan_remote = ag.sched_build(topo, packs[0][1], b, ag.make_policy(kind=ag.AG_AFFINITY, invert_affinity=1, b=bop, **kw))
        plan_obl = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, **kw))
        out = {}
        for name, plan, pset in (("die_local", plan_local, packs), ("remote", plan_remote, packs),
                                 ("die_local_single_pages", plan_local, packs_single),
                                 ("die_local_page_tables", plan_local, packs_tables),
                                 ("die_local_both_dies", plan_spread, packs_spread),
                                 ("pages_consecutive_oblivious", plan_obl, packs_consec),
                                 ("pages_consecutive_die_compact", plan_local, packs_consec)):
            state = {"i": 0}

            def run():
                pk = pset[state["i"] % n_buffers][0]
                state["i"] += 1
                ag.gemm_persistent_packed(dA.data_ptr(), pk, dC.data_ptr(), M, N, K, plan)
            ms = time_queued(run, warmup=4, iters=24)
            assert plan.last_status() == ag.AG_OK
            out[name] = algo_bytes / (ms * 1e-3) / 1e9
        for name, plan in (("rowmajor_oblivious", plan_obl), ("rowmajor_die_compact", plan_local), ("rowmajor_both_dies", plan_spread)):
            state = {"i": 0}

            def run2():
                wb = Bs[state["i"] % n_buffers]
                state["i"] += 1
                ag.gemm_persistent(dA.data_ptr(), wb.data_ptr(), dC.data_ptr(), M, N, K, plan)
            ms = time_queued(run2, warmup=4, iters=24)
            out[name] = algo_bytes / (ms * 1e-3) / 1e9
        emit(dict(config=4, workload=f"GEMM M=16 N=K=8192 bf16, 128-col units x {ksp} k-splits, 4 rotating weight buffers", k_splits=ksp,
                  sm_budget=b, overlap_launches=overlap, gbs=out, local_over_remote=out["die_local"] / out["remote"],
                  pages_on_owner_die=on_die, page_group_free_bit=packs[0][0].group_free_bit(), closed_form=packs[0][0].closed_form(), local_set=sm_set_summary(topo, plan_local),
                  remote_set=sm_set_summary(topo, plan_remote), both_dies_set=sm_set_summary(topo, plan_spread), algo_bytes=algo_bytes,
                  hbm_peak_measured_gbs=6534.1), fh)
        del packs, packs_single, packs_spread, packs_tables, packs_consec, dsts


def _unit_die(plan):
    p = plan.parsed()
    ud = np.zeros(p["n_units"], dtype=np.uint8)
    ud[p["die_q"][int(p["die_q_off"][1]):]] = 1
    return ud


# ---------------------------------------------------------------------------------------------
def config5(fh, topo):
    """Prefill-like GEMM (8192x4096x4096) and decode-like GEMM (32x4096x4096 over 8 weight matrices)
    on two streams and disjoint SM partitions; die-split against oblivious (lowest ids / the rest)."""
    for rec in config5_records(topo):
        emit(rec, fh)


def config5_records(topo, splits=((74, 74), (110, 38)), modes=("die_split", "gpc_spread", "oblivious"), n_alone=3, n_both=5):
    """The measurements of config5 as a generator of records (bench.py takes a trimmed set of them)."""
    Mp, Md, N, K = 8192, 32, 4096, 4096
    Ap, Bp = inputs.gemm_inputs(Mp, N, K)
    dAp, dBp = dev_bf16(Ap), dev_bf16(Bp)
    dCp = torch.empty((Mp, N), dtype=torch.float32, device="cuda")
    Ad = inputs.uniform_bf16(Md, K, 77)
    dAd = dev_bf16(Ad)
    Wd = [dev_bf16(inputs.uniform_bf16(K, N, 100 + i)) for i in range(8)]
    dCd = torch.empty((Md, N), dtype=torch.float32, device="cuda")
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    flops_p = 2.0 * Mp * N * K
    bytes_d = K * N * 2 + Md * K * 2 + Md * N * 4
    pre_kw = dict(M=Mp, N=N, K=K, tile_m=256, tile_n=256, raster_group=4)   # both partitions hold whole TPCs: block pairs
    dec_kw = dict(M=Md, N=N, K=K, tile_m=32, tile_n=128, k_splits=8, splitk_in_memory=1)
    for split in splits:
        for mode in modes:
            kind = ag.AG_OBLIVIOUS if mode == "oblivious" else ag.AG_DIE_COMPACT
            sel = 1 if mode == "gpc_spread" else 0      # whole TPCs dealt over the GPCs of both dies
            plan_p = ag.sched_build(topo, None, split[0], ag.make_policy(kind=kind, preferred_die=0, sm_select=sel, **pre_kw))
            taken = [int(s) for s in plan_p.parsed()["sm_list"]]
            plan_d = ag.sched_build(topo, None, split[1], ag.make_policy(kind=kind, avoid=taken, sm_select=sel, **dec_kw))
            n_pre, n_dec = 6, 6 * 8 * 4

            def pre():
                ag.gemm_persistent(dAp.data_ptr(), dBp.data_ptr(), dCp.data_ptr(), Mp, N, K, plan_p, s1.cuda_stream)

            def dec(i):
                ag.gemm_persistent(dAd.data_ptr(), Wd[i % 8].data_ptr(), dCd.data_ptr(), Md, N, K, plan_d, s2.cuda_stream)

            def run(do_pre, do_dec):
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
                torch.cuda.synchronize()
                if do_pre:
                    ev[0].record(s1)
                if do_dec:
                    ev[2].record(s2)
                # interleave the launches so that both streams are fed from the start
                for i in range(max(n_pre, n_dec)):
                    if do_pre and i < n_pre:
                        pre()
                    if do_dec and i < n_dec:
                        dec(i)
                if do_pre:
                    ev[1].record(s1)
                if do_dec:
                    ev[3].record(s2)
                torch.cuda.synchronize()
                tp = ev[0].elapsed_time(ev[1]) / n_pre if do_pre else None
                td = ev[2].elapsed_time(ev[3]) / n_dec if do_dec else None
                return tp, td

            for _ in range(2):
                run(True, True)
            alone_p = np.median([run(True, False)[0] for _ in range(n_alone)])
            alone_d = np.median([run(False, True)[1] for _ in range(n_alone)])
            both = [run(True, True) for _ in range(n_both)]
            ov_p = np.median([x[0] for x in both])
            ov_d = np.median([x[1] for x in both])
            assert plan_p.last_status() == ag.AG_OK and plan_d.last_status() == ag.AG_OK
            yield dict(config=5, split=list(split), partition=mode,
                       prefill_tflops=dict(alone=flops_p / (alone_p * 1e-3) / 1e12, overlapped=flops_p / (ov_p * 1e-3) / 1e12),
                       decode_gbs=dict(alone=bytes_d / (alone_d * 1e-3) / 1e9, overlapped=bytes_d / (ov_d * 1e-3) / 1e9),
                       prefill_set=sm_set_summary(topo, plan_p), decode_set=sm_set_summary(topo, plan_d),
                       note="decode time per GEMM includes the hand-over between back-to-back launches")


# ---------------------------------------------------------------------------------------------
def config5_attention(fh, topo):
    """The serving split of the paper's multiplexing study with attention as the decode side: a prefill-like GEMM
    (8192x4096x4096, block pairs) on one SM partition and decode attention (batch 128, 512 keys, 8 KV heads, 32 query
    heads) on the rest, on two streams.  Die split with die-local KV pages against the GPC-spread and the oblivious
    partitions with interleaved pages."""
    Mp, N, K = 8192, 4096, 4096
    Ap, Bp = inputs.gemm_inputs(Mp, N, K)
    dAp, dBp = dev_bf16(Ap), dev_bf16(Bp)
    dCp = torch.empty((Mp, N), dtype=torch.float32, device="cuda")
    B, Hq, Hkv, L, D = 128, 32, 8, 512, 128
    dK = torch.randn((B, Hkv, L, D), dtype=torch.bfloat16, device="cuda")
    dV = torch.randn((B, Hkv, L, D), dtype=torch.bfloat16, device="cuda")
    dQ = torch.randn((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    dO = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    kv_bytes = 2 * B * Hkv * L * D * 2
    algo = kv_bytes + B * Hq * D * 6
    dst_bytes = 2 * kv_bytes + (16 << 20)
    dst = ag.aligned_device_bytes(dst_bytes)
    amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    flops_p = 2.0 * Mp * N * K
    pre_kw = dict(M=Mp, N=N, K=K, tile_m=256, tile_n=256, raster_group=4)
    att_kw = dict(M=Hq // Hkv, N=128 * B * Hkv, K=L, tile_m=16, tile_n=128, k_splits=1)
    for split in ((74, 74), (110, 38)):
        for mode, placement in (("die_split", ag.KV_LOCAL), ("die_split", ag.KV_INTERLEAVED), ("gpc_spread", ag.KV_LOCAL),
                                ("gpc_spread", ag.KV_INTERLEAVED), ("oblivious", ag.KV_INTERLEAVED)):
            kind = ag.AG_OBLIVIOUS if mode == "oblivious" else ag.AG_DIE_COMPACT
            sel = 1 if mode == "gpc_spread" else 0
            plan_p = ag.sched_build(topo, None, split[0], ag.make_policy(kind=kind, preferred_die=0, sm_select=sel, **pre_kw))
            taken = [int(s) for s in plan_p.parsed()["sm_list"]]
            plan_d = ag.sched_build(topo, None, split[1], ag.make_policy(kind=kind, avoid=taken, sm_select=sel, **att_kw))
            kv = ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L, plan_d, amap, dst.data_ptr(), dst_bytes, placement)
            n_pre, n_dec = 6, 6 * 12

            def pre():
                ag.gemm_persistent(dAp.data_ptr(), dBp.data_ptr(), dCp.data_ptr(), Mp, N, K, plan_p, s1.cuda_stream)

            def dec():
                ag.attention_decode(dQ.data_ptr(), kv, None, dO.data_ptr(), B, Hq, plan_d, s2.cuda_stream)

            def run(do_pre, do_dec):
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
                torch.cuda.synchronize()
                if do_pre:
                    ev[0].record(s1)
                if do_dec:
                    ev[2].record(s2)
                for i in range(max(n_pre, n_dec)):
                    if do_pre and i < n_pre:
                        pre()
                    if do_dec and i < n_dec:
                        dec()
                if do_pre:
                    ev[1].record(s1)
                if do_dec:
                    ev[3].record(s2)
                torch.cuda.synchronize()
                tp = ev[0].elapsed_time(ev[1]) / n_pre if do_pre else None
                td = ev[2].elapsed_time(ev[3]) / n_dec if do_dec else None
                return tp, td

            for _ in range(2):
                run(True, True)
            alone_p = np.median([run(True, False)[0] for _ in range(3)])
            alone_d = np.median([run(False, True)[1] for _ in range(3)])
            both = [run(True, True) for _ in range(5)]
            ov_p = np.median([x[0] for x in both])
            ov_d = np.median([x[1] for x in both])
            assert plan_p.last_status() == ag.AG_OK and plan_d.last_status() == ag.AG_OK
            emit(dict(config="5_attention", split=list(split), partition=mode,
                      kv_pages={ag.KV_LOCAL: "die_local", ag.KV_INTERLEAVED: "interleaved"}[placement],
                      kv_local_fraction=kv.info()["local_fraction"],
                      prefill_tflops=dict(alone=flops_p / (alone_p * 1e-3) / 1e12, overlapped=flops_p / (ov_p * 1e-3) / 1e12),
                      decode_gbs=dict(alone=algo / (alone_d * 1e-3) / 1e9, overlapped=algo / (ov_d * 1e-3) / 1e9),
                      decode_us=dict(alone=alone_d * 1e3, overlapped=ov_d * 1e3),
                      prefill_set=sm_set_summary(topo, plan_p), decode_set=sm_set_summary(topo, plan_d)), fh)
            del kv


# ---------------------------------------------------------------------------------------------
RASTER_ARMS = [(g, name) for g in (1, 2, 4, 8, 16, 32) for name in ("oblivious", "die_compact")]


def raster(fh, topo, traffic_only=False):
    """Raster-group sweep of the headline GEMM (8192^3, 256x256 units on block pairs): TFLOP/s per group height and
    policy.  With traffic_only every arm is launched exactly once, in the order of RASTER_ARMS, so that a profiler's
    launch list can be matched to the arms (DRAM bytes per launch)."""
    M = N = K = 8192
    A, B = inputs.gemm_inputs(M, N, K)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    flops = 2.0 * M * N * K
    plans = {}
    for g, name in RASTER_ARMS:
        kind = ag.AG_OBLIVIOUS if name == "oblivious" else ag.AG_DIE_COMPACT
        plans[(g, name)] = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=kind, M=M, N=N, K=K, tile_m=256, tile_n=256,
                                                                                raster_group=g))
    if traffic_only:
        for i, (k, plan) in enumerate(plans.items()):
            ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
            torch.cuda.synchronize()
            emit(dict(config="raster_traffic", launch=i, raster_group=k[0], policy=k[1]), fh)
        return
    acc = {k: [] for k in plans}
    for _ in range(3):
        for k, plan in plans.items():
            acc[k] += time_launches(lambda: ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan),
                                    warmup=2, iters=6, batches=1)
    for (g, name), v in acc.items():
        emit(dict(config="raster", raster_group=g, policy=name, tflops=flops / (float(np.median(v)) * 1e-3) / 1e12), fh)


def raster_burst(fh, topo, groups=(1, 2, 4, 6, 8, 12, 16, 32), steps=40, warmup=5, idle_s=2.0, runs=2):
    """The raster-group sweep of the headline GEMM in burst state: every arm after its own idle pause, so that all of
    its steps run at the full clock, where the kernel is bound by what the L2 side delivers and the order of the units
    (and which die takes which) shows in the throughput."""
    import time
    M = N = K = 8192
    A, B = inputs.gemm_inputs(M, N, K)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.float32, device="cuda")
    flops = 2.0 * M * N * K

    def burst(plan):
        torch.cuda.synchronize()
        time.sleep(idle_s)
        for _ in range(warmup):
            ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan)
        e1.record()
        torch.cuda.synchronize()
        return flops / (e0.elapsed_time(e1) / steps * 1e-3) / 1e12

    for kind, name in ((ag.AG_DIE_COMPACT, "die_compact"), (ag.AG_OBLIVIOUS, "oblivious")):
        for g in groups:
            plan = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=kind, M=M, N=N, K=K, tile_m=256, tile_n=256, raster_group=g))
            emit(dict(config="raster_burst", policy=name, raster_group=g, tflops=[burst(plan) for _ in range(runs)]), fh)


# ---------------------------------------------------------------------------------------------
def time_queued(fn, warmup=3, iters=16, batches=3):
    """Median GPU time per call in ms.  The calls of a batch are queued behind a device-side blocker, so that
    host-side launch cost is not on the clock (the kernels here take tens of microseconds), and the batch is
    bracketed by one event pair."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    s = torch.cuda.current_stream()
    out = []
    for _ in range(batches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(int(2e7))
        e0.record(s)
        for _ in range(iters):
            fn()
        e1.record(s)
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) / iters)
    return float(np.median(out))


def groupgemm(fh, topo, seeds=(1, 2, 3, 4, 5)):
    """The decode-shaped settings of the paper's GroupGEMM study (its workload appendix): (G, M) in
    {(32, 20), (6, 20)}, (N, K) in {(6144, 7168), (7168, 3072), (4096, 4096), (4096, 2048)}, rows per
    expert M_i = floor(M U_i), U_i ~ U(0.7, 1.3).  Random weights are made on the device (timing only;
    parity is covered by the tests)."""
    for G, M in ((32, 20), (6, 20)):
        for N, K in ((6144, 7168), (7168, 3072), (4096, 4096), (4096, 2048)):
            tiles = G * N // 128
            ksp = 1
            while tiles * ksp < 6 * topo.n_sm and K // 64 // (2 * ksp) >= 4:
                ksp *= 2
            Bs = [torch.randn((K, N), dtype=torch.bfloat16, device="cuda") for _ in range(G)]
            w_bytes = G * K * N * 2
            dst_bytes = 2 * w_bytes + (16 << 20)
            dst = ag.aligned_device_bytes(dst_bytes)
            amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
            for seed in seeds:
                rows = inputs.group_rows(G, M, seed)
                total = int(rows.sum())
                dA = torch.randn((total, K), dtype=torch.bfloat16, device="cuda")
                dC = torch.empty((total, N), dtype=torch.float32, device="cuda")
                kw = dict(M=int(rows.max()), N=G * N, K=K, tile_m=32, tile_n=128, k_splits=ksp, splitk_in_memory=1)
                plan_obl = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_OBLIVIOUS, **kw))
                plan_dc = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
                packed = ag.pack_weights_grouped([b.data_ptr() for b in Bs], K, N, plan_dc, amap, dst.data_ptr(), dst_bytes)
                bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=packed.page_table())
                plan_rem = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, invert_affinity=1, b=bop, **kw))
                # the units shared equally between the dies instead of by SM count (each die's memory is equally fast)
                plan_eq = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, die_quota=1, **kw))
                dst_eq = ag.aligned_device_bytes(dst_bytes)
                amap_eq = ag.affinity_probe(dst_eq.data_ptr(), dst_bytes, topo)
                packed_eq = ag.pack_weights_grouped([b.data_ptr() for b in Bs], K, N, plan_eq, amap_eq, dst_eq.data_ptr(), dst_bytes)
                desc_rm = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in Bs], N, K, 32)
                algo = w_bytes + total * K * 2 + total * N * 4
                res = {}
                for name, pk, plan in (("rowmajor_oblivious", None, plan_obl), ("rowmajor_die_compact", None, plan_dc),
                                       ("packed_die_local", packed, plan_dc), ("packed_die_local_equal_quota", packed_eq, plan_eq),
                                       ("packed_remote", packed, plan_rem)):
                    ms = time_queued(lambda: ag.gemm_persistent_grouped(desc_rm, pk, plan))
                    assert plan.last_status() == ag.AG_OK
                    res[name] = algo / (ms * 1e-3) / 1e9
                emit(dict(config="groupgemm", G=G, M=M, N=N, K=K, seed=seed, rows_total=total, k_splits=ksp,
                          weight_gb=w_bytes / 1e9, gbs=res, local_over_remote=res["packed_die_local"] / res["packed_remote"],
                          local_over_rowmajor_oblivious=res["packed_die_local"] / res["rowmajor_oblivious"]), fh)
                del packed, packed_eq, dst_eq, amap_eq, desc_rm, dA, dC
            del Bs, dst, amap
            torch.cuda.empty_cache()


def groupgemm_dense(fh, topo, seeds=(1,)):
    """The settings of the paper's GroupGEMM study with many rows per expert: (G, M) in {(32, 192), (6, 1024)},
    same (N, K) list; block pairs with per-expert views."""
    for G, M in ((32, 192), (6, 1024)):
        for N, K in ((6144, 7168), (7168, 3072), (4096, 4096), (4096, 2048)):
            Bs = [torch.randn((K, N), dtype=torch.bfloat16, device="cuda") for _ in range(G)]
            w_bytes = G * K * N * 2
            dst_bytes = 2 * w_bytes + (16 << 20)
            dst = ag.aligned_device_bytes(dst_bytes)
            amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
            for seed in seeds:
                rows = inputs.group_rows(G, M, seed)
                total = int(rows.sum())
                dA = torch.randn((total, K), dtype=torch.bfloat16, device="cuda")
                dC = torch.empty((total, N), dtype=torch.float32, device="cuda")
                kw = dict(M=int(rows.max()), N=G * N, K=K, tile_m=256, tile_n=256, raster_group=1)
                plan_obl = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_OBLIVIOUS, **kw))
                plan_dc = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
                packed = ag.pack_weights_grouped([b.data_ptr() for b in Bs], K, N, plan_dc, amap, dst.data_ptr(), dst_bytes)
                bop = dict(offset=0, row_stride=0, elem_bytes=2, layout=ag.AG_LAYOUT_PAGED, page_table=packed.page_table())
                plan_rem = ag.sched_build(topo, amap, topo.n_sm, ag.make_policy(kind=ag.AG_AFFINITY, invert_affinity=1, b=bop, **kw))
                desc = ag.GroupDesc(dA.data_ptr(), dC.data_ptr(), rows, [b.data_ptr() for b in Bs], N, K, 256)
                flops = 2.0 * total * N * K
                algo = w_bytes + total * K * 2 + total * N * 4
                res = {}
                for name, pk, plan in (("rowmajor_oblivious", None, plan_obl), ("rowmajor_die_compact", None, plan_dc),
                                       ("packed_die_local", packed, plan_dc), ("packed_remote", packed, plan_rem)):
                    ms = time_queued(lambda: ag.gemm_persistent_grouped(desc, pk, plan))
                    assert plan.last_status() == ag.AG_OK
                    res[name] = dict(tflops=flops / (ms * 1e-3) / 1e12, gbs=algo / (ms * 1e-3) / 1e9, us=ms * 1e3)
                emit(dict(config="groupgemm_dense", G=G, M=M, N=N, K=K, seed=seed, rows_total=total, weight_gb=w_bytes / 1e9,
                          flop_per_byte=flops / algo, results=res,
                          local_over_remote=res["packed_remote"]["us"] / res["packed_die_local"]["us"],
                          local_over_rowmajor_oblivious=res["rowmajor_oblivious"]["us"] / res["packed_die_local"]["us"]), fh)
                del packed, desc, dA, dC
            del Bs, dst, amap
            torch.cuda.empty_cache()


def gpc_bandwidth(fh, topo):
    """Section 5.1.2 (per-GPC L2 bandwidth figure): aggregate L2 read bandwidth of k SMs taken from one GPC
    against k SMs spread over all GPCs."""
    by_gpc = {g: [s for s in range(topo.n_sm) if topo.gpc[s] == g] for g in range(topo.n_gpc)}
    biggest = max(by_gpc, key=lambda g: len(by_gpc[g]))
    spread, i = [], 0
    while len(spread) < len(by_gpc[biggest]):
        for g in range(topo.n_gpc):
            if 2 * i + 1 < len(by_gpc[g]):
                spread += by_gpc[g][2 * i:2 * i + 2]
        i += 1
    for k in range(2, len(by_gpc[biggest]) + 1, 2):
        emit(dict(config="gpc_bandwidth", n_sms=k, gpc=biggest,
                  same_gpc_gbs=ag.probe_l2_bandwidth(by_gpc[biggest][:k]) / 1e9,
                  spread_gbs=ag.probe_l2_bandwidth(spread[:k]) / 1e9), fh)


def latency_histograms(fh, topo):
    """Section 6.1.1 (latency histogram figures): samples from one SM of each die over 1024 lines; the first
    sample of a line after the L2 invalidation is an HBM access, a plain reload is an L2 hit."""
    sms = [0, next(s for s in range(topo.n_sm) if topo.die[s] == 1)]
    edges = list(range(150, 1301, 50))
    for sm in sms:
        hbm = ag.probe_latency_samples(sm, mode=0, n_lines=1024, reps=1)[:, 0]
        l2 = ag.probe_latency_samples(sm, mode=0, n_lines=1024, reps=4)[:, 1:].min(axis=1)   # later samples: served by L2
        for name, v in (("first_touch_after_invalidate", hbm), ("repeat_after_invalidate", l2)):
            hist, _ = np.histogram(v, bins=edges)
            emit(dict(config="latency", sm=int(sm), die=int(topo.die[sm]), kind=name, bin_edges_cycles=edges,
                      counts=[int(x) for x in hist], median=float(np.median(v))), fh)


def cluster_sets(fh, topo, budgets=(64, 72, 96), n_subsets=16):
    """Cluster eligibility of equal-size SM sets (Sections 5.1.1, 7.3): how many thread-block clusters of 4 and 8 blocks
    a set can host.  Two counts per set: the capacity computed from the map (per GPC floor(normal SMs / c)), and the
    number of clusters of one full-chip launch that the hardware placed wholly inside the set."""
    full = ag.sched_build(topo, None, topo.n_sm, ag.make_policy(kind=ag.AG_DIE_COMPACT, M=4096, N=4096, K=4096))
    for c in (4, 8):
        cap_chip = full.cluster_capacity(topo, c)
        lay = ag.probe_cluster_layout(c, cap_chip)[:topo.n_sm]
        clusters = {}
        for s in range(topo.n_sm):
            if lay[s] >= 0:
                clusters.setdefault(int(lay[s]), []).append(s)

        def inside(sms):
            ss = set(sms)
            return sum(1 for m in clusters.values() if len(m) == c and set(m) <= ss)
        for b in budgets:
            kw = dict(M=4096, N=4096, K=4096)
            sets = {f"random_{i}": ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, seed=i, **kw)) for i in range(1, n_subsets + 1)}
            sets["lowest_ids"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, **kw))
            sets["highest_ids"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_OBLIVIOUS, avoid=list(range(topo.n_sm - b)), **kw))
            sets["die_compact_tpc"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, **kw))
            sets["die_compact_cluster"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, cluster_size=c, **kw))
            sets["gpc_spread_cluster"] = ag.sched_build(topo, None, b, ag.make_policy(kind=ag.AG_DIE_COMPACT, sm_select=1, cluster_size=c, **kw))
            res = {}
            for n, pl in sets.items():
                sms = [int(x) for x in pl.parsed()["sm_list"]]
                res[n] = dict(capacity=pl.cluster_capacity(topo, c), placed_inside=inside(sms))
            rnd = [res[f"random_{i}"] for i in range(1, n_subsets + 1)]
            emit(dict(config="cluster_sets", cluster_size=c, sm_budget=b, ideal=b // c, chip_capacity=cap_chip,
                      clusters_seen=len(clusters),
                      random_capacity=dict(min=min(r["capacity"] for r in rnd), max=max(r["capacity"] for r in rnd),
                                           median=float(np.median([r["capacity"] for r in rnd]))),
                      random_placed_inside=dict(min=min(r["placed_inside"] for r in rnd), max=max(r["placed_inside"] for r in rnd)),
                      **{n: res[n] for n in ("lowest_ids", "highest_ids", "die_compact_tpc", "die_compact_cluster", "gpc_spread_cluster")}), fh)


def attention(fh, topo, shapes=((128, 32, 8, 512), (256, 32, 8, 1024), (16, 32, 8, 8192), (4, 32, 8, 32768)), budgets=None, overlap=1):
    """Decode attention over a paged KV cache (Section 6.4's die-local KV direction): batch B, H_q query heads over
    H_kv KV heads, L keys of 128 dimensions per head; pages of a unit on the die of the SM that owns it (local),
    on the other die (remote) or wherever the allocation put them (interleaved).  GB/s of KV bytes."""
    budgets = budgets or (topo.n_sm, topo.n_sm // 2, topo.n_sm // 4)
    D = 128
    for B, Hq, Hkv, L in shapes:
        dK = torch.randn((B, Hkv, L, D), dtype=torch.bfloat16, device="cuda")
        dV = torch.randn((B, Hkv, L, D), dtype=torch.bfloat16, device="cuda")
        dQ = torch.randn((B, Hq, D), dtype=torch.bfloat16, device="cuda")
        dO = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
        kv_bytes = 2 * B * Hkv * L * D * 2
        algo = kv_bytes + B * Hq * D * (2 + 4)
        dst_bytes = 2 * kv_bytes + (16 << 20)
        dst = ag.aligned_device_bytes(dst_bytes)
        amap = ag.affinity_probe(dst.data_ptr(), dst_bytes, topo)
        lib_us = None
        try:    # context: the library's fused attention on the same shapes (row-major cache)
            q4 = dQ.view(B, Hq, 1, D)
            f = lambda: torch.nn.functional.scaled_dot_product_attention(q4, dK, dV, enable_gqa=True)
            lib_us = time_queued(f) * 1e3
        except Exception as e:  # noqa: BLE001
            lib_us = str(e)[:80]
        for b in budgets:
            for both in ((0, 1) if b < topo.n_sm else (0,)):
                n_chunks = (L + 1023) // 1024      # requests over 1024 keys run as one unit per chunk of 1024 keys
                kw = dict(kind=ag.AG_DIE_COMPACT, M=Hq // Hkv, N=128 * B * Hkv * n_chunks, K=L, tile_m=16, tile_n=128, k_splits=1,
                          sm_select=1 if both else 0, overlap_launches=overlap)
                plan = ag.sched_build(topo, None, b, ag.make_policy(**kw))
                plan_eq = ag.sched_build(topo, None, b, ag.make_policy(die_quota=1, **kw))   # units shared equally between the dies
                res, info = {}, {}
                for name, pl, pn in (("local", ag.KV_LOCAL, plan), ("local_equal_quota", ag.KV_LOCAL, plan_eq), ("remote", ag.KV_REMOTE, plan),
                                     ("interleaved", ag.KV_INTERLEAVED, plan)):
                    kv = ag.kv_pack(dK.data_ptr(), dV.data_ptr(), B, Hkv, L, pn, amap, dst.data_ptr(), dst_bytes, pl)
                    ms = time_queued(lambda: ag.attention_decode(dQ.data_ptr(), kv, None, dO.data_ptr(), B, Hq, pn))
                    assert pn.last_status() == ag.AG_OK
                    res[name] = dict(us=ms * 1e3, gbs=algo / (ms * 1e-3) / 1e9)
                    info[name] = kv.info()["local_fraction"]
                    del kv
                emit(dict(config="attention", B=B, H_q=Hq, H_kv=Hkv, L=L, kv_gb=kv_bytes / 1e9, sm_budget=b,
                          sm_set="gpc_spread" if both else "die_compact", sets=sm_set_summary(topo, plan), results=res,
                          local_fraction=info, local_over_remote=res["remote"]["us"] / res["local"]["us"],
                          local_over_interleaved=res["interleaved"]["us"] / res["local"]["us"],
                          overlap_launches=int(bool(overlap)), library_sdpa_us=lib_us), fh)
        del dst, amap, dK, dV
        torch.cuda.empty_cache()


def attention_sweep(fh, topo):
    """The decode sweep of the paper's attention study (workload appendix): one query token per request, 32 query
    heads of 128 dimensions on 32 (MHA) or 8 (GQA) KV heads, batch 1 to 64, keys from 512 doubling, full chip;
    working sets up to 8.6 GB here."""
    shapes = []
    for Hkv in (32, 8):
        for B in (1, 8, 64):
            L = 512
            while 4 * B * L * Hkv * 128 <= 8.6e9 and L <= (1 << 17):
                shapes.append((B, 32, Hkv, L))
                L *= 4
    attention(fh, topo, shapes=tuple(shapes), budgets=(topo.n_sm,))


def copy_ring(fh, topo):
    """What sets policy.ring_stages: the copy side of the streaming kernels alone (rings of 32 KB stages filled by bulk
    copies) on 1, 37, 74 and all SMs, over the ring depth, the stage size and the time a stage is held."""
    nbytes = 4 << 30
    buf = ag.aligned_device_bytes(nbytes)
    for n_blocks in (1, 37, 74, topo.n_sm):
        share = nbytes if n_blocks > 1 else 256 << 20
        for stage_bytes, depths in ((32768, (1, 2, 3, 4, 5, 6)), (16384, (2, 4, 8)), (65536, (1, 2, 3))):
            for stages in depths:
                for hold_ns in (0, 400):
                    producers = min(stages, 3)
                    gbs = ag.probe_ring_bandwidth(buf.data_ptr(), share, n_blocks, stages, stage_bytes, producers, hold_ns) / 1e9
                    emit(dict(config="copy_ring", n_blocks=n_blocks, stage_bytes=stage_bytes, stages=stages, producers=producers,
                              hold_ns=hold_ns, in_flight_mb=n_blocks * stages * stage_bytes / 1e6, gbs=gbs,
                              gbs_per_sm=gbs / n_blocks), fh)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", required=True)
    ap.add_argument("--out", default=None)
    args = ap.parse_args()
    fh = open(args.out, "a") if args.out else None
    topo = ag.topo_discover()
    emit(dict(config="topology", n_sm=topo.n_sm, die_sm_count=list(topo.die_sm_count),
              gpc_sm_count=list(topo.gpc_sm_count[:topo.n_gpc]), gpc_die=list(topo.gpc_die[:topo.n_gpc]),
              lat_near_cycles=topo.lat_near_cycles, lat_far_cycles=topo.lat_far_cycles), fh)
    {"3": config3, "4": config4, "5": config5, "raster": raster, "groupgemm": groupgemm, "groupgemm_dense": groupgemm_dense,
     "gpc_bandwidth": gpc_bandwidth, "latency": latency_histograms, "cluster_sets": cluster_sets, "attention": attention,
     "raster_traffic": lambda f, t: raster(f, t, traffic_only=True), "5_attention": config5_attention,
     "attention_sweep": attention_sweep, "copy_ring": copy_ring, "raster_burst": raster_burst}[args.config](fh, topo)


if __name__ == "__main__":
    sys.exit(main())

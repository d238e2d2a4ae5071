"""CPU-only: the C-ABI library loads and exports every symbol the header declares; host-side
logic that needs no device (union-find over cluster observations, die split from latency
vectors, the bandwidth-gain decision rule)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2609_24270_b200 import binding as ag
from paper_2609_24270_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "asymgemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\([^;{}]*\)\s*;", text)))


def test_every_declared_symbol_is_exported():
    L = ag.lib()
    names = declared_functions()
    assert {"topo_discover", "affinity_probe", "sched_build", "gemm_persistent"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(ag.EXPORTED)


def test_struct_sizes_match_header_layout():
    # int32 x4 + 3 arrays of 256 int32 + 256 bytes + 2 + 32 + 32 int32 + 9 x 4 bytes
    assert ag.C.sizeof(ag.TopoMap) == 16 + 3 * 1024 + 256 + 4 * (2 + 32 + 32) + 36
    assert ag.C.sizeof(ag.OperandDesc) == 48
    assert ag.C.sizeof(ag.Policy) == 12 * 4 + 8 + 8 + 8 + 8 + 8 + 8 + 32 + 3 * 48


def test_null_arguments_are_rejected_without_a_device():
    L = ag.lib()
    assert L.topo_discover(None) == ag.AG_ERR_ARG
    assert L.sched_build(None, None, 1, None, None) == ag.AG_ERR_ARG
    assert L.gemm_persistent(None, None, None, 1, 1, 1, None, None) == ag.AG_ERR_ARG
    assert L.affinity_probe(None, 4096, None) != ag.AG_OK
    bw = C.c_double()
    for bad in [(None, 1 << 20, 4, 4, 32768, 2, 0), (4096, 1 << 20, 4, 9, 16384, 2, 0), (4096, 1 << 20, 4, 4, 5000, 2, 0),
                (4096, 1 << 20, 4, 2, 32768, 3, 0), (4096, 1 << 20, 4, 8, 32768, 2, 0), (4096, 1 << 20, 0, 4, 32768, 2, 0),
                (4104, 1 << 20, 4, 4, 32768, 2, 0), (4096, 1 << 16, 4, 4, 32768, 2, 0), (4096, 1 << 20, 4, 4, 32768, 2, -1)]:
        assert L.ag_probe_ring_bandwidth(*bad, C.byref(bw)) == ag.AG_ERR_ARG, bad
    assert ag.strerror(ag.AG_ERR_TIMEOUT) != ag.strerror(ag.AG_OK)


def synthetic_observations(topo, seed=0, far=920, near=552, n_ref=64):
    rng = np.random.default_rng(seed)
    clusters = []
    for cs in range(3, 9):
        for g in range(topo["n_gpc"]):
            members = [s for s in range(topo["n_sm"]) if topo["gpc"][s] == g and not topo["is_random"][s]]
            for _ in range(6):
                clusters.append(list(rng.choice(members, size=cs, replace=False)))
    chunk_die = rng.integers(0, 2, size=n_ref)
    chunk_die[:2] = [0, 1]
    lat = np.empty((topo["n_sm"], n_ref), dtype=np.uint32)
    for s in range(topo["n_sm"]):
        base = np.where(chunk_die == topo["die"][s], near, far)
        lat[s] = base + rng.integers(-15, 40, size=n_ref)
    return clusters, lat


@pytest.mark.parametrize("die0", [70, 74])
def test_topology_from_recorded_observations(die0):
    topo = inputs.synthetic_topo(die0_sms=die0, seed=5)
    if topo["die"][0] != 0:                                   # die 0 is by definition the die of SM 0
        topo["die"] = 1 - topo["die"]
    clusters, lat = synthetic_observations(topo)
    m = ag.topo_from_observations(148, clusters, lat).as_dict()
    assert m["n_sm"] == 148 and m["n_gpc"] == 8
    assert m["die"] == [int(d) for d in topo["die"]]
    assert m["is_random"] == [int(r) for r in topo["is_random"]]
    assert sum(m["die_sm_count"]) == 148 and m["die_sm_count"][0] == int((topo["die"] == 0).sum())
    # GPC classes equal the synthetic ones up to relabelling, for the normal SMs
    lab = {}
    for s in range(148):
        if topo["is_random"][s]:
            assert m["gpc"][s] == -1
        else:
            assert lab.setdefault(int(topo["gpc"][s]), m["gpc"][s]) == m["gpc"][s]
    assert len(set(lab.values())) == 8
    assert all(m["tpc"][s] == s // 2 for s in range(148))
    assert abs(m["lat_near_cycles"] - 560) < 40 and abs(m["lat_far_cycles"] - 930) < 40
    assert m["n_unplaced"] == 20


def test_noisy_latency_is_refused():
    topo = inputs.synthetic_topo()
    clusters, lat = synthetic_observations(topo)
    flat = np.full_like(lat, 600)
    L = ag.lib()
    m = ag.TopoMap()
    off = np.zeros(1, dtype=np.int32)
    st = L.ag_topo_from_observations(148, None, off.ctypes.data, 0, flat.ctypes.data, 64, ag.C.byref(m))
    assert st == ag.AG_ERR_NOISY_PROBE


def test_bandwidth_gain_rule():
    # one GPC gains far less than a TPC's own bandwidth: that GPC holds the TPC (Section 5.1.2)
    assert ag.topo_place_by_gain([200e9, 195e9, 60e9, 205e9], 200e9) == 2
    # every GPC gains a full TPC's worth: nothing contended, undecided
    assert ag.topo_place_by_gain([200e9, 195e9, 199e9, 205e9], 200e9) == -1
    # two equally contended candidates: ambiguous
    assert ag.topo_place_by_gain([60e9, 61e9, 200e9], 200e9) == -1


def test_topo_map_file_roundtrip(tmp_path):
    topo = inputs.synthetic_topo(die0_sms=72, seed=3)
    m = ag.TopoMap.from_dict(topo)
    path = str(tmp_path / "topo.bin")
    ag.topo_save(m, path)
    back = ag.topo_load(path)
    assert bytes(back) == bytes(m)
    # a truncated or foreign file is refused
    blob = open(path, "rb").read()
    open(path, "wb").write(blob[:-5])
    with pytest.raises(ag.AgError):
        ag.topo_load(path)
    open(path, "wb").write(b"NOTATOPO" + blob[8:])
    with pytest.raises(ag.AgError):
        ag.topo_load(path)
    with pytest.raises(ag.AgError):
        ag.topo_load(str(tmp_path / "missing.bin"))


def test_ctypes_structs_match_the_header_as_a_c_compiler_sees_it(tmp_path):
    """The header is plain C: compile it with gcc and compare sizes and field offsets with the binding."""
    import subprocess
    fields = {
        "ag_topo_map": ["n_sm", "tpc", "gpc", "die", "is_random", "die_sm_count", "gpc_sm_count", "gpc_die",
                        "lat_near_cycles", "l2_near_cycles", "n_unplaced", "device", "sm_clock_khz", "flags"],
        "ag_operand_desc": ["present", "layout", "offset", "row_stride", "elem_bytes", "page_table", "n_pages"],
        "ag_policy": ["kind", "M", "tile_m", "k_splits", "k_unit", "raster_group", "preferred_die", "invert_affinity",
                      "static_assign", "seed", "min_margin", "splitk_in_memory", "sm_select", "pair_lists", "overlap_launches", "cluster_size", "die_quota", "decode_shaped", "ring_stages",
                      "avoid_sm_mask", "a", "b", "c"],
    }
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "asymgemm.h"', 'int main(void) {']
    for sname, fl in fields.items():
        lines.append(f'  printf("{sname} %zu\\n", sizeof({sname}));')
        for f in fl:
            lines.append(f'  printf("{sname}.{f} %zu\\n", offsetof({sname}, {f}));')
    lines += ['  return 0;', '}']
    src = tmp_path / "abi.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "abi"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    seen = dict(l.split() for l in subprocess.check_output([str(exe)], text=True).splitlines())
    py = {"ag_topo_map": ag.TopoMap, "ag_operand_desc": ag.OperandDesc, "ag_policy": ag.Policy}
    for sname, fl in fields.items():
        assert int(seen[sname]) == ag.C.sizeof(py[sname]), sname
        for f in fl:
            assert int(seen[f"{sname}.{f}"]) == getattr(py[sname], f).offset, (sname, f)


def test_suggested_k_splits_follow_the_measurements():
    """Host arithmetic: the settings that measured best (N = K = 8192: 4 splits on the full chip with overlapping launches
    and on 37 SMs, 8 on 74 SMs), and every suggestion is a valid one (no empty split, at least four k-slabs per split)."""
    assert ag.suggest_k_splits(8192, 8192, 148, True) == 4
    assert ag.suggest_k_splits(8192, 8192, 74) == 8
    assert ag.suggest_k_splits(8192, 8192, 37) == 4
    assert ag.suggest_k_splits(128, 64, 148) == 1            # one k-slab cannot be split
    assert ag.suggest_k_splits(0, 0, 0) == 1
    for N, K, b in ((4096, 2048, 148), (1024, 200, 37), (49152, 7168, 148), (384, 12288, 11)):
        ksp = ag.suggest_k_splits(N, K, b)
        n_slab = (K + 63) // 64
        per = -(-n_slab // ksp)
        assert ksp >= 1 and (ksp == 1 or (per >= 4 and (ksp - 1) * per < n_slab))

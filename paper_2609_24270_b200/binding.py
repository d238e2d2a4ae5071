"""ctypes binding over the C ABI declared in include/asymgemm.h (argument marshalling only).

Every step of the path runs inside libasymgemm.so; this module never computes anything
itself and has no fallback: if the library is missing, importing it raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libasymgemm.so")

AG_MAX_SM, AG_MAX_GPC, AG_MAX_DIE, AG_CHUNK_BYTES = 256, 32, 2, 4096
AG_OBLIVIOUS, AG_DIE_COMPACT, AG_AFFINITY = 0, 1, 2
AG_LAYOUT_ROWMAJOR, AG_LAYOUT_PAGED = 0, 1
AG_TOPO_CENSUS, AG_TOPO_CLUSTER, AG_TOPO_LATENCY, AG_TOPO_BANDWIDTH = 1, 2, 4, 8
(AG_OK, AG_ERR_ARG, AG_ERR_CUDA, AG_ERR_UNSUPPORTED_ARCH, AG_ERR_TIMEOUT, AG_ERR_UNMANNED_SM,
 AG_ERR_NOISY_PROBE, AG_ERR_STALE_AMAP, AG_ERR_NOMEM) = range(9)

EXPORTED = [
    "topo_discover", "ag_topo_discover_phases", "ag_topo_from_observations", "ag_topo_place_by_gain",
    "ag_probe_l2_bandwidth", "ag_probe_latency_samples",
    "affinity_probe", "ag_affinity_probe_with_map", "ag_affinity_from_table", "ag_affinity_export",
    "ag_affinity_cycles", "ag_affinity_check_complement", "ag_affinity_fit_hash", "ag_probe_die_bandwidth", "ag_probe_ring_bandwidth", "ag_affinity_destroy",
    "sched_build", "ag_plan_export", "ag_plan_margins", "ag_plan_tile_record", "ag_plan_reset_record",
    "ag_plan_set_grid", "ag_plan_adopted", "ag_cluster_capacity", "ag_probe_cluster_layout", "ag_plan_trace", "ag_plan_unit_times", "ag_last_status", "ag_last_status_where", "ag_suggest_k_splits", "ag_plan_destroy", "gemm_persistent", "ag_pack_weights", "ag_pack_weights_ex", "ag_packed_info", "ag_packed_closed_form", "ag_packed_page_table",
    "ag_packed_destroy", "gemm_persistent_packed", "gemm_persistent_noalloc", "ag_wait_probe", "ag_topo_save",
    "ag_topo_load", "ag_group_desc_create", "ag_group_desc_destroy", "ag_pack_weights_grouped",
    "gemm_persistent_grouped", "ag_strerror", "ag_last_cuda_error",
    "ag_kernel_launch_count", "ag_kv_pack", "ag_kv_info", "ag_kv_append", "ag_kv_destroy", "attention_decode_persistent",
]


class TopoMap(C.Structure):
    _fields_ = [
        ("n_sm", C.c_int32), ("n_tpc", C.c_int32), ("n_gpc", C.c_int32), ("n_die", C.c_int32),
        ("tpc", C.c_int32 * AG_MAX_SM), ("gpc", C.c_int32 * AG_MAX_SM), ("die", C.c_int32 * AG_MAX_SM),
        ("is_random", C.c_uint8 * AG_MAX_SM),
        ("die_sm_count", C.c_int32 * AG_MAX_DIE), ("gpc_sm_count", C.c_int32 * AG_MAX_GPC),
        ("gpc_die", C.c_int32 * AG_MAX_GPC),
        ("lat_near_cycles", C.c_uint32), ("lat_far_cycles", C.c_uint32), ("lat_threshold", C.c_uint32),
        ("l2_near_cycles", C.c_uint32), ("l2_far_cycles", C.c_uint32),
        ("n_unplaced", C.c_int32), ("device", C.c_int32), ("sm_clock_khz", C.c_uint32), ("flags", C.c_uint32),
    ]

    def as_dict(self) -> dict:
        n = self.n_sm
        return dict(n_sm=n, n_tpc=self.n_tpc, n_gpc=self.n_gpc, n_die=self.n_die,
                    tpc=list(self.tpc[:n]), gpc=list(self.gpc[:n]), die=list(self.die[:n]),
                    is_random=list(self.is_random[:n]), die_sm_count=list(self.die_sm_count),
                    gpc_sm_count=list(self.gpc_sm_count[:max(self.n_gpc, 0)]),
                    gpc_die=list(self.gpc_die[:max(self.n_gpc, 0)]),
                    lat_near_cycles=self.lat_near_cycles, lat_far_cycles=self.lat_far_cycles,
                    lat_threshold=self.lat_threshold, l2_near_cycles=self.l2_near_cycles,
                    l2_far_cycles=self.l2_far_cycles, n_unplaced=self.n_unplaced, device=self.device,
                    sm_clock_khz=self.sm_clock_khz, flags=self.flags)

    @classmethod
    def from_dict(cls, d: dict) -> "TopoMap":
        m = cls()
        m.n_sm, m.n_tpc, m.n_gpc, m.n_die = d["n_sm"], d["n_tpc"], d["n_gpc"], d.get("n_die", 2)
        for s in range(d["n_sm"]):
            m.tpc[s], m.gpc[s], m.die[s] = int(d["tpc"][s]), int(d["gpc"][s]), int(d["die"][s])
            m.is_random[s] = int(d["is_random"][s])
        for g in range(d["n_gpc"]):
            m.gpc_die[g] = int(d["gpc_die"][g])
        m.die_sm_count[0] = sum(1 for s in range(d["n_sm"]) if d["die"][s] == 0)
        m.die_sm_count[1] = d["n_sm"] - m.die_sm_count[0]
        m.flags = AG_TOPO_CENSUS | AG_TOPO_CLUSTER | AG_TOPO_LATENCY
        return m


class OperandDesc(C.Structure):
    _fields_ = [("present", C.c_int32), ("layout", C.c_int32), ("offset", C.c_int64),
                ("row_stride", C.c_int64), ("elem_bytes", C.c_int32), ("reserved", C.c_int32),
                ("page_table", C.POINTER(C.c_int32)), ("n_pages", C.c_int64)]


class Policy(C.Structure):
    _fields_ = [("kind", C.c_int32), ("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
                ("tile_m", C.c_int32), ("tile_n", C.c_int32), ("k_splits", C.c_int32), ("k_unit", C.c_int32),
                ("raster_group", C.c_int32), ("preferred_die", C.c_int32), ("invert_affinity", C.c_int32),
                ("static_assign", C.c_int32), ("seed", C.c_uint64), ("min_margin", C.c_int64),
                ("splitk_in_memory", C.c_int32), ("sm_select", C.c_int32), ("pair_lists", C.c_int32), ("overlap_launches", C.c_int32), ("cluster_size", C.c_int32), ("die_quota", C.c_int32), ("decode_shaped", C.c_int32), ("ring_stages", C.c_int32),
                ("avoid_sm_mask", C.c_uint64 * 4),
                ("a", OperandDesc), ("b", OperandDesc), ("c", OperandDesc)]


class AgError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {strerror(status)} (status {status}, cuda error {lib().ag_last_cuda_error()})")


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_24270_b200.build` "
                          "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int32
    L.topo_discover.argtypes = [C.POINTER(TopoMap)]
    L.ag_topo_discover_phases.argtypes = [C.POINTER(TopoMap), C.c_uint32]
    L.ag_topo_from_observations.argtypes = [i32, vp, vp, i32, vp, i32, C.POINTER(TopoMap)]
    L.ag_topo_place_by_gain.argtypes = [C.POINTER(C.c_double), i32, C.c_double]
    L.ag_topo_place_by_gain.restype = i32
    L.ag_probe_latency_samples.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, vp]
    L.ag_probe_l2_bandwidth.argtypes = [C.POINTER(C.c_uint64), C.POINTER(C.c_double)]
    L.affinity_probe.argtypes = [vp, sz, C.POINTER(vp)]
    L.ag_affinity_probe_with_map.argtypes = [vp, sz, C.POINTER(TopoMap), C.POINTER(vp)]
    L.ag_affinity_from_table.argtypes = [vp, sz, vp, sz, C.POINTER(vp)]
    L.ag_affinity_export.argtypes = [vp, vp, sz, C.POINTER(sz)]
    L.ag_affinity_cycles.argtypes = [vp, vp, sz]
    L.ag_affinity_check_complement.argtypes = [vp, C.POINTER(TopoMap), C.POINTER(sz)]
    L.ag_affinity_fit_hash.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(sz)]
    L.ag_probe_die_bandwidth.argtypes = [vp, C.POINTER(TopoMap), C.c_int, C.c_int, C.POINTER(C.c_double)]
    L.ag_probe_ring_bandwidth.argtypes = [vp, sz, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_double)]
    L.ag_affinity_destroy.argtypes = [vp]
    L.ag_affinity_destroy.restype = None
    L.sched_build.argtypes = [C.POINTER(TopoMap), vp, C.c_int, C.POINTER(Policy), C.POINTER(vp)]
    L.ag_plan_export.argtypes = [vp, vp, sz, C.POINTER(sz)]
    L.ag_plan_margins.argtypes = [vp, vp, sz]
    L.ag_plan_tile_record.argtypes = [vp, vp, vp, sz]
    L.ag_plan_reset_record.argtypes = [vp]
    L.ag_plan_trace.argtypes = [vp, C.c_int]
    L.ag_plan_unit_times.argtypes = [vp, vp, vp, sz]
    L.ag_plan_set_grid.argtypes = [vp, C.c_int]
    L.ag_plan_adopted.argtypes = [vp, C.POINTER(C.c_uint32)]
    L.ag_last_status.argtypes = [vp]
    L.ag_suggest_k_splits.argtypes = [i32, i32, i32, i32]
    L.ag_suggest_k_splits.restype = i32
    L.ag_last_status_where.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.ag_plan_destroy.argtypes = [vp]
    L.ag_plan_destroy.restype = None
    L.gemm_persistent.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp]
    L.ag_pack_weights.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, sz, C.POINTER(vp)]
    L.ag_pack_weights_ex.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp, vp, sz, C.c_uint32, C.POINTER(vp)]
    L.ag_packed_info.argtypes = [vp, C.POINTER(C.c_int32)]
    L.ag_packed_closed_form.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_uint32), C.POINTER(sz), C.POINTER(sz)]
    L.ag_packed_page_table.argtypes = [vp, vp, sz, C.POINTER(sz)]
    L.ag_packed_destroy.argtypes = [vp]
    L.ag_packed_destroy.restype = None
    L.gemm_persistent_packed.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp]
    L.gemm_persistent_noalloc.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp]
    L.ag_wait_probe.argtypes = [C.c_uint64, C.POINTER(C.c_uint64)]
    L.ag_kv_pack.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp, sz, C.c_int, C.POINTER(vp)]
    L.ag_kv_info.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_double)]
    L.ag_kv_append.argtypes = [vp, vp, vp, vp, vp]
    L.ag_kv_destroy.argtypes = [vp]
    L.ag_kv_destroy.restype = None
    L.attention_decode_persistent.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, vp, vp]
    L.ag_cluster_capacity.argtypes = [vp, C.POINTER(TopoMap), C.c_int, C.POINTER(C.c_int32)]
    L.ag_probe_cluster_layout.argtypes = [C.c_int, C.c_int, vp]
    L.ag_topo_save.argtypes = [C.POINTER(TopoMap), C.c_char_p]
    L.ag_topo_load.argtypes = [C.c_char_p, C.POINTER(TopoMap)]
    L.ag_group_desc_create.argtypes = [vp, vp, vp, C.c_int, vp, C.c_int, C.c_int, C.c_int, C.POINTER(vp)]
    L.ag_group_desc_destroy.argtypes = [vp]
    L.ag_group_desc_destroy.restype = None
    L.ag_pack_weights_grouped.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp, vp, sz, C.POINTER(vp)]
    L.gemm_persistent_grouped.argtypes = [vp, vp, vp, vp]
    L.ag_strerror.argtypes = [C.c_int]
    L.ag_strerror.restype = C.c_char_p
    L.ag_last_cuda_error.restype = C.c_int
    L.ag_kernel_launch_count.restype = C.c_uint64
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().ag_strerror(status).decode()


def _check(status: int, what: str):
    if status != AG_OK:
        raise AgError(status, what)


def kernel_launch_count() -> int:
    return int(lib().ag_kernel_launch_count())


# ---- topology -----------------------------------------------------------------------------
def topo_discover(phases: int | None = None) -> TopoMap:
    m = TopoMap()
    if phases is None:
        _check(lib().topo_discover(C.byref(m)), "topo_discover")
    else:
        _check(lib().ag_topo_discover_phases(C.byref(m), phases), "ag_topo_discover_phases")
    return m


def topo_from_observations(n_sm: int, clusters: list[list[int]], lat: np.ndarray | None) -> TopoMap:
    flat = np.array([s for c in clusters for s in c], dtype=np.int32)
    off = np.zeros(len(clusters) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(c) for c in clusters])
    m = TopoMap()
    if lat is not None:
        lat = np.ascontiguousarray(lat, dtype=np.uint32)
        n_ref, lp = lat.shape[1], lat.ctypes.data
    else:
        n_ref, lp = 0, None
    _check(lib().ag_topo_from_observations(n_sm, flat.ctypes.data if len(flat) else None, off.ctypes.data,
                                           len(clusters), lp, n_ref, C.byref(m)), "ag_topo_from_observations")
    return m


def topo_save(topo: TopoMap, path: str):
    _check(lib().ag_topo_save(C.byref(topo), path.encode()), "ag_topo_save")


def topo_load(path: str) -> TopoMap:
    m = TopoMap()
    _check(lib().ag_topo_load(path.encode(), C.byref(m)), "ag_topo_load")
    return m


def wait_probe(limit_ns: int):
    """Returns (status, waited_ns) of a device-side wait that is designed to run out."""
    w = C.c_uint64()
    st = lib().ag_wait_probe(limit_ns, C.byref(w))
    return int(st), int(w.value)


def topo_place_by_gain(gains, solo_bw: float) -> int:
    arr = (C.c_double * len(gains))(*gains)
    return int(lib().ag_topo_place_by_gain(arr, len(gains), solo_bw))


def probe_latency_samples(sm: int, mode: int = 0, n_lines: int = 256, reps: int = 8) -> np.ndarray:
    """n_lines x reps raw latency samples (SM cycles) taken from SM `sm`."""
    out = np.zeros((n_lines, reps), dtype=np.uint32)
    _check(lib().ag_probe_latency_samples(sm, mode, n_lines, reps, out.ctypes.data), "ag_probe_latency_samples")
    return out


def probe_l2_bandwidth(sms) -> float:
    """Aggregate L2 read bandwidth in bytes/s of the given SM ids."""
    mask = (C.c_uint64 * 4)()
    for s in sms:
        mask[s >> 6] |= 1 << (s & 63)
    out = C.c_double()
    _check(lib().ag_probe_l2_bandwidth(mask, C.byref(out)), "ag_probe_l2_bandwidth")
    return out.value


# ---- affinity ---------------------------------------------------------------------------------
class AffinityMap:
    def __init__(self, handle):
        self.handle = handle

    def export(self) -> np.ndarray:
        n = C.c_size_t()
        _check(lib().ag_affinity_export(self.handle, None, 0, C.byref(n)), "ag_affinity_export")
        out = np.empty(n.value, dtype=np.uint8)
        _check(lib().ag_affinity_export(self.handle, out.ctypes.data, out.size, C.byref(n)), "ag_affinity_export")
        return out

    def cycles(self) -> np.ndarray:
        out = np.empty((2, len(self.export())), dtype=np.uint32)
        _check(lib().ag_affinity_cycles(self.handle, out.ctypes.data, out.size), "ag_affinity_cycles")
        return out

    def check_complement(self, topo: TopoMap) -> int:
        n = C.c_size_t()
        _check(lib().ag_affinity_check_complement(self.handle, C.byref(topo), C.byref(n)), "ag_affinity_check_complement")
        return int(n.value)

    def die_bandwidth(self, topo: TopoMap, reader_die: int, chunk_die: int) -> float:
        """Bytes/s at which the SMs of reader_die stream the chunks of chunk_die."""
        out = C.c_double()
        _check(lib().ag_probe_die_bandwidth(self.handle, C.byref(topo), reader_die, chunk_die, C.byref(out)),
               "ag_probe_die_bandwidth")
        return out.value

    def fit_hash(self):
        """(mask over the 9 in-page chunk-index bits, number of chunks the fitted parity hash gets wrong)."""
        m, v = C.c_uint32(), C.c_size_t()
        _check(lib().ag_affinity_fit_hash(self.handle, C.byref(m), C.byref(v)), "ag_affinity_fit_hash")
        return int(m.value), int(v.value)

    def destroy(self):
        if self.handle:
            lib().ag_affinity_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def probe_ring_bandwidth(dev_ptr: int, nbytes: int, n_blocks: int, stages: int, stage_bytes: int = 32768,
                         producers: int = 3, hold_ns: int = 0) -> float:
    """Bytes/s that n_blocks blocks read through rings of `stages` bulk-copy stages of `stage_bytes`."""
    out = C.c_double()
    _check(lib().ag_probe_ring_bandwidth(dev_ptr, nbytes, n_blocks, stages, stage_bytes, producers, hold_ns, C.byref(out)),
           "ag_probe_ring_bandwidth")
    return out.value


def aligned_device_bytes(nbytes: int):
    """A zeroed uint8 torch tensor of nbytes on the current CUDA device that starts on a 4096-byte boundary, as buffers that
    are probed or packed into must (a block handed out by torch's caching allocator may start off one)."""
    import torch
    raw = torch.zeros(nbytes + AG_CHUNK_BYTES, dtype=torch.uint8, device="cuda")
    return raw[(-raw.data_ptr()) % AG_CHUNK_BYTES:][:nbytes]


def affinity_probe(dev_ptr: int, nbytes: int, topo: TopoMap | None = None) -> AffinityMap:
    h = C.c_void_p()
    if topo is None:
        _check(lib().affinity_probe(dev_ptr, nbytes, C.byref(h)), "affinity_probe")
    else:
        _check(lib().ag_affinity_probe_with_map(dev_ptr, nbytes, C.byref(topo), C.byref(h)), "ag_affinity_probe_with_map")
    return AffinityMap(h)


def affinity_from_table(dev_ptr: int, die_of_chunk: np.ndarray) -> AffinityMap:
    t = np.ascontiguousarray(die_of_chunk, dtype=np.uint8)
    h = C.c_void_p()
    _check(lib().ag_affinity_from_table(dev_ptr, t.size * AG_CHUNK_BYTES, t.ctypes.data, t.size, C.byref(h)),
           "ag_affinity_from_table")
    return AffinityMap(h)


# ---- plan -------------------------------------------------------------------------------------
def make_policy(kind=AG_OBLIVIOUS, M=0, N=0, K=0, tile_m=128, tile_n=256, k_splits=1, k_unit=64, raster_group=1,
                preferred_die=-1, invert_affinity=0, static_assign=1, seed=0, min_margin=0, splitk_in_memory=0,
                sm_select=0, pair_lists=None, overlap_launches=0, cluster_size=1, die_quota=0, decode_shaped=0, ring_stages=0, avoid=(), a=None, b=None, c=None):
    """a/b/c: None or dict(offset, row_stride, elem_bytes[, layout, page_table]).  pair_lists=None means
    "on for plans of block pairs (tile_m == 256)"."""
    p = Policy()
    p.kind, p.M, p.N, p.K, p.tile_m, p.tile_n = kind, M, N, K, tile_m, tile_n
    p.k_splits, p.k_unit, p.raster_group = k_splits, k_unit, raster_group
    p.preferred_die, p.invert_affinity, p.static_assign, p.seed = preferred_die, invert_affinity, static_assign, seed
    p.min_margin = min_margin
    p.splitk_in_memory = splitk_in_memory
    p.sm_select = sm_select
    p.pair_lists = (1 if tile_m == 256 else 0) if pair_lists is None else pair_lists
    p.overlap_launches = overlap_launches
    p.cluster_size = cluster_size
    p.die_quota = die_quota
    p.decode_shaped = decode_shaped
    p.ring_stages = ring_stages
    for s in avoid:
        p.avoid_sm_mask[s >> 6] |= 1 << (s & 63)
    keep = []
    for name, op in (("a", a), ("b", b), ("c", c)):
        d = getattr(p, name)
        if op is None:
            d.present = 0
            continue
        d.present = 1
        d.layout = op.get("layout", AG_LAYOUT_ROWMAJOR)
        d.offset, d.row_stride, d.elem_bytes = op["offset"], op["row_stride"], op["elem_bytes"]
        if op.get("page_table") is not None:
            t = np.ascontiguousarray(op["page_table"], dtype=np.int32)
            keep.append(t)
            d.page_table = t.ctypes.data_as(C.POINTER(C.c_int32))
            d.n_pages = t.size
    p._keepalive = keep
    return p


class Plan:
    def __init__(self, handle):
        self.handle = handle

    def export(self) -> np.ndarray:
        n = C.c_size_t()
        _check(lib().ag_plan_export(self.handle, None, 0, C.byref(n)), "ag_plan_export")
        out = np.empty(n.value, dtype=np.int32)
        _check(lib().ag_plan_export(self.handle, out.ctypes.data, out.size, C.byref(n)), "ag_plan_export")
        return out

    def parsed(self) -> dict:
        w = self.export()
        b, n_u, n_sm = int(w[3]), int(w[5]), int(w[2])
        o = 16
        d = dict(kind=int(w[1]), n_sm=n_sm, b=b, n_units=n_u, tiles_m=int(w[6]), tiles_n=int(w[7]))
        for name, ln in (("sm_list", b), ("sm_die", b), ("rank_in_die", b), ("die_sm_count", 2), ("die_q_off", 3),
                         ("die_q", n_u), ("sm_q_off", b + 1), ("sm_q", n_u), ("smid_to_slot", n_sm)):
            d[name] = w[o:o + ln].copy()
            o += ln
        return d

    def margins(self) -> np.ndarray:
        n_u = int(self.export()[5])
        out = np.empty(n_u, dtype=np.int64)
        _check(lib().ag_plan_margins(self.handle, out.ctypes.data, out.size), "ag_plan_margins")
        return out

    def tile_record(self):
        n_u = int(self.export()[5])
        owner = np.empty(n_u, dtype=np.int32)
        count = np.empty(n_u, dtype=np.int32)
        _check(lib().ag_plan_tile_record(self.handle, owner.ctypes.data, count.ctypes.data, n_u), "ag_plan_tile_record")
        return owner, count

    def reset_record(self):
        _check(lib().ag_plan_reset_record(self.handle), "ag_plan_reset_record")

    def cluster_capacity(self, topo, cluster_size: int) -> int:
        n = C.c_int32()
        _check(lib().ag_cluster_capacity(self.handle, C.byref(topo), cluster_size, C.byref(n)), "ag_cluster_capacity")
        return int(n.value)

    def trace(self, on: bool = True):
        _check(lib().ag_plan_trace(self.handle, 1 if on else 0), "ag_plan_trace")

    def unit_times(self):
        """(start_ns, end_ns) per unit of the last launch (tracing must be on)."""
        n_u = int(self.export()[5])
        t0 = np.zeros(n_u, dtype=np.uint64)
        t1 = np.zeros(n_u, dtype=np.uint64)
        _check(lib().ag_plan_unit_times(self.handle, t0.ctypes.data, t1.ctypes.data, n_u), "ag_plan_unit_times")
        return t0, t1

    def set_grid(self, blocks: int):
        _check(lib().ag_plan_set_grid(self.handle, blocks), "ag_plan_set_grid")

    def adopted(self) -> int:
        n = C.c_uint32()
        _check(lib().ag_plan_adopted(self.handle, C.byref(n)), "ag_plan_adopted")
        return int(n.value)

    def last_status(self) -> int:
        return int(lib().ag_last_status(self.handle))

    def last_status_where(self) -> tuple:
        """(role, smid) of the first bounded wait that ran out; (0, -1) when none did."""
        r, s_ = C.c_int32(), C.c_int32()
        _check(lib().ag_last_status_where(self.handle, C.byref(r), C.byref(s_)), "ag_last_status_where")
        return int(r.value), int(s_.value)

    def destroy(self):
        if self.handle:
            lib().ag_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def sched_build(topo: TopoMap, amap: AffinityMap | None, sm_budget: int, policy: Policy) -> Plan:
    h = C.c_void_p()
    _check(lib().sched_build(C.byref(topo), amap.handle if amap is not None else None, sm_budget,
                             C.byref(policy), C.byref(h)), "sched_build")
    return Plan(h)


def gemm_persistent(a_ptr: int, b_ptr: int, c_ptr: int, M: int, N: int, K: int, plan: Plan, stream: int = 0):
    """Raw device pointers in, asynchronous on `stream` (a cudaStream_t value, 0 = default)."""
    _check(lib().gemm_persistent(a_ptr, b_ptr, c_ptr, M, N, K, plan.handle, stream), "gemm_persistent")


class PackedWeights:
    def __init__(self, handle):
        self.handle = handle

    def group_free_bit(self) -> int:
        """>= 2: pages are stored in groups of four same-die chunks (one copy per k-slab); -1: single pages."""
        f = C.c_int32()
        _check(lib().ag_packed_info(self.handle, C.byref(f)), "ag_packed_info")
        return int(f.value)

    def closed_form(self) -> dict:
        """Whether the kernels compute page addresses from the fitted hash (Eq. 1 in closed form) or read tables."""
        en, mask, tb, cb = C.c_int32(), C.c_uint32(), C.c_size_t(), C.c_size_t()
        _check(lib().ag_packed_closed_form(self.handle, C.byref(en), C.byref(mask), C.byref(tb), C.byref(cb)), "ag_packed_closed_form")
        return dict(enabled=bool(en.value), mask=int(mask.value), table_bytes=int(tb.value), closed_bytes=int(cb.value))

    def page_table(self) -> np.ndarray:
        n = C.c_size_t()
        _check(lib().ag_packed_page_table(self.handle, None, 0, C.byref(n)), "ag_packed_page_table")
        out = np.empty(n.value, dtype=np.int32)
        _check(lib().ag_packed_page_table(self.handle, out.ctypes.data, out.size, C.byref(n)), "ag_packed_page_table")
        return out

    def destroy(self):
        if self.handle:
            lib().ag_packed_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def pack_weights(b_ptr: int, K: int, N: int, plan: Plan, amap: AffinityMap, dst_ptr: int, dst_bytes: int,
                 single_pages: bool = False, tables_only: bool = False, consecutive: bool = False) -> PackedWeights:
    h = C.c_void_p()
    bl = (C.c_void_p * 1)(b_ptr)
    _check(lib().ag_pack_weights_ex(bl, 1, K, N, plan.handle, amap.handle, dst_ptr, dst_bytes,
                                    (1 if single_pages else 0) | (2 if tables_only else 0) | (4 if consecutive else 0), C.byref(h)),
           "ag_pack_weights_ex")
    return PackedWeights(h)


def gemm_persistent_packed(a_ptr: int, packed: PackedWeights, c_ptr: int, M: int, N: int, K: int, plan: Plan,
                           stream: int = 0):
    _check(lib().gemm_persistent_packed(a_ptr, packed.handle, c_ptr, M, N, K, plan.handle, stream),
           "gemm_persistent_packed")


def gemm_persistent_noalloc(a_ptr: int, b_ptr: int, c_ptr: int, M: int, N: int, K: int, plan: Plan, stream: int = 0):
    """Decode-shaped GEMM (M <= 32) that takes its split-K workspace from the library's built-in
    device array instead of allocated memory; for callers that may not allocate.  Calls on one GPU
    must not overlap.  Limits: k_splits * M * N * 4 <= 8 MiB, N <= 131072."""
    _check(lib().gemm_persistent_noalloc(a_ptr, b_ptr, c_ptr, M, N, K, plan.handle, stream), "gemm_persistent_noalloc")


KV_LOCAL, KV_REMOTE, KV_INTERLEAVED = 0, 1, 2


class KVCache:
    def __init__(self, handle):
        self.handle = handle

    def info(self) -> dict:
        f, frac = C.c_int32(), C.c_double()
        _check(lib().ag_kv_info(self.handle, C.byref(f), C.byref(frac)), "ag_kv_info")
        return dict(group_free_bit=int(f.value), local_fraction=float(frac.value))

    def append(self, k_new_ptr: int, v_new_ptr: int, pos_ptr: int, stream: int = 0):
        """One new token per request at position pos[b] (device int32 [B]); k_new, v_new: [B][H_kv][128] bf16."""
        _check(lib().ag_kv_append(self.handle, k_new_ptr, v_new_ptr, pos_ptr, stream), "ag_kv_append")

    def destroy(self):
        if getattr(self, "handle", None):
            lib().ag_kv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def kv_pack(k_ptr: int, v_ptr: int, B: int, H_kv: int, L: int, plan: Plan, amap: AffinityMap, dst_ptr: int, dst_bytes: int,
            placement: int = KV_LOCAL, D: int = 128) -> KVCache:
    h = C.c_void_p()
    _check(lib().ag_kv_pack(k_ptr, v_ptr, B, H_kv, L, D, plan.handle, amap.handle, dst_ptr, dst_bytes, placement, C.byref(h)),
           "ag_kv_pack")
    return KVCache(h)


def attention_decode(q_ptr: int, kv: KVCache, kv_len_ptr, o_ptr: int, B: int, H_q: int, plan: Plan, stream: int = 0):
    _check(lib().attention_decode_persistent(q_ptr, kv.handle, kv_len_ptr, o_ptr, B, H_q, plan.handle, stream),
           "attention_decode_persistent")


def suggest_k_splits(N: int, K: int, sm_budget: int, overlapping_full_chip: bool = False) -> int:
    return int(lib().ag_suggest_k_splits(N, K, sm_budget, 1 if overlapping_full_chip else 0))


def probe_cluster_layout(cluster_size: int, n_clusters: int) -> np.ndarray:
    """Cluster id that the hardware ran first on every SM (-1: none) for a launch of n_clusters clusters."""
    out = np.full(AG_MAX_SM, -1, dtype=np.int32)
    _check(lib().ag_probe_cluster_layout(cluster_size, n_clusters, out.ctypes.data), "ag_probe_cluster_layout")
    return out


class GroupDesc:
    """Stacked activations / outputs and per-expert weights of a grouped decode GEMM."""

    def __init__(self, a_ptr: int, c_ptr: int, rows, b_ptrs, n_expert: int, K: int, tile_m: int):
        r = np.ascontiguousarray(rows, dtype=np.int32)
        bl = (C.c_void_p * len(b_ptrs))(*b_ptrs) if b_ptrs is not None else None
        h = C.c_void_p()
        _check(lib().ag_group_desc_create(a_ptr, c_ptr, r.ctypes.data, r.size, bl, n_expert, K, tile_m, C.byref(h)),
               "ag_group_desc_create")
        self.handle = h

    def destroy(self):
        if self.handle:
            lib().ag_group_desc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def pack_weights_grouped(b_ptrs, K: int, n_expert: int, plan: Plan, amap: AffinityMap, dst_ptr: int,
                         dst_bytes: int, single_pages: bool = False, consecutive: bool = False) -> PackedWeights:
    bl = (C.c_void_p * len(b_ptrs))(*b_ptrs)
    h = C.c_void_p()
    _check(lib().ag_pack_weights_ex(bl, len(b_ptrs), K, n_expert, plan.handle, amap.handle, dst_ptr, dst_bytes,
                                    (1 if single_pages else 0) | (4 if consecutive else 0), C.byref(h)), "ag_pack_weights_ex")
    return PackedWeights(h)


def gemm_persistent_grouped(desc: GroupDesc, packed, plan: Plan, stream: int = 0):
    _check(lib().gemm_persistent_grouped(desc.handle, packed.handle if packed is not None else None, plan.handle, stream),
           "gemm_persistent_grouped")

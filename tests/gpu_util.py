"""Helpers for the GPU parity tests: torch is used only for device memory and streams."""
import numpy as np
import torch

from oracle import plan as op
from paper_2609_24270_b200 import binding as ag

_TOPO = None


def device_topo():
    """Census + latency phases only (fast); cached for the test session."""
    global _TOPO
    if _TOPO is None:
        _TOPO = ag.topo_discover(ag.AG_TOPO_CENSUS | ag.AG_TOPO_CLUSTER | ag.AG_TOPO_LATENCY)
    return _TOPO


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda()


def run_gemm(A_bits, B_bits, plan, stream=None):
    M, K = A_bits.shape
    N = B_bits.shape[1]
    dA, dB = to_dev_bf16(A_bits), to_dev_bf16(B_bits)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    s = 0 if stream is None else stream.cuda_stream
    ag.gemm_persistent(dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), M, N, K, plan, s)
    torch.cuda.synchronize()
    st = plan.last_status()
    assert st == ag.AG_OK, ag.strerror(st)
    return dC.cpu().numpy()


def check_close(C_gpu, C_ref):
    """Tolerance fixed by the benchmark spec: relative Frobenius error <= 1e-4, max abs error <= 1e-2."""
    assert np.isfinite(C_gpu).all()
    diff = C_gpu.astype(np.float64) - C_ref
    rel = np.linalg.norm(diff) / max(np.linalg.norm(C_ref), 1e-30)
    mx = np.abs(diff).max()
    assert rel <= 1e-4 and mx <= 1e-2, (rel, mx)
    return rel, mx


def oracle_policy(**kw):
    """Oracle-side policy dict from the same keyword arguments as ag.make_policy."""
    d = dict(kw)
    if d.get("pair_lists") is None:                      # same default as ag.make_policy
        d["pair_lists"] = 1 if d.get("tile_m", 128) == 256 else 0
    for name in ("a", "b", "c"):
        o = d.get(name)
        if o is not None:
            d[name] = op.operand(o["offset"], o["row_stride"], o["elem_bytes"],
                                 o.get("layout", op.LAYOUT_ROWMAJOR), o.get("page_table"))
    return op.default_policy(**d)

"""Hand-off timeline of the backward main kernel (development aid).

``python -m paper_2606_10415_b200.timeline [config] [first] [last]`` builds ``liblt_attn_timeline.so`` (the
backward compiled with ``-DLT_BWD_TIMELINE=0``: CTA 0 stamps ``clock64`` at every hand-off of its first 256 tile
pairs), runs one backward call of the named workload through it and prints, for the tile pairs ``first..last-1``
of that CTA, the cycle at which each role passed each hand-off (relative to the first dP issue shown).  The product
library is not touched; the forward state comes from it.
"""
from __future__ import annotations

import ctypes
import sys

import torch

from . import binding as lt, build, workloads

EVENTS = [
    "issuer: dO landed", "issuer: dQ drained, dP issue begins", "issuer: dP issued", "issuer: P ready",
    "issuer: dV and next S issued", "issuer: dS ready", "issuer: dK and dQ issued",
    "softmax: S complete", "softmax: P handed over", "softmax: dP complete", "softmax: dS handed over",
    "reduce: dQ complete", "reduce: dP columns released", "reduce: last group issued",
    "issuer: first S of a work item issued", "reduce: dK/dV accumulators released",
]
N_EVENTS, N_ITER = 20, 256


def run(name: str = "llama2_7b", first: int = 8, last: int = 18) -> list[list[int]]:
    cfg = workloads.ALL_CONFIGS[name]
    lib = ctypes.CDLL(str(build.build_timeline_variant()))
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.lt_attn_bwd.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_bwd.restype = i
    lib.lt_dbg_bwd_timeline.argtypes = [vp]
    lib.lt_dbg_bwd_timeline.restype = i
    Q, K, V, dO = (t.cuda() for t in workloads.make_inputs(cfg))
    O = torch.empty_like(Q)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D)
    lt.lt_attn_fwd(Q, K, V, O, LSE, cfg.causal, cfg.scale, lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(*dims)))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(*dims))
    ptr = lambda t: ctypes.c_void_p(t.data_ptr())
    for call in range(4):  # warm-up calls, then the stamps of the last call alone
        if call == 3:
            torch.cuda.synchronize()
            lib.lt_dbg_bwd_timeline(None)
        rc = lib.lt_attn_bwd(ptr(Q), ptr(K), ptr(V), ptr(O), ptr(dO), ptr(LSE), ptr(dQ), ptr(dK), ptr(dV), *dims,
                             int(cfg.causal), cfg.scale, ptr(ws), ws.numel() * ws.element_size(), None)
        if rc != 0:
            raise RuntimeError(f"lt_attn_bwd (timeline build) returned {rc}")
    torch.cuda.synchronize()
    buf = (ctypes.c_longlong * (N_EVENTS * N_ITER))()
    if lib.lt_dbg_bwd_timeline(buf) != 0:
        raise RuntimeError("lt_dbg_bwd_timeline failed")
    t = [list(buf[e * N_ITER:(e + 1) * N_ITER]) for e in range(N_EVENTS)]
    base = t[1][first]
    print(f"{name}: CTA 0, tile pairs {first}..{last - 1}; cycles relative to the first dP issue shown")
    print(f"{'':44s}" + " ".join(f"{n:7d}" for n in range(first, last)))
    for e, label in enumerate(EVENTS):
        cells = [f"{t[e][n] - base:7d}" if t[e][n] > 0 else "      ." for n in range(first, last)]
        print(f"{label:44s}" + " ".join(cells))
    print("period (dP issue to dP issue):", [t[1][n + 1] - t[1][n] for n in range(first, last - 1)])
    return t


if __name__ == "__main__":
    a = sys.argv[1:]
    run(a[0] if a else "llama2_7b", int(a[1]) if len(a) > 1 else 8, int(a[2]) if len(a) > 2 else 18)

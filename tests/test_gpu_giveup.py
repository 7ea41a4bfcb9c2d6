"""The main backward kernel's own give-up path, exercised without hanging or faulting the GPU.

A test build of the backward (``build.build_giveup_variant``: one tensor-core hand-off is dropped on
purpose and every device-side wait gives up after about 10 ms) is loaded beside the product library.
Its main kernel cannot finish its second tile pair, so the waits downstream of the dropped hand-off run
out: one thread raises the shared abort flag and records the wait's code, every role leaves its loops,
copies in flight are given time to land, tensor memory is released and the kernel returns normally.
The host then reads LT_ERR_DEVICE_TIMEOUT, and the product library still runs in the same context."""
import ctypes

import pytest
import torch

from paper_2606_10415_b200 import workloads
from parity_checks import check_grads

pytestmark = pytest.mark.gpu

# Codes of the main kernel's waits (lt_attn_bwd.cu).  The dropped hand-off starves every role; which of the
# starved waits began first, and so runs out first and gets recorded, depends on timing.
MAIN_KERNEL_WAIT_CODES = set(range(200, 215))


def test_main_kernel_gives_up_cleanly_and_the_context_survives(oracle):
    from paper_2606_10415_b200 import binding as lt, build
    lib = ctypes.CDLL(str(build.build_giveup_variant()))
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.lt_attn_bwd.argtypes = [vp] * 9 + [i] * 6 + [f, vp, sz, vp]
    lib.lt_attn_bwd.restype = i
    lib.lt_attn_check_status.argtypes = [vp, vp]
    lib.lt_attn_check_status.restype = i
    lib.lt_last_cuda_error.restype = ctypes.c_char_p

    cfg = workloads.custom(1, 2, 1, 384, 128, True, seed=5)  # three key tiles, up to six tile pairs per work item
    Q, K, V, dO = (t.cuda() for t in workloads.make_inputs(cfg))
    O = torch.empty_like(Q)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D)
    fws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(*dims))
    lt.lt_attn_fwd(Q, K, V, O, LSE, cfg.causal, cfg.scale, fws)
    assert lt.lt_attn_check_status(fws) == lt.LT_OK
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(*dims))
    stream = torch.cuda.current_stream().cuda_stream
    ptrs = [t.data_ptr() for t in (Q, K, V, O, dO, LSE, dQ, dK, dV)]

    rc = lib.lt_attn_bwd(*ptrs, *dims, 1, cfg.scale, ws.data_ptr(), ws.numel(), stream)
    assert rc == lt.LT_OK  # the launch itself succeeds; the failure is the device's to report
    assert lib.lt_attn_check_status(ws.data_ptr(), stream) == lt.LT_ERR_DEVICE_TIMEOUT
    message = lib.lt_last_cuda_error().decode()  # "device timeout: wait code NNN"
    assert int(message.rsplit(" ", 1)[1]) in MAIN_KERNEL_WAIT_CODES, message

    # the kernel returned (no hang, no fault): the context is usable and the product library is correct
    lt.lt_attn_bwd(Q, K, V, O, dO, LSE, dQ, dK, dV, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    ref = oracle.attn_bwd(*(t.cpu().double().numpy() for t in (Q, K, V, dO)), cfg.causal, cfg.scale)
    check_grads((dQ, dK, dV), ref, "after a give-up")

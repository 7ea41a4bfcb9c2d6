"""Host-side checks of the C ABI: the library loads, exports what the header declares,
and rejects bad arguments before touching the GPU.  No kernel is launched here."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def binding():
    from paper_2606_10415_b200 import build
    build.build()
    from paper_2606_10415_b200 import binding as b
    return b


def declared_functions(header="lt_attn.h"):
    text = (ROOT / "include" / header).read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lt_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_documented_entry_points():
    names = declared_functions()
    for must in ("lt_attn_fwd", "lt_attn_bwd", "lt_attn_bwd_workspace_bytes", "lt_attn_check_status",
                 "lt_status_string", "lt_attn_fwd_bwd_host"):
        assert must in names


def test_library_exports_every_declared_symbol(binding):
    lib = ctypes.CDLL(str(binding.LIB_PATH))
    for name in declared_functions() + declared_functions("lt_attn_debug.h"):
        assert hasattr(lib, name), name
    assert set(declared_functions()) == set(binding.EXPORTS)
    # the test-support entry points live in a header of their own, outside the product interface
    assert set(declared_functions("lt_attn_debug.h")) == set(binding.DEBUG_EXPORTS)
    assert not any(n.startswith("lt_dbg") for n in declared_functions())


def test_workspace_sizes(binding):
    # 256-byte status block + two [B,Hq,S] arrays of 16-byte rows + dQ accumulator fp32 [B,Hq,S,D]
    assert binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 128, 64) == 256 + 2 * 4096 + 65536
    assert binding.lt_attn_bwd_workspace_bytes(1, 32, 32, 4096, 128) == 256 + 2 * 2097152 + 67108864
    assert binding.lt_attn_fwd_workspace_bytes(1, 2, 2, 128, 64) == 256
    # unsupported shapes report 0
    assert binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 0, 64) == 0
    # a ragged length is padded to whole 128-row tiles inside the workspace
    assert binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 100, 64) == binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 128, 64)
    assert binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 129, 64) == binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 256, 64)
    assert binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 128, 96) == 0
    assert binding.lt_attn_bwd_workspace_bytes(1, 3, 2, 128, 64) == 0
    assert binding.lt_attn_host_arena_bytes(1, 2, 2, 128, 64) > binding.lt_attn_bwd_workspace_bytes(1, 2, 2, 128, 64)


def test_launch_counts(binding):
    # three kernels per backward call; four on grouped-query shapes with few, heavy work items
    assert binding.lt_attn_bwd_num_launches(1, 32, 32, 4096, 128, True) == 3
    assert binding.lt_attn_bwd_num_launches(1, 40, 8, 4096, 128, True) == 3
    assert binding.lt_attn_bwd_num_launches(1, 40, 8, 2048, 128, True) == 4
    # groups are also split when whole-group items are too few for L2-sized batches on a working set of several L2s
    assert binding.lt_attn_bwd_num_launches(2, 64, 8, 4096, 128, True) == 4
    assert binding.lt_attn_bwd_num_launches(4, 64, 8, 4096, 128, True) == 3
    assert binding.lt_attn_bwd_num_launches(1, 2, 2, 128, 96, True) == 0
    assert binding.lt_attn_fwd_num_launches() == 1


def test_status_strings(binding):
    seen = {binding.status_string(s) for s in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def _bwd_args(ptr=0x1000, B=1, Hq=2, Hkv=2, S=128, D=64, scale=0.125, ws=0x10000, ws_bytes=1 << 20):
    return [ptr] * 9 + [B, Hq, Hkv, S, D, 1, scale, ws, ws_bytes, 0]


def test_bwd_rejects_bad_arguments_without_launching(binding):
    b = binding
    args = _bwd_args()
    args[3] = 0
    assert b.lt_attn_bwd_raw(*args) == b.LT_ERR_INVALID_ARG               # NULL tensor
    assert b.lt_attn_bwd_raw(*_bwd_args(B=0)) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_bwd_raw(*_bwd_args(Hq=3, Hkv=2)) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_bwd_raw(*_bwd_args(scale=float("nan"))) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_bwd_raw(*_bwd_args(scale=0.0)) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_bwd_raw(*_bwd_args(S=100, ws_bytes=1 << 10)) == b.LT_ERR_WORKSPACE  # ragged S is a shape like any other
    assert b.lt_attn_bwd_raw(*_bwd_args(D=96)) == b.LT_ERR_UNSUPPORTED
    assert b.lt_attn_bwd_raw(*_bwd_args(ptr=0x1004)) == b.LT_ERR_UNSUPPORTED  # misaligned
    assert b.lt_attn_bwd_raw(*_bwd_args(ws=0)) == b.LT_ERR_WORKSPACE
    assert b.lt_attn_bwd_raw(*_bwd_args(ws=0x10010)) == b.LT_ERR_WORKSPACE    # not 256-byte aligned
    assert b.lt_attn_bwd_raw(*_bwd_args(ws_bytes=1000)) == b.LT_ERR_WORKSPACE


def test_fwd_rejects_bad_arguments_without_launching(binding):
    b = binding

    def args(ptr=0x1000, B=1, Hq=2, Hkv=2, S=128, D=64, scale=0.125, ws=0x10000, ws_bytes=256):
        return [ptr] * 5 + [B, Hq, Hkv, S, D, 1, scale, ws, ws_bytes, 0]

    a = args()
    a[4] = 0
    assert b.lt_attn_fwd_raw(*a) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_fwd_raw(*args(S=0)) == b.LT_ERR_INVALID_ARG
    assert b.lt_attn_fwd_raw(*args(D=256)) == b.LT_ERR_UNSUPPORTED
    assert b.lt_attn_fwd_raw(*args(ws_bytes=16)) == b.LT_ERR_WORKSPACE


def test_no_gpu_means_a_loud_error_not_a_fallback(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    # arguments are valid, so the call reaches the device check and must fail there
    rc = binding.lt_attn_bwd_raw(*_bwd_args())
    assert rc in (binding.LT_ERR_CUDA, binding.LT_ERR_UNSUPPORTED)


def test_strided_entry_points_reject_bad_strides(binding):
    """Layout checks happen on the host before anything is launched."""
    import ctypes
    b = binding
    lib = b._lib

    def layout(**over):
        lay = b.AttnLayout()
        for name in ("q", "k", "v", "o", "d_o", "dq", "dk", "dv"):
            setattr(lay, name, b.TensorStrides(2 * 128 * 64, 128 * 64, 64))
        for name, st in over.items():
            setattr(lay, name, b.TensorStrides(*st))
        return lay

    def bwd(lay, ws_bytes=1 << 20):
        return lib.lt_attn_bwd_strided(*([0x1000] * 9), ctypes.byref(lay), 1, 2, 2, 128, 64, 1, 0.125, 0x10000,
                                       ws_bytes, 0)

    def fwd(lay, ws_bytes=256):
        return lib.lt_attn_fwd_strided(*([0x1000] * 5), ctypes.byref(lay), 1, 2, 2, 128, 64, 1, 0.125, 0x10000,
                                       ws_bytes, 0)

    # a valid layout gets past the stride checks (and then fails for lack of a workspace / device)
    assert bwd(layout(), ws_bytes=16) == b.LT_ERR_WORKSPACE
    assert bwd(layout(dk=(2 * 128 * 64, 128 * 64, 60))) == b.LT_ERR_UNSUPPORTED      # row stride below D
    assert bwd(layout(q=(2 * 128 * 64, 128 * 64 + 4, 64))) == b.LT_ERR_UNSUPPORTED   # not a multiple of 8 elements
    assert bwd(layout(d_o=(0, 128 * 64, 64))) == b.LT_ERR_UNSUPPORTED                # zero stride
    assert fwd(layout(o=(2 * 128 * 64, 128 * 64, -64))) == b.LT_ERR_UNSUPPORTED
    # the forward ignores the gradient entries: it gets as far as the workspace check (nothing is launched)
    assert fwd(layout(dq=(1, 1, 1)), ws_bytes=16) == b.LT_ERR_WORKSPACE


def test_gemm_rejects_bad_arguments_without_launching(binding):
    b = binding
    lib = b._lib

    def call(A=0x1000, W=0x2000, C=0x3000, M=128, N=256, K=64, ws=0x10000, ws_bytes=256):
        return lib.lt_gemm_f16(A, W, C, M, N, K, ws, ws_bytes, 0)

    assert b.lt_gemm_f16_workspace_bytes() == 256
    assert call(A=0) == b.LT_ERR_INVALID_ARG
    assert call(M=0) == b.LT_ERR_INVALID_ARG
    assert call(K=-8) == b.LT_ERR_INVALID_ARG
    assert call(K=12) == b.LT_ERR_UNSUPPORTED        # row pitch of 24 bytes: no 16-byte tile loads
    assert call(W=0x2002) == b.LT_ERR_UNSUPPORTED    # misaligned
    assert call(ws=0) == b.LT_ERR_WORKSPACE
    assert call(ws_bytes=16) == b.LT_ERR_WORKSPACE


def test_saved_p_entry_points_reject_bad_arguments_without_launching(binding):
    b = binding
    lib = b._lib
    assert b.lt_attn_p_store_bytes(2, 4, 2, 300, 128) == 2 * 4 * 3 * 3 * 128 * 128 * 2  # ceil(300/128) = 3 tiles
    assert b.lt_attn_p_store_bytes(1, 1, 1, 128, 64) == 32768
    assert b.lt_attn_p_store_bytes(1, 3, 2, 128, 64) == 0      # heads do not divide
    assert b.lt_attn_p_store_bytes(1, 2, 2, 128, 96) == 0      # unsupported head dim

    def save(Q=0x1000, K=0x2000, LSE=0x3000, P=0x4000, S=128, D=128, scale=0.1, ws=0x10000, ws_bytes=256):
        return lib.lt_attn_save_p(Q, K, LSE, P, 1, 2, 2, S, D, 1, scale, ws, ws_bytes, 0)

    assert save(P=0) == b.LT_ERR_INVALID_ARG
    assert save(S=0) == b.LT_ERR_INVALID_ARG
    assert save(scale=0.0) == b.LT_ERR_INVALID_ARG
    assert save(D=96) == b.LT_ERR_UNSUPPORTED
    assert save(P=0x4010) == b.LT_ERR_UNSUPPORTED     # the store must be 256-byte aligned
    assert save(LSE=0x3002) == b.LT_ERR_UNSUPPORTED
    assert save(ws_bytes=16) == b.LT_ERR_WORKSPACE

    def bwd(P=0x4000, ptr=0x1000, S=128, ws=0x10000, ws_bytes=16):
        return lib.lt_attn_bwd_saved_p(ptr, ptr, ptr, ptr, ptr, P, ptr, ptr, ptr, 1, 2, 2, S, 128, 1, 0.1, ws, ws_bytes, 0)

    assert bwd(P=0) == b.LT_ERR_INVALID_ARG
    assert bwd(S=-1) == b.LT_ERR_INVALID_ARG
    assert bwd(P=0x4020) == b.LT_ERR_UNSUPPORTED
    assert bwd(ptr=0x1004) == b.LT_ERR_UNSUPPORTED
    assert bwd() == b.LT_ERR_WORKSPACE                # 16 bytes of workspace: stops before any launch

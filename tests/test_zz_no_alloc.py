"""The allocation-free backward entry point against the ordinary one and against the CPU oracle.

Some users of the library cannot allocate device memory where they call the backward (a
fixed memory pool, a plugin without an allocator, an allocation-free steady state), so
``lt_attn_bwd_noalloc`` takes its scratch from an array built into the library.  This file is
collected last on purpose: if it fails, a run that stops at the first failure has already
run everything else.  It passes on its own in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2606_10415_b200 import workloads
from parity_checks import check_grads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lt():
    from paper_2606_10415_b200 import binding
    return binding


def _rel_fro(a, b):
    a, b = a.double().numpy(), b.double().numpy()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def _inputs(lt, cfg):
    Q, K, V, dO = (t.cuda() for t in workloads.make_inputs(cfg))
    O = torch.empty_like(Q)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    fws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd(Q, K, V, O, LSE, cfg.causal, cfg.scale, fws)
    assert lt.lt_attn_check_status(fws) == lt.LT_OK
    return Q, K, V, O, dO, LSE


def test_noalloc_matches_workspace_entry_point_twice_in_a_row(lt, oracle):
    # two different shapes back to back: the second call finds the first call's leftovers in the scratch
    for cfg in (workloads.custom(1, 4, 2, 512, 128, True, seed=21), workloads.custom(2, 2, 2, 256, 64, True, seed=22)):
        Q, K, V, O, dO, LSE = _inputs(lt, cfg)
        ref = [torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)]
        ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
        lt.lt_attn_bwd(Q, K, V, O, dO, LSE, *ref, cfg.causal, cfg.scale, ws)
        assert lt.lt_attn_check_status(ws) == lt.LT_OK
        for _ in range(2):
            got = [torch.full_like(t, float("nan")) for t in ref]
            lt.lt_attn_bwd_noalloc(Q, K, V, O, dO, LSE, *got, cfg.causal, cfg.scale)
            # the status word of the built-in scratch: no wait gave up (this call synchronises the stream)
            assert lt.lt_attn_bwd_noalloc_check_status() == lt.LT_OK, lt.last_cuda_error()
            # dK and dV have a fixed summation order; dQ is reduced with atomics
            assert torch.equal(got[1].cpu(), ref[1].cpu())
            assert torch.equal(got[2].cpu(), ref[2].cpu())
            assert torch.isfinite(got[0].float()).all()
            assert _rel_fro(got[0].cpu(), ref[0].cpu()) < 1e-3
        # and the entry point's own output against the fp64 oracle, to the gates of the parity tests
        exact = oracle.attn_bwd(*(t.cpu().double().numpy() for t in (Q, K, V, dO)), cfg.causal, cfg.scale)
        check_grads(got, exact, f"noalloc {cfg}")


def test_noalloc_rejects_shapes_beyond_its_scratch(lt):
    cfg = workloads.CONFIGS["llama2_7b"]
    assert lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D) > lt.NOALLOC_MAX_SCRATCH_BYTES
    # arguments are only inspected, never dereferenced, before the size check fails
    Q = torch.empty((cfg.B, cfg.Hq, cfg.S, cfg.D), dtype=torch.float16, device="cuda")
    K = torch.empty((cfg.B, cfg.Hkv, cfg.S, cfg.D), dtype=torch.float16, device="cuda")
    L = torch.empty((cfg.B, cfg.Hq, cfg.S), dtype=torch.float32, device="cuda")
    with pytest.raises(lt.LtError) as err:
        lt.lt_attn_bwd_noalloc(Q, K, K, Q, Q, L, Q, K, K, True, cfg.scale)
    assert err.value.status == lt.LT_ERR_WORKSPACE
    assert "built-in scratch" in str(err.value)

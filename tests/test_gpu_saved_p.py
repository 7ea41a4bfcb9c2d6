"""GPU parity of the saved-probability route (Section 4.1: the backward loads the tile P_ij the
forward saved) against the fp64 CPU oracle.

Two halves, tested apart and together:
  * lt_attn_save_p: every stored tile against the oracle's probability matrix (fp16 rounding of a
    value in [0, 1]: |error| <= 2^-11 * P + 2^-24, plus the exponential's own error; 1e-3 absolute
    is the bar), masked entries exactly zero;
  * lt_attn_bwd_saved_p: fed with tiles built on the host from the ORACLE's P (rounded to fp16), and
    fed with lt_attn_save_p's own tiles; gradients to the same bar as lt_attn_bwd."""
import numpy as np
import pytest
import torch

from paper_2606_10415_b200 import workloads
from parity_checks import check_grads

pytestmark = pytest.mark.gpu

P_ABS_TOL = 1e-3


SHAPES = [
    # B, Hq, Hkv, S, D, causal
    (1, 2, 2, 128, 128, True),
    (2, 4, 2, 384, 128, True),
    (1, 4, 1, 300, 128, True),    # ragged last tile, one kv head for four query heads
    (2, 2, 2, 256, 128, False),
    (1, 3, 3, 200, 64, True),     # D = 64, ragged
    (1, 4, 2, 512, 64, False),
    (1, 1, 1, 1, 128, True),      # one row
]


@pytest.fixture(scope="module")
def lt():
    from paper_2606_10415_b200 import binding
    return binding


def tiles_from_matrix(P, causal):
    """Host restatement of the store layout: P [B,Hq,S,S] (float64) -> fp16 tiles
    [B,Hq,nT,nT,16,128,8] with tile (j, i)[c, key, q] = P[query row 128 i + 8 c + q, key column 128 j + key],
    zero padded (sixteen blocks of eight query columns per tile)."""
    B, Hq, S, _ = P.shape
    nT = (S + 127) // 128
    padded = np.zeros((B, Hq, nT * 128, nT * 128))
    padded[:, :, :S, :S] = P
    t = padded.reshape(B, Hq, nT, 16, 8, nT, 128)    # b, h, i, c, q, j, key
    return np.ascontiguousarray(t.transpose(0, 1, 5, 2, 3, 6, 4)).astype(np.float16)  # b, h, j, i, c, key, q


def forward_state(oracle, cfg):
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, cfg.causal, cfg.scale)
    return (Q, K, V, dO), (Qn, Kn, Vn, dOn), torch.from_numpy(O_ref).half(), torch.from_numpy(LSE_ref).float()


def run_save_p(lt, Q, K, LSE, cfg):
    nbytes = lt.lt_attn_p_store_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D)
    nT = (cfg.S + 127) // 128
    assert nbytes == cfg.B * cfg.Hq * nT * nT * 128 * 128 * 2
    P = torch.full((cfg.B, cfg.Hq, nT, nT, 16, 128, 8), float("nan"), dtype=torch.float16, device="cuda")
    ws = lt.alloc_workspace(256)
    lt.lt_attn_save_p(Q.cuda(), K.cuda(), LSE.cuda(), P, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    return P


def run_bwd_saved_p(lt, Q, K, V, O, dO, P, cfg):
    Qd, Kd, Vd, Od, dOd = (t.cuda() for t in (Q, K, V, O, dO))
    dQ, dK, dV = torch.empty_like(Qd), torch.empty_like(Kd), torch.empty_like(Vd)
    for t in (dQ, dK, dV):
        t.fill_(float("nan"))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    ws.fill_(0xFF)
    lt.lt_attn_bwd_saved_p(Qd, Kd, Vd, Od, dOd, P, dQ, dK, dV, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    return dQ.cpu(), dK.cpu(), dV.cpu()


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", SHAPES)
def test_saved_tiles_match_oracle_probabilities(lt, oracle, B, Hq, Hkv, S, D, causal):
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, seed=31 + S)
    (Q, K, V, dO), (Qn, Kn, Vn, dOn), O16, LSE = forward_state(oracle, cfg)
    got = run_save_p(lt, Q, K, LSE, cfg).cpu().double().numpy()
    ref = tiles_from_matrix(oracle.attn_probabilities(Qn, Kn, causal, cfg.scale), causal).astype(np.float64)
    nT = got.shape[2]
    for j in range(nT):
        for i in range(nT):
            if causal and i < j:
                continue  # not written, never read
            g, r = got[:, :, j, i], ref[:, :, j, i]
            assert np.all(np.isfinite(g)), f"tile ({j},{i}) has unwritten entries"
            assert np.abs(g - r).max() <= P_ABS_TOL, f"tile ({j},{i}): {np.abs(g - r).max():.3e}"
            assert np.all(g[r == 0.0] == 0.0), f"tile ({j},{i}): hidden entries must be exact zeros"


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", SHAPES)
def test_backward_from_oracle_tiles_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal):
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, seed=57 + S)
    (Q, K, V, dO), (Qn, Kn, Vn, dOn), O16, LSE = forward_state(oracle, cfg)
    P = oracle.attn_probabilities(Qn, Kn, causal, cfg.scale)
    tiles = torch.from_numpy(tiles_from_matrix(P, causal)).cuda()
    got = run_bwd_saved_p(lt, Q, K, V, O16, dO, tiles, cfg)
    if S > 1:  # (one row: dQ is exactly zero, nothing to divide by)
        check_grads(got, oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale), f"saved-P {cfg}")
    else:
        assert float(got[0].abs().max()) == 0.0
    # and the route's own definition: the oracle's backward from the same fp16-rounded P
    P16 = P.astype(np.float16).astype(np.float64)
    if S > 1:
        check_grads(got, oracle.attn_bwd_from_p(P16, Qn, Kn, Vn, dOn, cfg.scale), f"saved-P (rounded P) {cfg}")


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", [s for s in SHAPES if s[3] > 1])
def test_save_then_backward_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal):
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, seed=91 + S)
    (Q, K, V, dO), (Qn, Kn, Vn, dOn), O16, LSE = forward_state(oracle, cfg)
    P = run_save_p(lt, Q, K, LSE, cfg)
    got = run_bwd_saved_p(lt, Q, K, V, O16, dO, P, cfg)
    check_grads(got, oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale), f"save+bwd {cfg}")


def test_saved_p_route_agrees_with_recompute_route_at_several_tiles_per_cta(lt, oracle):
    """A shape with more work items than SMs and long inner loops (S = 2048, 16 heads): the two CUDA
    routes against each other everywhere, and against the oracle on the last 128 query rows of two
    heads (their dQ rows need every key tile)."""
    cfg = workloads.custom(2, 16, 16, 2048, 128, True, seed=5)
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
    O = torch.empty_like(Qd)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd(Qd, Kd, Vd, O, LSE, True, cfg.scale, ws)
    P = torch.empty(lt.lt_attn_p_store_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D) // 2, dtype=torch.float16, device="cuda")
    lt.lt_attn_save_p(Qd, Kd, LSE, P, True, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    a = [torch.empty_like(t) for t in (Qd, Kd, Vd)]
    b = [torch.empty_like(t) for t in (Qd, Kd, Vd)]
    lt.lt_attn_bwd(Qd, Kd, Vd, O, dOd, LSE, *a, True, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    lt.lt_attn_bwd_saved_p(Qd, Kd, Vd, O, dOd, P, *b, True, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    for name, x, y in zip(("dQ", "dK", "dV"), a, b):
        x, y = x.double(), y.double()
        assert torch.isfinite(y).all()
        rel = float((x - y).norm() / x.norm())
        assert rel <= 5e-3, f"{name}: routes differ by {rel:.3e}"
    # oracle on a slice: heads (0, 3) and (1, 9), all rows (S = 2048 finishes in seconds for two heads)
    for bb, hh in ((0, 3), (1, 9)):
        sl = lambda t: t[bb:bb + 1, hh:hh + 1].double().numpy()
        ref = oracle.attn_bwd(sl(Q), sl(K), sl(V), sl(dO), True, cfg.scale)
        got = tuple(t[bb:bb + 1, hh:hh + 1].cpu() for t in b)
        check_grads(got, ref, f"saved-P slice ({bb},{hh})")


@pytest.mark.parametrize("name,units", [
    ("llama2_7b", [(0, 0), (0, 13), (0, 31)]),            # the launch bench.py's saved_p leg times
    ("qwen25_32b_gqa", [(0, 5)]),                          # groups of five query heads per kv head
    ("llama2_7b_s3000_ragged", [(0, 20)]),                 # ragged last tile at full width
])
def test_saved_p_route_on_benchmark_configurations(lt, oracle, name, units):
    """Forward, lt_attn_save_p and lt_attn_bwd_saved_p at full size on the GPU; the (batch, kv head)
    units in `units` -- all query heads of the group -- against the oracle."""
    cfg = workloads.ALL_CONFIGS[name]
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
    O = torch.empty_like(Qd)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D)
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(*dims))
    lt.lt_attn_fwd(Qd, Kd, Vd, O, LSE, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    P = torch.empty(lt.lt_attn_p_store_bytes(*dims) // 2, dtype=torch.float16, device="cuda")
    lt.lt_attn_save_p(Qd, Kd, LSE, P, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    got = [torch.full_like(t, float("nan")) for t in (Qd, Kd, Vd)]
    lt.lt_attn_bwd_saved_p(Qd, Kd, Vd, O, dOd, P, *got, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    got = [t.cpu() for t in got]
    for t in got:
        assert torch.isfinite(t.float()).all()
    G = cfg.Hq // cfg.Hkv
    for (b, g) in units:
        hs = slice(g * G, (g + 1) * G)
        sub_n = [t.double().numpy() for t in (Q[b:b + 1, hs], K[b:b + 1, g:g + 1], V[b:b + 1, g:g + 1], dO[b:b + 1, hs])]
        ref = oracle.attn_bwd(*sub_n, cfg.causal, cfg.scale)
        sub_got = (got[0][b:b + 1, hs], got[1][b:b + 1, g:g + 1], got[2][b:b + 1, g:g + 1])
        check_grads(sub_got, ref, f"saved-P {name} unit {(b, g)}")

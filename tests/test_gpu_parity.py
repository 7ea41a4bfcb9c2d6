"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle
on the same seeded inputs.  Tolerances per gradient tensor: relative Frobenius error <= 5e-3 and
max abs error <= 2e-2 (as the target states) plus a scale-normalised element bound and a per-row
bound (parity_checks.py).  Forward (not specified by the target): O relative Frobenius <= 2e-3,
LSE max abs <= 1e-3."""
import numpy as np
import pytest
import torch

from paper_2606_10415_b200 import workloads
from parity_checks import REL_FRO_TOL, MAX_ABS_TOL, check_grads, check_tensor, max_abs, rel_fro

pytestmark = pytest.mark.gpu

FWD_O_REL_FRO_TOL = 2e-3
FWD_LSE_ABS_TOL = 1e-3


@pytest.fixture(scope="module")
def lt():
    from paper_2606_10415_b200 import binding
    return binding


def run_fwd(lt, Q, K, V, cfg):
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O = torch.empty_like(Qd)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd(Qd, Kd, Vd, O, LSE, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    return O, LSE


def run_bwd(lt, Q, K, V, O, dO, LSE, cfg):
    Qd, Kd, Vd, Od, dOd, Ld = (t.cuda() for t in (Q, K, V, O, dO, LSE))
    dQ, dK, dV = torch.empty_like(Qd), torch.empty_like(Kd), torch.empty_like(Vd)
    # poison the outputs: the call must overwrite every element
    for t in (dQ, dK, dV):
        t.fill_(float("nan"))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    ws.fill_(0xFF)
    lt.lt_attn_bwd(Qd, Kd, Vd, Od, dOd, Ld, dQ, dK, dV, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    return dQ.cpu(), dK.cpu(), dV.cpu()


# ------------------------------------------------------------------ tensor-core tile conventions

@pytest.mark.parametrize("mode", [0, 1, 2, 3, 4, 5])
def test_tile_gemm_operand_conventions(lt, mode):
    gen = torch.Generator().manual_seed(100 + mode)
    A = torch.randn(128, 128, generator=gen).half()
    B = torch.randn(128, 128, generator=gen).half()
    ref = {0: A.double() @ B.double().T, 1: A.double() @ B.double(),
           2: A.double().T @ B.double(), 3: A.double() @ B.double(), 4: A.double() @ B.double().T,
           5: A.double() @ B.double().T + 1000.0 * B.double()[:, 0][None, :]}[mode]
    C = torch.full((128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(256)
    lt.lt_dbg_tile_gemm(A.cuda(), B.cuda(), C, mode, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    err = (C.cpu().double() - ref).abs().max().item()
    assert err < (2e-2 if mode == 5 else 1e-3), f"mode {mode}: max abs error {err}"


def test_tensor_memory_store_arrangements(lt):
    """The two 16-lane store shapes put every register where the kernels assume (mode 6 writes
    1000 * row + column through them and reads the tile back with the 32-lane shape)."""
    A = torch.zeros(128, 128).half().cuda()
    C = torch.full((128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(256)
    lt.lt_dbg_tile_gemm(A, A, C, 6, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    rows = torch.arange(128, dtype=torch.float32)[:, None]
    cols = torch.arange(96, dtype=torch.float32)[None, :]
    assert torch.equal(C.cpu()[:, :96], 1000.0 * rows + cols)


def test_bounded_wait_reports_timeout_and_context_survives(lt):
    """A wait that nothing satisfies gives up, records its code, and the next call still works."""
    ws = lt.alloc_workspace(256)
    lt.lt_dbg_wait_timeout(ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_ERR_DEVICE_TIMEOUT
    assert "901" in lt.last_cuda_error()
    # the context is intact: a normal kernel runs and reports ok
    A = torch.eye(128).half().cuda()
    C = torch.zeros(128, 128, device="cuda")
    lt.lt_dbg_tile_gemm(A, A, C, 0, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK
    assert torch.equal(C.cpu(), torch.eye(128))


# ------------------------------------------------------------------ forward

FWD_SHAPES = [
    (1, 2, 2, 128, 64, True), (1, 2, 2, 128, 128, True), (2, 4, 2, 384, 64, True),
    (1, 5, 1, 512, 128, True), (1, 2, 2, 256, 128, False), (2, 2, 1, 384, 64, False),
    # ragged last tiles: shorter than one tile, one row past a tile, odd tile counts
    (2, 2, 1, 1, 64, True), (1, 2, 2, 100, 128, True), (2, 4, 2, 129, 64, True), (1, 3, 1, 333, 128, True),
    (1, 2, 2, 100, 128, False), (2, 2, 1, 257, 64, False), (1, 2, 1, 200, 128, False),
]


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", FWD_SHAPES)
def test_forward_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal):
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, qkv_std=1.0, do_std=1.0, seed=S + D)
    Q, K, V, _ = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    O_ref, LSE_ref = oracle.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(), causal, cfg.scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL


# ------------------------------------------------------------------ backward

def test_delta_preprocess_matches_oracle(lt, oracle):
    """-delta is stored after the status block of the backward workspace as 16-byte rows
    of fp16 (hi, lo, 0...) with 256*hi + lo = -delta."""
    cfg = workloads.custom(2, 3, 3, 256, 128, True, seed=7)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O_ref, LSE_ref = oracle.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(), True, cfg.scale)
    O16 = torch.from_numpy(O_ref).half()
    Qd, Kd, Vd, Od, dOd = (t.cuda() for t in (Q, K, V, O16, dO))
    Ld = torch.from_numpy(LSE_ref).float().cuda()
    dQ, dK, dV = torch.empty_like(Qd), torch.empty_like(Kd), torch.empty_like(Vd)
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_bwd(Qd, Kd, Vd, Od, dOd, Ld, dQ, dK, dV, True, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK
    n = cfg.B * cfg.Hq * cfg.S  # S is a whole number of tiles here, so the row space has no padding
    rows = ws[256:256 + 16 * n].view(torch.float16).cpu().double().numpy().reshape(n, 8)
    assert np.all(rows[:, 2:] == 0)
    delta = -(256.0 * rows[:, 0] + rows[:, 1]).reshape(cfg.B, cfg.Hq, cfg.S)
    ref = oracle.delta(dO.double().numpy(), O16.double().numpy())
    # The stored row is a two-term fp16 split (256*hi + lo): hi carries 11 bits of delta/256 and lo 11 bits of
    # the remainder, so a value keeps about 22 bits relative to its own size, but lo goes subnormal (absolute
    # step 2^-24) for deltas far below the largest one: hence an absolute term of 2e-6 of the largest |delta|
    # beside the relative one.
    np.testing.assert_allclose(delta, ref, rtol=1e-5, atol=2e-6 * np.abs(ref).max())


BWD_SHAPES = [
    # B, Hq, Hkv, S, D, causal
    (1, 2, 2, 128, 64, True), (1, 2, 2, 128, 128, True), (1, 1, 1, 256, 128, True),
    (2, 4, 2, 384, 64, True), (1, 5, 1, 512, 128, True), (2, 8, 1, 256, 128, True),
    (1, 2, 2, 256, 128, False), (2, 4, 2, 384, 64, False), (1, 1, 1, 128, 128, False),
    # ragged last tiles
    (2, 2, 1, 3, 64, True), (1, 2, 2, 100, 128, True), (2, 4, 2, 129, 64, True), (1, 6, 2, 333, 128, True),
    (1, 2, 2, 100, 128, False), (2, 2, 1, 257, 64, False), (1, 4, 1, 200, 128, False),
]


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", BWD_SHAPES)
@pytest.mark.parametrize("stds", [(1.0, 1.0), (None, 1e-2)])
def test_backward_matches_oracle_small(lt, oracle, B, Hq, Hkv, S, D, causal, stds):
    """Several tiles, GQA groups, both head dims; forward state taken from the oracle
    (O rounded to fp16, LSE to fp32) so the backward is checked on its own."""
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, qkv_std=stds[0], do_std=stds[1], seed=B * 1000 + S + D)
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, causal, cfg.scale)
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale)
    got = run_bwd(lt, Q, K, V, torch.from_numpy(O_ref).half(), dO, torch.from_numpy(LSE_ref).float(), cfg)
    check_grads(got, ref, f"{cfg}")


def test_tiny_config_end_to_end(lt, oracle):
    """The tiny benchmark configuration with the library's own forward feeding its backward."""
    cfg = workloads.CONFIGS["tiny"]
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    got = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    ref = oracle.attn_bwd(*(t.double().numpy() for t in (Q, K, V, dO)), cfg.causal, cfg.scale)
    check_grads(got, ref, "tiny")


def test_backward_is_linear_in_dO_and_repeatable(lt, oracle):
    cfg = workloads.custom(1, 4, 2, 256, 128, True, seed=11)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    a = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    b = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    # dK and dV have a fixed summation order; dQ is reduced with atomics
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    assert rel_fro(a[0].double().numpy(), b[0].double().numpy()) < 1e-3
    c = run_bwd(lt, Q, K, V, O.cpu(), (dO.float() * 4).half(), LSE.cpu(), cfg)
    for x, y in zip(a, c):
        assert rel_fro(y.double().numpy() / 4, x.double().numpy()) < 2e-3


def test_zero_dO_gives_zero_gradients(lt):
    cfg = workloads.custom(1, 2, 1, 256, 64, True, seed=12)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    got = run_bwd(lt, Q, K, V, O.cpu(), torch.zeros_like(dO), LSE.cpu(), cfg)
    for g in got:
        assert torch.count_nonzero(g) == 0


@pytest.mark.parametrize("do_std", [1e-3, 30.0])
def test_gradient_magnitude_extremes(lt, oracle, do_std):
    """The fp16 dS operand carries a per-work-item power-of-two factor chosen from a bound on
    |dP - delta|; upstream gradients far below and above the usual range must keep the relative
    accuracy.  (Below about 1e-3 the fp16 outputs themselves go subnormal, which no kernel can mend.)"""
    cfg = workloads.custom(1, 4, 2, 384, 128, True, qkv_std=128.0 ** -0.25, do_std=do_std, seed=21)
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, True, cfg.scale)
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, True, cfg.scale)
    got = run_bwd(lt, Q, K, V, torch.from_numpy(O_ref).half(), dO, torch.from_numpy(LSE_ref).float(), cfg)
    check_grads(got, ref, f"dO std {do_std}", absolute=False)


@pytest.mark.parametrize("v_scale,do_std", [(1e-3, 1.0), (40.0, 1e-2), (600.0, 1e-4), (600.0, 1e-2)])
def test_value_magnitude_extremes(lt, oracle, v_scale, do_std):
    """The bound behind that factor uses the row norms of V, summed in packed half precision after a
    2^-4 pre-scaling: tiny values (squares below fp16's range), outlier-sized values (elements of several
    hundred, whose plain squares would overflow fp16) and their combination with small upstream gradients
    must keep the relative accuracy (the tiny values come with a large upstream gradient, so that the fp16
    outputs themselves stay representable).  D = 128 and D = 64, fp16 and bf16."""
    for D, bf16 in ((128, False), (64, False), (128, True)):
        cfg = workloads.custom(1, 4, 2, 300, D, True, do_std=do_std, seed=77)
        Q, K, V, dO = workloads.make_inputs(cfg)
        V = (V.float() * v_scale).half()
        if bf16:
            Q, K, V, dO = (t.float().bfloat16() for t in (Q, K, V, dO))
        Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
        O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, True, cfg.scale)
        ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, True, cfg.scale)
        O = torch.from_numpy(O_ref).to(Q.dtype)
        LSE = torch.from_numpy(LSE_ref).float()
        Qd, Kd, Vd, Od, dOd, Ld = (t.cuda() for t in (Q, K, V, O, dO, LSE))
        dQ, dK, dV = torch.empty_like(Qd), torch.empty_like(Kd), torch.empty_like(Vd)
        ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
        if bf16:
            lt.lt_attn_bwd_bf16(Qd, Kd, Vd, Od, dOd, Ld, dQ, dK, dV, True, cfg.scale, ws)
        else:
            lt.lt_attn_bwd(Qd, Kd, Vd, Od, dOd, Ld, dQ, dK, dV, True, cfg.scale, ws)
        assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
        check_grads((dQ, dK, dV), ref, f"D={D} bf16={bf16} V x{v_scale}, dO std {do_std}",
                    dtype="bf16" if bf16 else "fp16", absolute=False)


def test_sharp_softmax_and_large_scores(lt, oracle):
    """Large |scores| (std 4 after scaling): rows dominated by one key, LSE far from 0, probabilities
    spanning the whole fp16 range; also exercises the forward's running-maximum updates."""
    cfg = workloads.custom(1, 2, 2, 512, 64, True, qkv_std=2.0, do_std=1.0, seed=22)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, True, cfg.scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    got = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, True, cfg.scale)
    check_grads(got, ref, "sharp softmax")


def test_negative_scale(lt, oracle):
    """A negative softmax scale is legal (finite, non-zero): the row maximum then comes from the
    smallest raw score."""
    cfg = workloads.custom(1, 2, 1, 256, 128, True, qkv_std=1.0, do_std=1.0, seed=23)
    Q, K, V, dO = workloads.make_inputs(cfg)
    scale = -cfg.scale
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O = torch.empty_like(Qd)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    fws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd(Qd, Kd, Vd, O, LSE, True, scale, fws)
    assert lt.lt_attn_check_status(fws) == lt.LT_OK
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, True, scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    dQ, dK, dV = torch.empty_like(Qd), torch.empty_like(Kd), torch.empty_like(Vd)
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_bwd(Qd, Kd, Vd, O, dO.cuda(), LSE, dQ, dK, dV, True, scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, True, scale)
    check_grads((dQ.cpu(), dK.cpu(), dV.cpu()), ref, "negative scale")


def test_long_sequence_and_wide_group(lt, oracle):
    """S = 8192 (64 key tiles, long dQ accumulation chains) with a group of 16 query heads on one
    key/value head."""
    cfg = workloads.custom(1, 16, 1, 8192, 128, True, seed=24)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    got = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    ref = oracle.attn_bwd(*(t.double().numpy() for t in (Q, K, V, dO)), True, cfg.scale)
    check_grads(got, ref, "S=8192, group of 16")


def test_two_streams_with_distinct_workspaces(lt, oracle):
    """Calls are re-entrant across streams as long as each has its own workspace: two different
    problems enqueued on two streams at once give the results they give alone."""
    cfgs = [workloads.custom(1, 4, 2, 640, 128, True, seed=51), workloads.custom(2, 2, 2, 384, 64, False, seed=52)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    jobs = []
    for cfg in cfgs:
        Q, K, V, dO = workloads.make_inputs(cfg)
        O, LSE = run_fwd(lt, Q, K, V, cfg)
        alone = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
        dev = [t.cuda() for t in (Q, K, V)] + [O, dO.cuda(), LSE]
        outs = [torch.empty_like(dev[0]), torch.empty_like(dev[1]), torch.empty_like(dev[2])]
        ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
        jobs.append((cfg, dev, outs, ws, alone))
    torch.cuda.synchronize()
    for _ in range(3):  # several rounds, so that the two kernels really overlap on the device
        for (cfg, dev, outs, ws, _), st in zip(jobs, streams):
            lt.lt_attn_bwd(*dev, *outs, cfg.causal, cfg.scale, ws, st)
    torch.cuda.synchronize()
    for cfg, dev, outs, ws, alone in jobs:
        assert lt.lt_attn_check_status(ws) == lt.LT_OK
        # dK and dV have a fixed summation order; dQ is reduced with atomics
        assert torch.equal(outs[1].cpu(), alone[1]) and torch.equal(outs[2].cpu(), alone[2])
        assert rel_fro(outs[0].cpu().double().numpy(), alone[0].double().numpy()) < 1e-3


def test_very_long_sequence(lt, oracle):
    """S = 16384: 128 key tiles per head, 8 256 tile pairs per head, dQ rows that receive up to 128
    partial sums."""
    cfg = workloads.custom(1, 2, 1, 16384, 128, True, seed=25)
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    got = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, True, cfg.scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    check_grads(got, oracle.attn_bwd(Qn, Kn, Vn, dOn, True, cfg.scale), "S=16384")


def test_host_buffer_entry_point(lt, oracle):
    cfg = workloads.custom(1, 4, 2, 256, 128, True, seed=13)
    Q, K, V, dO = (t.pin_memory() for t in workloads.make_inputs(cfg))
    O = torch.empty_like(Q).pin_memory()
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32).pin_memory()
    dQ, dK, dV = torch.empty_like(Q).pin_memory(), torch.empty_like(K).pin_memory(), torch.empty_like(V).pin_memory()
    arena = lt.alloc_workspace(lt.lt_attn_host_arena_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd_bwd_host(Q, K, V, dO, O, LSE, dQ, dK, dV, cfg.causal, cfg.scale, arena)
    torch.cuda.synchronize()
    ref = oracle.attn_bwd(*(t.double().numpy() for t in (Q, K, V, dO)), cfg.causal, cfg.scale)
    check_grads((dQ, dK, dV), ref, "host entry")


def test_host_buffer_entry_point_chunked(lt, oracle):
    """A problem large enough for the host entry point to pipeline it in several chunks of
    (batch, kv head) units; every output must be complete and match the oracle on sampled units."""
    cfg = workloads.custom(2, 8, 4, 4096, 128, True, seed=14)
    Q, K, V, dO = (t.pin_memory() for t in workloads.make_inputs(cfg))
    O = torch.full_like(Q, float("nan")).pin_memory()
    LSE = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32).pin_memory()
    dQ, dK, dV = (torch.full_like(t, float("nan")).pin_memory() for t in (Q, K, V))
    arena = lt.alloc_workspace(lt.lt_attn_host_arena_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    for _ in range(2):  # the second call reuses the arena while nothing else orders the two calls
        lt.lt_attn_fwd_bwd_host(Q, K, V, dO, O, LSE, dQ, dK, dV, cfg.causal, cfg.scale, arena)
    torch.cuda.synchronize()
    for t in (O, LSE, dQ, dK, dV):
        assert torch.isfinite(t.float()).all()
    G = cfg.Hq // cfg.Hkv
    for (b, g) in [(0, 0), (0, 3), (1, 1), (1, 3)]:
        hs = slice(g * G, (g + 1) * G)
        sub = [t.double().numpy() for t in (Q[b:b + 1, hs], K[b:b + 1, g:g + 1], V[b:b + 1, g:g + 1], dO[b:b + 1, hs])]
        O_ref, LSE_ref = oracle.attn_fwd(*sub[:3], True, cfg.scale)
        assert rel_fro(O[b:b + 1, hs].double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
        assert max_abs(LSE[b:b + 1, hs].double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
        ref = oracle.attn_bwd(*sub, True, cfg.scale)
        check_grads((dQ[b:b + 1, hs], dK[b:b + 1, g:g + 1], dV[b:b + 1, g:g + 1]), ref, f"host chunked unit {(b, g)}")


# ------------------------------------------------------------------ strided layouts

def _strided_case(lt, oracle, cfg, make_views):
    """Run forward and backward on [B,H,S,D] views built by `make_views` and compare with the
    oracle on contiguous copies of the same values."""
    Q, K, V, dO = workloads.make_inputs(cfg)
    Qv, Kv, Vv, Ov, dOv, dQv, dKv, dVv = make_views(Q, K, V, dO)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    fws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    lt.lt_attn_fwd_strided(Qv, Kv, Vv, Ov, LSE, cfg.causal, cfg.scale, fws)
    assert lt.lt_attn_check_status(fws) == lt.LT_OK, lt.last_cuda_error()
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, cfg.causal, cfg.scale)
    assert rel_fro(Ov.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.S, cfg.D))
    ws.fill_(0xFF)
    lt.lt_attn_bwd_strided(Qv, Kv, Vv, Ov, dOv, LSE, dQv, dKv, dVv, cfg.causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, cfg.causal, cfg.scale)
    check_grads((dQv.cpu(), dKv.cpu(), dVv.cpu()), ref, f"strided {cfg}")


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", [
    (2, 4, 2, 256, 128, True), (1, 3, 3, 200, 64, True), (2, 2, 1, 130, 128, False),
])
def test_bshd_layout_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal):
    """Every tensor stored [B,S,H,D] and handed over as a permuted [B,H,S,D] view."""
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, qkv_std=1.0, do_std=1.0, seed=31 + S)

    def views(Q, K, V, dO):
        def bshd(t):
            return t.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3)

        def out_like(t):
            return torch.full_like(t.permute(0, 2, 1, 3).contiguous(), float("nan"), device="cuda").permute(0, 2, 1, 3)

        return bshd(Q), bshd(K), bshd(V), out_like(Q), bshd(dO), out_like(Q), out_like(K), out_like(V)

    _strided_case(lt, oracle, cfg, views)


def test_fused_qkv_buffer_matches_oracle(lt, oracle):
    """Q, K, V are slices of one [B, S, (Hq + 2 Hkv) * D] projection output; dQ, dK, dV are written
    into the matching slices of one gradient buffer; untouched bytes of that buffer stay as they were."""
    B, Hq, Hkv, S, D = 2, 4, 2, 300, 128
    cfg = workloads.custom(B, Hq, Hkv, S, D, True, seed=77)
    width = (Hq + 2 * Hkv) * D
    pad = 64  # spare elements at the end of every row, never written

    def views(Q, K, V, dO):
        buf = torch.zeros(B, S, width + pad, dtype=torch.float16, device="cuda")
        grad = torch.full((B, S, width + pad), 7.0, dtype=torch.float16, device="cuda")

        def split(t):
            q = t[..., :Hq * D].unflatten(-1, (Hq, D)).permute(0, 2, 1, 3)
            k = t[..., Hq * D:(Hq + Hkv) * D].unflatten(-1, (Hkv, D)).permute(0, 2, 1, 3)
            v = t[..., (Hq + Hkv) * D:width].unflatten(-1, (Hkv, D)).permute(0, 2, 1, 3)
            return q, k, v

        q, k, v = split(buf)
        q.copy_(Q.cuda()); k.copy_(K.cuda()); v.copy_(V.cuda())
        dq, dk, dv = split(grad)
        views.grad = grad
        O = torch.empty(B, Hq, S, D, dtype=torch.float16, device="cuda")
        return q, k, v, O, dO.cuda(), dq, dk, dv

    _strided_case(lt, oracle, cfg, views)
    assert torch.all(views.grad[..., width:] == 7.0)


# ------------------------------------------------------------------ bfloat16

# bf16 keeps 8 significant bits: outputs, P and dS each carry about 2^-9 relative rounding.  The output
# rounding alone gives O a relative Frobenius error of 2^-9 / sqrt(3) = 1.1e-3 (1.9e-3 measured with
# the rounding of P), so the forward gate is twice the fp16 one; the gradients keep the 5e-3 gate.
BF16_FWD_O_REL_FRO_TOL = 4e-3


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal", [
    (1, 2, 2, 128, 64, True), (2, 4, 2, 384, 128, True), (1, 6, 2, 333, 128, True), (1, 2, 1, 256, 64, False),
    (1, 8, 2, 1024, 128, True),
])
def test_bf16_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal):
    """bfloat16 inputs and outputs; the oracle works in fp64 on the bf16-rounded inputs."""
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, seed=41 + S)
    Q, K, V, dO = (t.float().bfloat16() for t in workloads.make_inputs(cfg))
    Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
    O = torch.empty_like(Qd)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    fws = lt.alloc_workspace(lt.lt_attn_fwd_workspace_bytes(B, Hq, Hkv, S, D))
    lt.lt_attn_fwd_bf16(Qd, Kd, Vd, O, LSE, causal, cfg.scale, fws)
    assert lt.lt_attn_check_status(fws) == lt.LT_OK, lt.last_cuda_error()
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, causal, cfg.scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= BF16_FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    dQ, dK, dV = (torch.full_like(t, float("nan")) for t in (Qd, Kd, Vd))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))
    ws.fill_(0xFF)
    lt.lt_attn_bwd_bf16(Qd, Kd, Vd, O, dOd, LSE, dQ, dK, dV, causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale)
    check_grads((dQ, dK, dV), ref, f"bf16 {cfg}", dtype="bf16")


# ------------------------------------------------------------------ benchmark configurations, full size

def _full_size_check(lt, oracle, name):
    """Run the whole configuration on the GPU (the launch the benchmark times) and compare EVERY
    (batch, kv head) unit with the oracle: one oracle call over the whole problem, so that its threads
    work on all heads at once; the gates are applied per batch."""
    cfg = workloads.ALL_CONFIGS[name]
    Q, K, V, dO = workloads.make_inputs(cfg)
    O, LSE = run_fwd(lt, Q, K, V, cfg)
    got = run_bwd(lt, Q, K, V, O.cpu(), dO, LSE.cpu(), cfg)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, cfg.causal, cfg.scale)
    assert rel_fro(O.cpu().double().numpy(), O_ref) <= FWD_O_REL_FRO_TOL
    assert max_abs(LSE.cpu().double().numpy(), LSE_ref) <= FWD_LSE_ABS_TOL
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, cfg.causal, cfg.scale)
    for b in range(cfg.B):
        check_grads([t[b:b + 1] for t in got], [r[b:b + 1] for r in ref], f"{name} batch {b}")
    # a head-sized gate as well: a wrong head must not hide in the norm of the whole tensor
    G = cfg.Hq // cfg.Hkv
    for b in range(cfg.B):
        for g in range(cfg.Hkv):
            hs = slice(g * G, (g + 1) * G)
            for nm, t, r in (("dQ", got[0][b, hs], ref[0][b, hs]), ("dK", got[1][b, g], ref[1][b, g]),
                             ("dV", got[2][b, g], ref[2][b, g])):
                rf = rel_fro(t.double().numpy(), r)
                assert rf <= REL_FRO_TOL, f"{name} unit {(b, g)} {nm}: rel Frobenius {rf:.3e}"
    if cfg.causal:
        assert torch.count_nonzero(got[0][:, :, 0]) == 0  # the first query row sees one key: dQ = 0


@pytest.mark.parametrize("name", ["llama2_7b", "baichuan2_13b", "qwen25_32b_gqa", "llama2_70b_gqa"])
def test_benchmark_config_all_units(lt, oracle, name):
    _full_size_check(lt, oracle, name)


@pytest.mark.parametrize("name", ["llama2_7b_s1024", "llama2_7b_s2048", "qwen25_32b_gqa_s2048",
                                  "llama2_7b_s3000_ragged", "llama2_7b_full_mask_off"])
def test_other_sequence_lengths_and_unmasked(lt, oracle, name):
    """The other lengths and layer shape of the paper's Attention-BP measurement, a ragged length and
    no mask; every unit compared."""
    _full_size_check(lt, oracle, name)


# ------------------------------------------------------------------ head dimension 64 at length

@pytest.mark.parametrize("B,Hq,Hkv,S,causal,bf16", [
    (1, 8, 8, 2048, True, False),    # 16 key tiles per head: long dQ accumulation chains through the tiled reductions
    (2, 8, 2, 1900, True, True),     # grouped heads, ragged last tile, bf16
    (1, 4, 4, 1536, False, False),   # no mask
])
def test_head_dim_64_matches_oracle(lt, oracle, B, Hq, Hkv, S, causal, bf16):
    """D = 64 takes its own dQ path (swizzled staging, tiled reductions through a tensor map over the
    accumulator); every unit is compared."""
    cfg = workloads.custom(B, Hq, Hkv, S, 64, causal, seed=91 + S)
    dt = torch.bfloat16 if bf16 else torch.float16
    Q, K, V, dO = (t.float().to(dt) for t in workloads.make_inputs(cfg))
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, causal, cfg.scale)
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale)
    Qd, Kd, Vd, dOd = (t.cuda() for t in (Q, K, V, dO))
    Od = torch.from_numpy(O_ref).to(dt).cuda()
    dQ, dK, dV = (torch.full_like(t, float("nan")) for t in (Qd, Kd, Vd))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, 64))
    ws.fill_(0xFF)
    bwd = lt.lt_attn_bwd_bf16 if bf16 else lt.lt_attn_bwd
    bwd(Qd, Kd, Vd, Od, dOd, torch.from_numpy(LSE_ref).float().cuda(), dQ, dK, dV, causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    check_grads((dQ, dK, dV), ref, f"D=64 {cfg} bf16={bf16}", dtype="bf16" if bf16 else "fp16")


# ------------------------------------------------------------------ split-group variant

# Shapes with few, heavy work items: a group's query heads are spread over several items per key tile
# and dK / dV are summed in fp32 in the workspace (a separate instantiation of the main kernel plus the
# dK/dV conversion kernel).  Every unit is compared.
SPLIT_CASES = [
    # B, Hq, Hkv, S, D, causal, bf16, layout
    (1, 8, 2, 3500, 64, True, False, "bhsd"),     # D = 64, ragged last tile (28 tiles, 3 248 iterations)
    (1, 8, 2, 3500, 64, True, True, "bshd"),      # the same in bf16 with [B,S,H,D] tensors (strided dK/dV stores)
    (1, 8, 2, 2560, 128, False, False, "bhsd"),   # no mask
    (1, 10, 2, 2989, 128, True, True, "bhsd"),    # D = 128 bf16, ragged, group of five
    (2, 8, 1, 2432, 128, True, False, "bshd"),    # two batches, group of eight, strided
]


@pytest.mark.parametrize("B,Hq,Hkv,S,D,causal,bf16,layout", SPLIT_CASES)
def test_split_group_variant_matches_oracle(lt, oracle, B, Hq, Hkv, S, D, causal, bf16, layout):
    assert lt.lt_attn_bwd_num_launches(B, Hq, Hkv, S, D, causal) == 4, "this shape no longer takes the split variant"
    cfg = workloads.custom(B, Hq, Hkv, S, D, causal, seed=61 + S)
    dt = torch.bfloat16 if bf16 else torch.float16
    Q, K, V, dO = (t.float().to(dt) for t in workloads.make_inputs(cfg))
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O_ref, LSE_ref = oracle.attn_fwd(Qn, Kn, Vn, causal, cfg.scale)
    ref = oracle.attn_bwd(Qn, Kn, Vn, dOn, causal, cfg.scale)

    def place(t, fill=None):
        if layout == "bshd":
            base = t.permute(0, 2, 1, 3).contiguous()
            base = (base if fill is None else torch.full_like(base, fill)).cuda()
            return base.permute(0, 2, 1, 3)
        return t.cuda() if fill is None else torch.full_like(t, fill).cuda()

    O = torch.from_numpy(O_ref).to(dt)
    Qd, Kd, Vd, Od, dOd = (place(t) for t in (Q, K, V, O, dO))
    dQ, dK, dV = (place(t, float("nan")) for t in (Q, K, V))
    ws = lt.alloc_workspace(lt.lt_attn_bwd_workspace_bytes(B, Hq, Hkv, S, D))
    ws.fill_(0xFF)
    bwd = lt.lt_attn_bwd_bf16 if bf16 else lt.lt_attn_bwd_strided
    bwd(Qd, Kd, Vd, Od, dOd, torch.from_numpy(LSE_ref).float().cuda(), dQ, dK, dV, causal, cfg.scale, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    check_grads((dQ, dK, dV), ref, f"split {cfg} bf16={bf16} {layout}", dtype="bf16" if bf16 else "fp16")

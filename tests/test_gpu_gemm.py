"""Parity of the FP16 GEMM (C = A W^T) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

# fp16 output rounding (2^-11 per element) dominates; fp32 accumulation adds far less
GEMM_REL_FRO_TOL = 1e-3


@pytest.fixture(scope="module")
def lt():
    from paper_2606_10415_b200 import binding
    return binding


def rel_fro(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def make_operands(M, N, K, seed):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    A = torch.randn((M, K), generator=gen, dtype=torch.float32).half()
    W = (torch.randn((N, K), generator=gen, dtype=torch.float32) * K ** -0.5).half()
    return A, W


def run_gemm(lt, A, W):
    Ad, Wd = A.cuda(), W.cuda()
    C = torch.full((A.shape[0], W.shape[0]), float("nan"), dtype=torch.float16, device="cuda")
    ws = lt.alloc_workspace(lt.lt_gemm_f16_workspace_bytes())
    lt.lt_gemm_f16(Ad, Wd, C, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    return C.cpu()


@pytest.mark.parametrize("M,N,K", [
    (128, 256, 64), (128, 256, 256), (256, 512, 512),            # whole tiles
    (1, 8, 8), (100, 200, 72), (129, 257, 136), (300, 1000, 520),  # ragged in every dimension
    (384, 250, 64), (77, 36, 1024),                                # N not a multiple of 8: scalar stores
    (2048, 1024, 768),                                             # more tiles than SMs would need twice
    (128, 40000, 128),   # one tile row: the single-CTA kernel, 157 tiles over 148 CTAs (accumulator ring reused)
    (520, 20000, 192),   # CTA pairs: 3 x 79 tiles of 256 x 256 over 74 pairs (both accumulators reused), ragged M and N
])
def test_gemm_matches_oracle(lt, oracle, M, N, K):
    A, W = make_operands(M, N, K, seed=M + N + K)
    C = run_gemm(lt, A, W)
    ref = oracle.gemm_nt(A.double().numpy(), W.double().numpy())
    got = C.double().numpy()
    assert np.all(np.isfinite(got))
    assert rel_fro(got, ref) <= GEMM_REL_FRO_TOL, f"{(M, N, K)}: {rel_fro(got, ref):.3e}"
    # element-wise: within fp16 rounding of the exact value plus accumulation slack
    assert np.max(np.abs(got - ref) - 2.0 ** -10 * np.abs(ref)) <= 1e-3


def test_gemm_integer_operands_are_exact(lt, oracle):
    """Small integers: every product and partial sum is exact in fp32 and fp16, so the result must
    equal the oracle bit for bit."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1)
    A = torch.randint(-3, 4, (200, 136), generator=gen).half()
    W = torch.randint(-2, 3, (300, 136), generator=gen).half()
    C = run_gemm(lt, A, W)
    ref = oracle.gemm_nt(A.double().numpy(), W.double().numpy())
    assert np.array_equal(C.double().numpy(), ref)


@pytest.mark.parametrize("N,K", [(4096, 4096), (11008, 4096), (4096, 11008), (6656, 6656), (8192, 8192)])
def test_gemm_paper_shapes_sampled_rows(lt, oracle, N, K):
    """The five weight shapes of the paper's GEMM profile (Section 6.6) at its sequence length of 2048
    rows; the launch the benchmark times, compared on sampled rows and columns."""
    M = 2048
    A, W = make_operands(M, N, K, seed=N + K)
    C = run_gemm(lt, A, W)
    assert torch.isfinite(C.float()).all()
    rows = [0, 1, 127, 128, 1000, 2047]
    ref = oracle.gemm_nt(A[rows].double().numpy(), W.double().numpy())
    assert rel_fro(C[rows].double().numpy(), ref) <= GEMM_REL_FRO_TOL
    cols = [0, 255, 256, N // 2 + 3, N - 1]
    ref_c = oracle.gemm_nt(A.double().numpy(), W[cols].double().numpy())
    assert rel_fro(C[:, cols].double().numpy(), ref_c) <= GEMM_REL_FRO_TOL


@pytest.mark.parametrize("M,N,K", [(129, 257, 136), (512, 768, 1024)])
def test_gemm_bf16_matches_oracle(lt, oracle, M, N, K):
    A, W = (t.float().bfloat16() for t in make_operands(M, N, K, seed=7 + M))
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = lt.alloc_workspace(lt.lt_gemm_f16_workspace_bytes())
    lt.lt_gemm_f16(A.cuda(), W.cuda(), C, ws)
    assert lt.lt_attn_check_status(ws) == lt.LT_OK, lt.last_cuda_error()
    ref = oracle.gemm_nt(A.double().numpy(), W.double().numpy())
    # bf16 output rounding: 2^-9 per element
    assert rel_fro(C.cpu().double().numpy(), ref) <= 4e-3


@pytest.mark.parametrize("seed", [0, 1])
def test_gemm_random_shapes(lt, oracle, seed):
    """Seeded sweep over ragged shapes on both kernels (one tile row: single CTA; more: CTA pairs):
    integer operands, so every result is exact and compared bit for bit."""
    rng = np.random.default_rng(1000 + seed)
    for case in range(12):
        M = int(rng.choice([1, 64, 127, 128, 129, 255, 256, 257, 384, 513, 700, 1100]))
        N = int(rng.integers(1, 1400))
        K = 8 * int(rng.integers(1, 90))
        gen = torch.Generator(device="cpu")
        gen.manual_seed(seed * 100 + case)
        A = torch.randint(-3, 4, (M, K), generator=gen).half()
        W = torch.randint(-2, 3, (N, K), generator=gen).half()
        C = run_gemm(lt, A, W)
        ref = oracle.gemm_nt(A.double().numpy(), W.double().numpy())
        assert np.array_equal(C.double().numpy(), ref), f"case {case}: M={M} N={N} K={K}"


def test_gemm_pair_kernel_on_two_streams(lt, oracle):
    """Two products on two streams at once (clusters of both launches share the SMs); each has its own
    status block and result."""
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    A1, W1 = make_operands(1024, 2048, 512, seed=21)
    A2, W2 = make_operands(768, 1536, 1024, seed=22)
    d = [t.cuda() for t in (A1, W1, A2, W2)]
    C1 = torch.full((1024, 2048), float("nan"), dtype=torch.float16, device="cuda")
    C2 = torch.full((768, 1536), float("nan"), dtype=torch.float16, device="cuda")
    w1, w2 = lt.alloc_workspace(256), lt.alloc_workspace(256)
    torch.cuda.synchronize()
    for _ in range(5):
        lt.lt_gemm_f16(d[0], d[1], C1, w1, s1)
        lt.lt_gemm_f16(d[2], d[3], C2, w2, s2)
    torch.cuda.synchronize()
    assert lt.lt_attn_check_status(w1) == lt.LT_OK and lt.lt_attn_check_status(w2) == lt.LT_OK, lt.last_cuda_error()
    for C, A, W in ((C1, A1, W1), (C2, A2, W2)):
        ref = oracle.gemm_nt(A.double().numpy(), W.double().numpy())
        assert rel_fro(C.cpu().double().numpy(), ref) <= GEMM_REL_FRO_TOL

"""Pins for the CPU oracle: each checks it against something other than itself.

The paper gives no worked numbers for Attention Backward, so the pins are what
the mathematics fixes: finite differences of the loss L = sum(O * dO), a
brute-force softmax Jacobian, closed forms, invariants that only hold if
rowsum(dS) = 0, an explicit-mask brute force, a hand-worked two-key example
(tests/golden), and torch's fp64 autograd as an independent library route.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

GOLDEN = Path(__file__).resolve().parent / "golden"


def rnd(shape, seed, std=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * std


def loss(oracle, Q, K, V, dO, causal, scale):
    O, _ = oracle.attn_fwd(Q, K, V, causal, scale)
    return float(np.sum(O * dO))


# ---------------------------------------------------------------- forward: P, LSE, mask

def brute_forward(Q, K, V, causal, scale):
    """Explicit S x S matrices, mask built by a double loop, long-double logsumexp."""
    B, Hq, S, D = Q.shape
    G = Hq // K.shape[1]
    O = np.zeros_like(Q)
    LSE = np.zeros((B, Hq, S))
    P = np.zeros((B, Hq, S, S))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            s = scale * (Q[b, h] @ K[b, g].T)
            hidden = np.zeros((S, S), dtype=bool)
            if causal:
                for i in range(S):
                    for j in range(S):
                        hidden[i, j] = i < j
            for i in range(S):
                vis = [j for j in range(S) if not hidden[i, j]]
                e = np.exp(s[i, vis].astype(np.longdouble))
                tot = e.sum()
                LSE[b, h, i] = float(np.log(tot))
                P[b, h, i, vis] = (e / tot).astype(np.float64)
            O[b, h] = P[b, h] @ V[b, g]
    return O, LSE, P


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (4, 2)])
def test_forward_matches_explicit_mask_brute_force(oracle, causal, Hq, Hkv):
    Q, K, V = rnd((2, Hq, 12, 8), 1), rnd((2, Hkv, 12, 8), 2), rnd((2, Hkv, 12, 8), 3)
    O, LSE = oracle.attn_fwd(Q, K, V, causal, 0.37)
    Ob, LSEb, P = brute_forward(Q, K, V, causal, 0.37)
    np.testing.assert_allclose(O, Ob, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(LSE, LSEb, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(P.sum(-1), 1.0, rtol=1e-13)
    if causal:
        assert np.all(np.triu(P, 1) == 0.0)


def test_causal_no_leak_from_future_keys(oracle):
    Q, K, V = rnd((1, 2, 16, 8), 4), rnd((1, 2, 16, 8), 5), rnd((1, 2, 16, 8), 6)
    O0, L0 = oracle.attn_fwd(Q, K, V, True, 0.5)
    K2, V2 = K.copy(), V.copy()
    K2[:, :, 9:] += 3.0
    V2[:, :, 9:] -= 7.0
    O1, L1 = oracle.attn_fwd(Q, K2, V2, True, 0.5)
    assert np.array_equal(O0[:, :, :9], O1[:, :, :9])
    assert np.array_equal(L0[:, :, :9], L1[:, :, :9])
    assert not np.array_equal(O0[:, :, 9:], O1[:, :, 9:])


def test_large_scores_do_not_overflow(oracle):
    Q, K, V = rnd((1, 1, 8, 4), 7, 30.0), rnd((1, 1, 8, 4), 8, 30.0), rnd((1, 1, 8, 4), 9)
    O, LSE = oracle.attn_fwd(Q, K, V, False, 1.0)
    assert np.all(np.isfinite(O)) and np.all(np.isfinite(LSE))
    _, LSEb, _ = brute_forward(Q / 30.0, K / 30.0, V, False, 1.0)  # sanity of the helper itself
    assert np.all(np.isfinite(LSEb))


# ---------------------------------------------------------------- whole backward

@pytest.mark.parametrize("causal", [False, True])
def test_finite_differences_all_coordinates(oracle, causal):
    """Central differences of L = sum(O*dO) at B=1, Hq=2, Hkv=1, S=16, D=8: every coordinate."""
    B, Hq, Hkv, S, D = 1, 2, 1, 16, 8
    Q, K, V = rnd((B, Hq, S, D), 10), rnd((B, Hkv, S, D), 11), rnd((B, Hkv, S, D), 12)
    dO = rnd((B, Hq, S, D), 13)
    scale = 0.41
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, causal, scale)
    for name, X, g in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        flat = X.reshape(-1)
        num = np.empty_like(flat)
        for idx in range(flat.size):
            old = flat[idx]
            eps = 1e-5 * max(1.0, abs(old))
            flat[idx] = old + eps
            lp = loss(oracle, Q, K, V, dO, causal, scale)
            flat[idx] = old - eps
            lm = loss(oracle, Q, K, V, dO, causal, scale)
            flat[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        err = np.abs(num - g.reshape(-1)).max() / np.abs(g).max()
        assert err < 1e-7, (name, err)


def test_finite_differences_sampled_config1_shape(oracle):
    """256 random coordinates at the tiny benchmark shape (B=1, H=2, S=128, D=64, causal)."""
    B, H, S, D = 1, 2, 128, 64
    Q, K, V, dO = (rnd((B, H, S, D), s) for s in (20, 21, 22, 23))
    scale = D ** -0.5
    grads = dict(zip("QKV", oracle.attn_bwd(Q, K, V, dO, True, scale)))
    tensors = {"Q": Q, "K": K, "V": V}
    rng = np.random.default_rng(24)
    for _ in range(256):
        name = "QKV"[rng.integers(3)]
        flat = tensors[name].reshape(-1)
        idx = int(rng.integers(flat.size))
        old = flat[idx]
        eps = 1e-5 * max(1.0, abs(old))
        flat[idx] = old + eps
        lp = loss(oracle, Q, K, V, dO, True, scale)
        flat[idx] = old - eps
        lm = loss(oracle, Q, K, V, dO, True, scale)
        flat[idx] = old
        num = (lp - lm) / (2 * eps)
        ref = grads[name].reshape(-1)[idx]
        assert abs(num - ref) <= 2e-7 * np.abs(grads[name]).max() + 1e-7 * abs(ref), (name, idx, num, ref)


def torch_grads(Q, K, V, dO, causal, scale, use_sdpa=False):
    Qt, Kt, Vt = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    G = Q.shape[1] // K.shape[1]
    Kr, Vr = Kt.repeat_interleave(G, dim=1), Vt.repeat_interleave(G, dim=1)
    if use_sdpa:
        O = torch.nn.functional.scaled_dot_product_attention(Qt, Kr, Vr, is_causal=causal, scale=scale)
    else:
        s = scale * Qt @ Kr.transpose(-1, -2)
        if causal:
            S = Q.shape[2]
            s = s.masked_fill(torch.triu(torch.ones(S, S, dtype=torch.bool), 1), float("-inf"))
        O = torch.softmax(s, dim=-1) @ Vr
    (O * torch.tensor(dO)).sum().backward()
    return O.detach().numpy(), Qt.grad.numpy(), Kt.grad.numpy(), Vt.grad.numpy()


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(2, 4, 2, 40, 16), (1, 6, 6, 33, 8), (1, 8, 1, 24, 32)])
@pytest.mark.parametrize("use_sdpa", [False, True])
def test_against_torch_fp64_autograd(oracle, causal, shape, use_sdpa):
    B, Hq, Hkv, S, D = shape
    Q, K, V, dO = rnd((B, Hq, S, D), 30), rnd((B, Hkv, S, D), 31), rnd((B, Hkv, S, D), 32), rnd((B, Hq, S, D), 33)
    scale = 0.29
    O, _ = oracle.attn_fwd(Q, K, V, causal, scale)
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, causal, scale)
    Ot, dQt, dKt, dVt = torch_grads(Q, K, V, dO, causal, scale, use_sdpa)
    for a, b in ((O, Ot), (dQ, dQt), (dK, dKt), (dV, dVt)):
        np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-11)


def test_against_torch_on_tiny_benchmark_inputs(oracle):
    from paper_2606_10415_b200 import workloads
    cfg = workloads.CONFIGS["tiny"]
    Q, K, V, dO = (t.double().numpy() for t in workloads.make_inputs(cfg))
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, cfg.causal, cfg.scale)
    _, dQt, dKt, dVt = torch_grads(Q, K, V, dO, cfg.causal, cfg.scale)
    for a, b in ((dQ, dQt), (dK, dKt), (dV, dVt)):
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-10)


# ---------------------------------------------------------------- pieces

def test_softmax_backward_is_the_softmax_jacobian(oracle):
    """One query row, D=n and K = I/scale makes the scores equal to q, V = I makes O = p.
    Then dQ = J^T dO with J = diag(p) - p p^T, built here by brute force."""
    n = 7
    q = rnd((n,), 40)
    dO = rnd((n,), 41)
    Q = q.reshape(1, 1, 1, n).repeat(n, axis=2)       # every row the same query; use the last (sees all keys)
    K = np.eye(n).reshape(1, 1, n, n)
    V = np.eye(n).reshape(1, 1, n, n)
    dOm = np.zeros((1, 1, n, n))
    dOm[0, 0, n - 1] = dO
    dQ, _, _ = oracle.attn_bwd(Q, K, V, dOm, True, 1.0)
    p = np.exp(q) / np.exp(q).sum()
    J = np.diag(p) - np.outer(p, p)
    np.testing.assert_allclose(dQ[0, 0, n - 1], J @ dO, rtol=1e-12, atol=1e-14)
    assert np.all(dQ[0, 0, : n - 1] == 0.0)


@pytest.mark.parametrize("causal", [False, True])
def test_rowsum_dS_is_zero(oracle, causal):
    """If every key has a feature equal to 1, that feature's dQ is scale * rowsum(dS) = 0."""
    Q, K, V, dO = rnd((1, 2, 24, 8), 50), rnd((1, 1, 24, 8), 51), rnd((1, 1, 24, 8), 52), rnd((1, 2, 24, 8), 53)
    K[..., -1] = 1.0
    dQ, _, _ = oracle.attn_bwd(Q, K, V, dO, causal, 0.6)
    assert np.abs(dQ[..., -1]).max() <= 1e-12 * np.abs(dQ).max()


@pytest.mark.parametrize("causal", [False, True])
def test_dV_is_P_transpose_dO(oracle, causal):
    Q, K, V, dO = rnd((1, 4, 10, 4), 60), rnd((1, 2, 10, 4), 61), rnd((1, 2, 10, 4), 62), rnd((1, 4, 10, 4), 63)
    _, _, dV = oracle.attn_bwd(Q, K, V, dO, causal, 0.8)
    _, _, P = brute_forward(Q, K, V, causal, 0.8)
    ref = np.zeros_like(V)
    for g in range(2):
        for j in range(10):             # column walk: key j gathers from every query row
            for h in (2 * g, 2 * g + 1):
                for i in range(10):
                    ref[0, g, j] += P[0, h, i, j] * dO[0, h, i]
    np.testing.assert_allclose(dV, ref, rtol=1e-12, atol=1e-14)


def test_first_row_has_zero_dQ_and_adds_nothing_to_dK(oracle):
    Q, K, V, dO = (rnd((1, 1, 9, 4), s) for s in (70, 71, 72, 73))
    dQ, dK, _ = oracle.attn_bwd(Q, K, V, dO, True, 0.7)
    assert np.all(dQ[0, 0, 0] == 0.0)
    Q2, dO2 = Q.copy(), dO.copy()
    Q2[0, 0, 0] *= -5.0
    dO2[0, 0, 0] += 11.0
    _, dK2, _ = oracle.attn_bwd(Q2, K, V, dO2, True, 0.7)
    assert np.array_equal(dK, dK2)


def test_closed_form_single_key(oracle):
    Q, K, V, dO = (rnd((2, 3, 1, 5), s) for s in (80, 81, 82, 83))
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, True, 1.3)
    assert np.all(dQ == 0) and np.all(dK == 0)
    np.testing.assert_array_equal(dV, dO)


def test_closed_form_equal_keys(oracle):
    """All keys equal: P_ij = 1/(i+1), O_i = running mean of V, dV_j = sum_{i>=j} dO_i/(i+1), dQ = 0."""
    S, D = 11, 6
    k = rnd((D,), 90)
    K = np.broadcast_to(k, (1, 1, S, D)).copy()
    Q, V, dO = rnd((1, 1, S, D), 91), rnd((1, 1, S, D), 92), rnd((1, 1, S, D), 93)
    O, LSE = oracle.attn_fwd(Q, K, V, True, 0.9)
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, True, 0.9)
    mean = np.cumsum(V[0, 0], axis=0) / np.arange(1, S + 1)[:, None]
    np.testing.assert_allclose(O[0, 0], mean, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(LSE[0, 0], 0.9 * Q[0, 0] @ k + np.log(np.arange(1, S + 1)), rtol=1e-13)
    w = dO[0, 0] / np.arange(1, S + 1)[:, None]
    dV_ref = np.cumsum(w[::-1], axis=0)[::-1]
    np.testing.assert_allclose(dV[0, 0], dV_ref, rtol=1e-13, atol=1e-14)
    assert np.abs(dQ).max() < 1e-13
    # dK_j = scale * sum_i ds_ij Q_i with ds_ij = (dO_i.V_j - dO_i.O_i)/(i+1)
    dK_ref = np.zeros((S, D))
    for j in range(S):
        for i in range(j, S):
            dK_ref[j] += 0.9 * (dO[0, 0, i] @ V[0, 0, j] - dO[0, 0, i] @ mean[i]) / (i + 1) * Q[0, 0, i]
    np.testing.assert_allclose(dK[0, 0], dK_ref, rtol=1e-11, atol=1e-13)


def test_zero_dO_and_zero_V(oracle):
    Q, K, V, dO = rnd((1, 2, 8, 4), 100), rnd((1, 1, 8, 4), 101), rnd((1, 1, 8, 4), 102), rnd((1, 2, 8, 4), 103)
    for g in oracle.attn_bwd(Q, K, V, np.zeros_like(dO), True, 0.5):
        assert np.all(g == 0)
    dQ, dK, dV = oracle.attn_bwd(Q, K, np.zeros_like(V), dO, True, 0.5)
    assert np.all(dQ == 0) and np.all(dK == 0)
    _, _, P = brute_forward(Q, K, V, True, 0.5)
    ref = sum(np.einsum("ij,id->jd", P[0, h], dO[0, h]) for h in range(2))
    np.testing.assert_allclose(dV[0, 0], ref, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_linearity_shift_invariance_and_permutation(oracle, causal):
    Q, K, V, dO = rnd((2, 4, 12, 8), 110), rnd((2, 2, 12, 8), 111), rnd((2, 2, 12, 8), 112), rnd((2, 4, 12, 8), 113)
    base = oracle.attn_bwd(Q, K, V, dO, causal, 0.45)
    # linear in dO
    for a, b in zip(oracle.attn_bwd(Q, K, V, -2.5 * dO, causal, 0.45), base):
        np.testing.assert_allclose(a, -2.5 * b, rtol=1e-12, atol=1e-14)
    # one constant vector added to every key: scores shift per row, nothing changes
    c = rnd((8,), 114)
    for a, b in zip(oracle.attn_bwd(Q, K + c, V, dO, causal, 0.45), base):
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-11)
    # one constant vector added to every value: dP and delta shift together
    for a, b in zip(oracle.attn_bwd(Q, K, V + c, dO, causal, 0.45), base):
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-11)
    # swapping the two batches swaps the outputs
    sw = oracle.attn_bwd(Q[::-1], K[::-1], V[::-1], dO[::-1], causal, 0.45)
    for a, b in zip(sw, base):
        np.testing.assert_array_equal(a, b[::-1])
    # swapping the two kv groups (and their query heads) swaps the outputs
    hp = [2, 3, 0, 1]
    sw = oracle.attn_bwd(Q[:, hp], K[:, ::-1], V[:, ::-1], dO[:, hp], causal, 0.45)
    np.testing.assert_array_equal(sw[0], base[0][:, hp])
    np.testing.assert_array_equal(sw[1], base[1][:, ::-1])
    np.testing.assert_array_equal(sw[2], base[2][:, ::-1])


@pytest.mark.parametrize("G", [2, 5])
def test_gqa_equals_repeated_mha_summed_over_group(oracle, G):
    Hkv = 2
    Q, dO = rnd((1, Hkv * G, 10, 4), 120), rnd((1, Hkv * G, 10, 4), 121)
    K, V = rnd((1, Hkv, 10, 4), 122), rnd((1, Hkv, 10, 4), 123)
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, True, 0.5)
    Kr, Vr = np.repeat(K, G, axis=1), np.repeat(V, G, axis=1)
    dQm, dKm, dVm = oracle.attn_bwd(Q, Kr, Vr, dO, True, 0.5)
    np.testing.assert_allclose(dQ, dQm, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dK, dKm.reshape(1, Hkv, G, 10, 4).sum(2), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dV, dVm.reshape(1, Hkv, G, 10, 4).sum(2), rtol=1e-12, atol=1e-14)


def test_given_forward_state_mode_agrees_with_recompute_mode(oracle):
    Q, K, V, dO = rnd((1, 4, 20, 8), 130), rnd((1, 2, 20, 8), 131), rnd((1, 2, 20, 8), 132), rnd((1, 4, 20, 8), 133)
    O, LSE = oracle.attn_fwd(Q, K, V, True, 0.3)
    a = oracle.attn_bwd(Q, K, V, dO, True, 0.3)
    b = oracle.attn_bwd(Q, K, V, dO, True, 0.3, O=O, LSE=LSE)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=1e-11, atol=1e-13)
    # a perturbed O must change the result: the mode really consumes what it is given
    c = oracle.attn_bwd(Q, K, V, dO, True, 0.3, O=O + 0.1, LSE=LSE)
    assert np.abs(c[0] - a[0]).max() > 1e-4


def test_delta_is_rowsum(oracle):
    dO, O = rnd((3, 5, 7), 140), rnd((3, 5, 7), 141)
    np.testing.assert_allclose(oracle.delta(dO, O), (dO * O).sum(-1), rtol=1e-14)


def test_hand_worked_two_key_example(oracle):
    vals = {}
    for line in (GOLDEN / "two_key_worked_example.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            name, *nums = line.split()
            vals[name] = np.array([float(x) for x in nums])
    Q = np.array([1.0, 1.0]).reshape(1, 1, 2, 1)
    K = np.array([0.0, np.log(3.0)]).reshape(1, 1, 2, 1)
    V = np.array([1.0, 5.0]).reshape(1, 1, 2, 1)
    dO = np.ones((1, 1, 2, 1))
    O, LSE = oracle.attn_fwd(Q, K, V, True, 1.0)
    dQ, dK, dV = oracle.attn_bwd(Q, K, V, dO, True, 1.0)
    for name, got in (("O", O), ("LSE", LSE), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        np.testing.assert_allclose(got.reshape(-1), vals[name], rtol=1e-14, atol=1e-15, err_msg=name)


def test_thread_count_does_not_change_results(oracle):
    import os
    import subprocess
    import sys
    code = (
        "import numpy as np, oracle, hashlib;"
        "r=np.random.default_rng(5);"
        "Q=r.standard_normal((1,6,32,8));K=r.standard_normal((1,2,32,8));"
        "V=r.standard_normal((1,2,32,8));dO=r.standard_normal((1,6,32,8));"
        "g=oracle.attn_bwd(Q,K,V,dO,True,0.3);"
        "print(hashlib.sha256(b''.join(x.tobytes() for x in g)).hexdigest())"
    )
    root = str(Path(__file__).resolve().parent.parent)
    outs = set()
    for n in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=n, PYTHONPATH=root)
        outs.add(subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True,
                                check=True).stdout.strip())
    assert len(outs) == 1


# ------------------------------------------------------------------ GEMM oracle (C = A W^T)

def test_gemm_oracle_hand_worked_example(oracle):
    lines = [ln for ln in (Path(__file__).parent / "golden" / "gemm_worked_example.txt").read_text().splitlines()
             if ln and not ln.startswith("#")]
    rows = [list(map(float, ln.split())) for ln in lines]
    A, W, C = np.array(rows[0:2]), np.array(rows[2:4]), np.array(rows[4:6])
    assert np.array_equal(oracle.gemm_nt(A, W), C)


def test_gemm_oracle_against_triple_loop_and_special_cases(oracle):
    rng = np.random.default_rng(3)
    M, N, K = 5, 7, 11
    A, W = rng.standard_normal((M, K)), rng.standard_normal((N, K))
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            for k in range(K):
                brute[m, n] += A[m, k] * W[n, k]
    np.testing.assert_allclose(oracle.gemm_nt(A, W), brute, rtol=1e-13, atol=1e-13)
    # identity weight returns A; a weight row that selects one input column returns that column
    assert np.array_equal(oracle.gemm_nt(A, np.eye(K)), A)
    sel = np.zeros((1, K)); sel[0, 4] = 1.0
    assert np.array_equal(oracle.gemm_nt(A, sel)[:, 0], A[:, 4])
    # not symmetric in its arguments (a swapped or untransposed operand changes the shape or the values)
    assert oracle.gemm_nt(A, W).shape == (M, N) and oracle.gemm_nt(W, A).shape == (N, M)
    np.testing.assert_allclose(oracle.gemm_nt(W, A), oracle.gemm_nt(A, W).T, rtol=1e-13)
    # linear in each argument
    A2 = rng.standard_normal((M, K))
    np.testing.assert_allclose(oracle.gemm_nt(A + 2 * A2, W), oracle.gemm_nt(A, W) + 2 * oracle.gemm_nt(A2, W), rtol=1e-12)
    with pytest.raises(ValueError):
        oracle.gemm_nt(A, rng.standard_normal((N, K + 1)))


# ---------------------------------------------------------------- saved-P route (Section 4.1)

def test_probabilities_hand_worked_example_and_invariants(oracle):
    # the two-key worked example: row 0 sees key 0 only, row 1 has P = (1/4, 3/4)
    Q = np.array([1.0, 1.0]).reshape(1, 1, 2, 1)
    K = np.array([0.0, np.log(3.0)]).reshape(1, 1, 2, 1)
    P = oracle.attn_probabilities(Q, K, True, 1.0)
    np.testing.assert_allclose(P[0, 0], [[1.0, 0.0], [0.25, 0.75]], rtol=1e-15, atol=0)
    # unmasked, the first row sees both keys: (1/4, 3/4) as well, since Q_0 = Q_1
    P = oracle.attn_probabilities(Q, K, False, 1.0)
    np.testing.assert_allclose(P[0, 0], [[0.25, 0.75], [0.25, 0.75]], rtol=1e-15, atol=0)
    # random GQA case: rows sum to one, the mask is exact zeros, and P agrees with the C forward
    # oracle through both of its outputs: P V = O and P = exp(scale * s - LSE)
    Q, K, V = rnd((2, 4, 37, 8), 1), rnd((2, 2, 37, 8), 2), rnd((2, 2, 37, 8), 3)
    for causal in (False, True):
        P = oracle.attn_probabilities(Q, K, causal, 0.3)
        O, LSE = oracle.attn_fwd(Q, K, V, causal, 0.3)
        np.testing.assert_allclose(P.sum(-1), 1.0, rtol=1e-13)
        if causal:
            assert np.all(P[..., np.triu_indices(37, 1)[0], np.triu_indices(37, 1)[1]] == 0.0)
        for h in range(4):
            np.testing.assert_allclose(P[:, h] @ V[:, h // 2], O[:, h], rtol=1e-12, atol=1e-13)
            s = 0.3 * np.einsum("bqd,bkd->bqk", Q[:, h], K[:, h // 2])
            ref = np.exp(s - LSE[:, h][..., None])
            if causal:
                ref = np.tril(ref)
            np.testing.assert_allclose(P[:, h], ref, rtol=1e-12, atol=1e-15)


def test_backward_from_p_hand_worked_example(oracle):
    vals = {}
    for line in (GOLDEN / "two_key_worked_example.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            name, *nums = line.split()
            vals[name] = np.array([float(x) for x in nums])
    Q = np.array([1.0, 1.0]).reshape(1, 1, 2, 1)
    K = np.array([0.0, np.log(3.0)]).reshape(1, 1, 2, 1)
    V = np.array([1.0, 5.0]).reshape(1, 1, 2, 1)
    dO = np.ones((1, 1, 2, 1))
    P = np.array([[1.0, 0.0], [0.25, 0.75]]).reshape(1, 1, 2, 2)  # typed in, not computed
    dQ, dK, dV = oracle.attn_bwd_from_p(P, Q, K, V, dO, 1.0)
    for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        np.testing.assert_allclose(got.reshape(-1), vals[name], rtol=1e-14, atol=1e-15, err_msg=name)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_from_p_agrees_with_recompute_oracle_and_autograd(oracle, causal):
    # with the exact P the saved-P route must give the gradients of the recompute route (the C
    # oracle, pinned above by finite differences) and of torch's fp64 autograd through an explicit
    # softmax; asymmetric shapes and distinct scale catch transposed operands and a dropped scale
    B, Hq, Hkv, S, D, scale = 2, 6, 2, 29, 5, 0.37
    Q, K, V, dO = rnd((B, Hq, S, D), 11), rnd((B, Hkv, S, D), 12), rnd((B, Hkv, S, D), 13), rnd((B, Hq, S, D), 14)
    P = oracle.attn_probabilities(Q, K, causal, scale)
    got = oracle.attn_bwd_from_p(P, Q, K, V, dO, scale)
    ref = oracle.attn_bwd(Q, K, V, dO, causal, scale)
    for name, g, r in zip(("dQ", "dK", "dV"), got, ref):
        np.testing.assert_allclose(g, r, rtol=1e-10, atol=1e-12, err_msg=name)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    s = scale * torch.einsum("bhqd,bhkd->bhqk", tq, tk.repeat_interleave(Hq // Hkv, dim=1))
    if causal:
        s = s.masked_fill(torch.triu(torch.ones(S, S, dtype=torch.bool), 1), float("-inf"))
    o = torch.softmax(s, -1) @ tv.repeat_interleave(Hq // Hkv, dim=1)
    (o * torch.tensor(dO)).sum().backward()
    for name, g, r in zip(("dQ", "dK", "dV"), got, (tq.grad, tk.grad, tv.grad)):
        np.testing.assert_allclose(g, r.numpy(), rtol=1e-10, atol=1e-12, err_msg=name)

"""The parity gates themselves (CPU only): on oracle gradients of a benchmark-like input (upstream gradient
with standard deviation 1e-2, so every value is far below the absolute gate of 2e-2) the gates accept fp16
rounding of the exact result and reject a wrong element, a wrong 16-byte chunk and a wrong row -- the
failures the absolute gate cannot see."""
import numpy as np
import pytest

from paper_2606_10415_b200 import workloads
from parity_checks import MAX_ABS_TOL, check_tensor, error_measures


@pytest.fixture(scope="module")
def exact(oracle):
    cfg = workloads.custom(1, 2, 1, 512, 128, True, seed=5)
    Q, K, V, dO = (t.double().numpy() for t in workloads.make_inputs(cfg))
    return oracle.attn_bwd(Q, K, V, dO, True, cfg.scale)


def rounded(x):
    return x.astype(np.float16).astype(np.float64)


def test_fp16_rounding_of_the_exact_gradients_passes(exact):
    for name, ref in zip(("dQ", "dK", "dV"), exact):
        m = check_tensor(name, rounded(ref), ref, "rounded oracle")
        assert m["max_abs"] < 1e-3 * MAX_ABS_TOL  # the absolute gate is three orders away from these values


@pytest.mark.parametrize("damage", ["element", "chunk", "row", "sign_of_row", "scaled_head"])
def test_damaged_gradients_fail_a_scale_free_gate(exact, damage):
    ref = exact[0]                       # dQ [1, 2, 512, 128]
    g = rounded(ref)
    typical = np.sqrt(np.mean(ref ** 2))
    if damage == "element":              # one element of typical size off by its own magnitude
        g[0, 1, 300, 17] += typical
    elif damage == "chunk":              # eight neighbouring elements (16 bytes of fp16) replaced by zeros
        g[0, 1, 300, 24:32] = 0.0
    elif damage == "row":                # one row of 512 replaced by another row
        g[0, 0, 400] = g[0, 0, 401]
    elif damage == "sign_of_row":
        g[0, 1, 200] = -g[0, 1, 200]
    else:                                # a whole head off by 2 %: the Frobenius and element gates
        g[0, 1] *= 1.02
    m = error_measures(g, ref)
    assert m["max_abs"] < MAX_ABS_TOL, "the absolute gate alone would have let this through"
    with pytest.raises(AssertionError):
        check_tensor("dQ", g, ref, damage)

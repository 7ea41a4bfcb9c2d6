"""Seeded synthetic inputs for the attention hot path.

This module holds no attention arithmetic: it only names the benchmark
configurations and draws their input tensors.  Both the CUDA tests/benchmark and
the CPU oracle's tests take their inputs from here so that the two sides see the
same bits.

Recipe (every configuration, seed 0 unless stated): a CPU ``torch.Generator`` is
seeded, then Q, K, V, dO are drawn in that order as fp32 ``randn`` of their
final ``[B, H, S, D]`` shapes, multiplied by the configuration's standard
deviation, and rounded to fp16.  The tensors stand in for the activations of the
decoder layers the paper trains (LLaMA-2-7B, Baichuan2-13B, Qwen2.5-32B,
LLaMA-2-70B attention shapes); the paper's token stream and weights are not
available, and the throughput of a dense attention kernel does not depend on
the values.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class AttnConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    S: int
    D: int
    causal: bool
    qkv_std: float
    do_std: float
    seed: int = 0

    @property
    def scale(self) -> float:
        return float(self.D) ** -0.5

    @property
    def flops(self) -> float:
        """FLOPs the metric counts: five contractions, half of them under a causal mask."""
        full = 10.0 * self.B * self.Hq * float(self.S) ** 2 * self.D
        return full / 2 if self.causal else full


def _cfg(name, B, Hq, Hkv, S, D, qkv_std, do_std, causal=True):
    return AttnConfig(name, B, Hq, Hkv, S, D, causal, qkv_std, do_std)


_STD128 = 128.0 ** -0.25

CONFIGS = {
    "tiny": _cfg("tiny", 1, 2, 2, 128, 64, 1.0, 1.0),
    "llama2_7b": _cfg("llama2_7b", 1, 32, 32, 4096, 128, _STD128, 1e-2),
    "baichuan2_13b": _cfg("baichuan2_13b", 1, 40, 40, 4096, 128, _STD128, 1e-2),
    "qwen25_32b_gqa": _cfg("qwen25_32b_gqa", 1, 40, 8, 4096, 128, _STD128, 1e-2),
    "llama2_70b_gqa": _cfg("llama2_70b_gqa", 2, 64, 8, 4096, 128, _STD128, 1e-2),
}


# Further workloads: the other sequence lengths and the layer shape the paper's Attention-BP
# measurement uses (Section 6.6: a LLaMA-2-7B layer at S = 1024, 2048, 4096 and a Qwen2.5-32B
# layer at S = 2048), an unmasked variant and a ragged length.  Same value distributions and seed.
EXTRA_CONFIGS = {
    "llama2_7b_s1024": _cfg("llama2_7b_s1024", 1, 32, 32, 1024, 128, _STD128, 1e-2),
    "llama2_7b_s2048": _cfg("llama2_7b_s2048", 1, 32, 32, 2048, 128, _STD128, 1e-2),
    "qwen25_32b_gqa_s2048": _cfg("qwen25_32b_gqa_s2048", 1, 40, 8, 2048, 128, _STD128, 1e-2),
    "llama2_7b_full_mask_off": _cfg("llama2_7b_full_mask_off", 1, 32, 32, 4096, 128, _STD128, 1e-2, causal=False),
    # a length that is not a whole number of 128-row tiles (the last tile holds 56 rows)
    "llama2_7b_s3000_ragged": _cfg("llama2_7b_s3000_ragged", 1, 32, 32, 3000, 128, _STD128, 1e-2),
}
ALL_CONFIGS = {**CONFIGS, **EXTRA_CONFIGS}


def custom(B, Hq, Hkv, S, D, causal=True, qkv_std=None, do_std=1e-2, seed=0, name="custom"):
    if qkv_std is None:
        qkv_std = float(D) ** -0.25
    return AttnConfig(name, B, Hq, Hkv, S, D, bool(causal), float(qkv_std), float(do_std), seed)


def make_inputs(cfg: AttnConfig):
    """Return fp16 CPU tensors (Q, K, V, dO), each contiguous ``[B, H, S, D]``."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(cfg.seed)
    qshape = (cfg.B, cfg.Hq, cfg.S, cfg.D)
    kshape = (cfg.B, cfg.Hkv, cfg.S, cfg.D)
    Q = (torch.randn(qshape, generator=gen, dtype=torch.float32) * cfg.qkv_std).half()
    K = (torch.randn(kshape, generator=gen, dtype=torch.float32) * cfg.qkv_std).half()
    V = (torch.randn(kshape, generator=gen, dtype=torch.float32) * cfg.qkv_std).half()
    dO = (torch.randn(qshape, generator=gen, dtype=torch.float32) * cfg.do_std).half()
    return Q, K, V, dO

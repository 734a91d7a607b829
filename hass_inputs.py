"""Seeded synthetic inputs for the fused LM-head + Top-K distillation path.

This module only draws random tensors and rounds them to bfloat16. It holds none
of the method's arithmetic (no logits, softmax, top-K or loss) and is the single
piece of code shared by the CPU oracle's tests and the CUDA path's tests/bench.

The tensors stand in for the *shapes* of the draft-training inputs of the paper's
four target models (LLaMA2-Chat 7B/13B, LLaMA3-Instruct 8B/70B; Section 4.1):
target features H_t, draft features H_d and the frozen, shared LM head W
(Section 2: the draft model reuses the target LLM's LM head). The real features
and weights are not available, so values are Gaussian:

    H_t ~ N(0, 1)            [N, d]
    H_d = H_t + 0.5 * eps    eps ~ N(0, 1) iid, one draw per aligning step
    W   ~ N(0, sigma_w^2)    [V, d]

Everything is drawn in fp32 from one CPU torch generator in the order
H_t, eps_1 .. eps_n, W and rounded to bf16 (round-to-nearest-even). The rounded
bit patterns are *the* inputs for both the oracle and the GPU.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    N: int
    d: int
    V: int
    K: int
    steps: int = 1          # aligning steps: independent H_d draws sharing H_t and W
    sigma_w: float = 0.02
    seed: int = 0
    k_sweep: tuple = ()     # extra K values timed/tested on the same tensors


# The five configurations: a tiny case the oracle finishes instantly, and the
# four draft-head shapes (hidden size d and vocabulary V of each target model).
WORKLOADS = {
    "tiny": Workload("tiny", N=64, d=256, V=1024, K=10),
    "l2-7b": Workload("l2-7b", N=8192, d=4096, V=32000, K=10),
    "l2-13b": Workload("l2-13b", N=8192, d=5120, V=32000, K=10, steps=3),
    "l3-8b": Workload("l3-8b", N=8192, d=4096, V=128256, K=10),
    "l3-70b": Workload("l3-70b", N=4096, d=8192, V=128256, K=10, sigma_w=0.015,
                       k_sweep=(1, 10, 64)),
}


@dataclass
class Inputs:
    """bf16 tensors (CPU, contiguous) for one workload."""
    wl: Workload
    H_t: torch.Tensor                      # [N, d] bf16
    H_d: List[torch.Tensor] = field(default_factory=list)   # steps x [N, d] bf16
    W: torch.Tensor = None                 # [V, d] bf16


def make_inputs(wl: Workload) -> Inputs:
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed)
    H_t32 = torch.randn(wl.N, wl.d, generator=g, dtype=torch.float32)
    H_d = []
    for _ in range(wl.steps):
        eps = torch.randn(wl.N, wl.d, generator=g, dtype=torch.float32)
        H_d.append((H_t32 + 0.5 * eps).to(torch.bfloat16).contiguous())
        del eps
    W = torch.empty(wl.V, wl.d, dtype=torch.float32)
    W.normal_(0.0, wl.sigma_w, generator=g)
    return Inputs(wl=wl, H_t=H_t32.to(torch.bfloat16).contiguous(), H_d=H_d,
                  W=W.to(torch.bfloat16).contiguous())


def make_custom(N: int, d: int, V: int, K: int, seed: int = 0, sigma_w: float = 0.02,
                steps: int = 1, name: str = "custom") -> Inputs:
    return make_inputs(Workload(name, N=N, d=d, V=V, K=K, steps=steps, sigma_w=sigma_w, seed=seed))


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a bf16 CPU tensor as a uint16 numpy array (no copy of values)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu" and t.is_contiguous()
    return t.view(torch.int16).numpy().view(np.uint16)


def sample_rows(N: int, n_rows: int, seed: int = 0) -> np.ndarray:
    """Row subset used when the oracle cannot afford all N rows: the first quarter of the
    sample from the head of the batch, a quarter from the tail, the rest drawn without
    replacement with the given seed. Rows are independent, so per-row results are exact."""
    if n_rows >= N:
        return np.arange(N, dtype=np.int64)
    q = max(n_rows // 4, 1)
    head = np.arange(0, q, dtype=np.int64)
    tail = np.arange(N - q, N, dtype=np.int64)
    rng = np.random.default_rng(seed)
    middle_pool = np.arange(q, N - q, dtype=np.int64)
    mid = rng.choice(middle_pool, size=n_rows - 2 * q, replace=False)
    return np.unique(np.concatenate([head, mid, tail]))


# ---- inputs of the HCA attention of the draft layer (Section 3.2) --------------------------------
@dataclass(frozen=True)
class HcaWorkload:
    name: str
    B: int            # sequences per batch
    T: int            # tokens per sequence
    H: int            # query heads
    Hkv: int          # key/value heads (H a multiple of it)
    m: int            # earlier draft passes whose features replace the target's (aligning step m + 1)
    D: int = 128      # head dimension
    seed: int = 0


# Shapes of the one-layer draft model, which copies its target's attention geometry: a tiny
# case, a ragged mid-size case, and LLaMA3-8B / LLaMA2-7B geometry at 4 x 2048 tokens (the
# 8192-token batch of the LM-head workloads) in the third aligning step.
HCA_WORKLOADS = {
    "hca-tiny": HcaWorkload("hca-tiny", B=2, T=80, H=2, Hkv=1, m=2),
    "hca-mid": HcaWorkload("hca-mid", B=2, T=333, H=4, Hkv=2, m=3),
    "hca-l3-8b": HcaWorkload("hca-l3-8b", B=4, T=2048, H=32, Hkv=8, m=2),
    "hca-l2-7b": HcaWorkload("hca-l2-7b", B=4, T=2048, H=32, Hkv=32, m=2),
}


@dataclass
class HcaInputs:
    """bf16 tensors (CPU, contiguous): Q [B, T, H, D]; K_t, V_t and every K_d[i], V_d[i] [B, T, Hkv, D]."""
    wl: HcaWorkload
    Q: torch.Tensor
    K_t: torch.Tensor
    V_t: torch.Tensor
    K_d: List[torch.Tensor] = field(default_factory=list)
    V_d: List[torch.Tensor] = field(default_factory=list)


def make_hca_inputs(wl: HcaWorkload) -> HcaInputs:
    """Projected queries, keys and values stand in for q_proj/k_proj/v_proj of real features:
    Q, K_t, V_t ~ N(0, 1); the keys/values of draft pass i are the target's plus 0.5 * N(0, 1),
    the same closeness the LM-head workloads give draft features. Draw order: Q, K_t, V_t,
    then (K_d[i], V_d[i]) for i = 0 .. m-1; everything rounded to bf16."""
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed)
    shape_q = (wl.B, wl.T, wl.H, wl.D)
    shape_kv = (wl.B, wl.T, wl.Hkv, wl.D)
    Q = torch.randn(shape_q, generator=g, dtype=torch.float32)
    K32 = torch.randn(shape_kv, generator=g, dtype=torch.float32)
    V32 = torch.randn(shape_kv, generator=g, dtype=torch.float32)
    K_d, V_d = [], []
    for _ in range(wl.m):
        K_d.append((K32 + 0.5 * torch.randn(shape_kv, generator=g, dtype=torch.float32)).to(torch.bfloat16).contiguous())
        V_d.append((V32 + 0.5 * torch.randn(shape_kv, generator=g, dtype=torch.float32)).to(torch.bfloat16).contiguous())
    return HcaInputs(wl=wl, Q=Q.to(torch.bfloat16).contiguous(), K_t=K32.to(torch.bfloat16).contiguous(),
                     V_t=V32.to(torch.bfloat16).contiguous(), K_d=K_d, V_d=V_d)

"""The five benchmark/parity workloads and their seeded synthetic tensors.

Shapes follow DeepSeek-style MoE-FFN layers; config 4 is the module shape the
paper evaluates (sequence 4096 x microbatch 2 = 8192 tokens, hidden 7168,
intermediate 2048, top-8; Section 5.2) placed on one device with 256 experts.
All tensors come from `workloads.gen`; nothing here computes the layer.
"""
from __future__ import annotations

import dataclasses
import math

import torch

from . import gen


@dataclasses.dataclass(frozen=True)
class MoeConfig:
    name: str
    T: int          # tokens
    d: int          # hidden size
    E: int          # routed experts
    k: int          # routed experts per token
    S: int          # shared experts (every token, weight 1)
    F: int          # expert intermediate size
    renorm: bool    # renormalise the k routing weights to sum to 1
    seed: int
    bwd: bool       # the config also runs the backward pass
    zipf_s: float = 0.0   # > 0: bias the router so expert popularity follows Zipf(s)
    n_dead: int = 0       # experts forced to receive no token

    @property
    def Ep(self) -> int:
        return self.E + self.S

    @property
    def kp(self) -> int:
        return self.k + self.S

    @property
    def R(self) -> int:
        return self.T * self.kp

    def flops_fwd(self) -> float:
        return 6.0 * self.R * self.d * self.F

    def weight_bytes(self) -> float:
        return 3.0 * self.Ep * self.d * self.F * 2


CONFIGS = [
    MoeConfig("cfg0_tiny_fwd_bwd", T=256, d=256, E=8, k=2, S=0, F=128, renorm=True, seed=0, bwd=True),
    MoeConfig("cfg1_v2lite_fwd", T=4096, d=2048, E=64, k=6, S=2, F=1408, renorm=False, seed=1, bwd=False),
    MoeConfig("cfg2_v3_fwd", T=4096, d=7168, E=256, k=8, S=1, F=2048, renorm=True, seed=2, bwd=False),
    MoeConfig("cfg3_zipf_fwd", T=16384, d=4096, E=128, k=8, S=0, F=1536, renorm=True, seed=3, bwd=False,
              zipf_s=1.2, n_dead=4),
    MoeConfig("cfg4_train_fwd_bwd", T=8192, d=7168, E=256, k=8, S=0, F=2048, renorm=True, seed=4, bwd=True),
]


def small_variant(cfg: MoeConfig, T: int, d: int, F: int, E: int | None = None) -> MoeConfig:
    """Same routing recipe at reduced sizes (used by CPU tests and ncu-sized captures)."""
    return dataclasses.replace(cfg, name=cfg.name + f"_small_T{T}_d{d}_F{F}", T=T, d=d, F=F,
                               E=cfg.E if E is None else E)


def make_x(cfg: MoeConfig, device="cpu") -> torch.Tensor:
    return gen.normal_bf16(cfg.seed, gen.TID_X, (cfg.T, cfg.d), 1.0, device)


def make_dout(cfg: MoeConfig, device="cpu") -> torch.Tensor:
    return gen.normal_bf16(cfg.seed, gen.TID_DOUT, (cfg.T, cfg.d), 1.0, device)


def w_gate_up_slab(cfg: MoeConfig, e: int, device="cpu") -> torch.Tensor:
    """Expert e of W_gate_up, shape [2F, d]: rows 0..F-1 gate, F..2F-1 up; d contiguous."""
    n = 2 * cfg.F * cfg.d
    return gen.normal_bf16(cfg.seed, gen.TID_W_GATE_UP, (2 * cfg.F, cfg.d), cfg.d ** -0.5, device, start=e * n)


def w_down_slab(cfg: MoeConfig, e: int, device="cpu") -> torch.Tensor:
    """Expert e of W_down, shape [d, F]; F contiguous."""
    n = cfg.d * cfg.F
    return gen.normal_bf16(cfg.seed, gen.TID_W_DOWN, (cfg.d, cfg.F), cfg.d ** -0.5, device, start=e * n)


def make_w_gate_up(cfg: MoeConfig, device="cpu") -> torch.Tensor:
    return gen.normal_bf16(cfg.seed, gen.TID_W_GATE_UP, (cfg.Ep, 2 * cfg.F, cfg.d), cfg.d ** -0.5, device)


def make_w_down(cfg: MoeConfig, device="cpu") -> torch.Tensor:
    return gen.normal_bf16(cfg.seed, gen.TID_W_DOWN, (cfg.Ep, cfg.d, cfg.F), cfg.d ** -0.5, device)


def router_bias(cfg: MoeConfig) -> torch.Tensor:
    """fp32 [E] additive logit bias (zeros unless the config skews expert popularity)."""
    bias = torch.zeros(cfg.E, dtype=torch.float32)
    if cfg.zipf_s > 0:
        rank = gen.permutation(cfg.seed, gen.TID_PERM, cfg.E)  # rank[e] = popularity rank of expert e
        vals = [-cfg.zipf_s * math.log(int(r) + 1.0) for r in rank.tolist()]
        bias = torch.tensor(vals, dtype=torch.float64).to(torch.float32)
        if cfg.n_dead:
            bias[rank >= cfg.E - cfg.n_dead] = -1.0e4
    return bias


def make_logits(cfg: MoeConfig, x: torch.Tensor) -> torch.Tensor:
    """Router logits fp32 [T, E] = x . W_r (+ bias); W_r ~ N(0, std 0.02) in fp32.

    The product's rounding depends on the device that runs it; callers hand the SAME
    array to every implementation under comparison.
    """
    w_r = gen.normal_f32(cfg.seed, gen.TID_W_ROUTER, 0, cfg.d * cfg.E, 0.02, x.device).reshape(cfg.d, cfg.E)
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        logits = x.to(torch.float32) @ w_r
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev
    return (logits + router_bias(cfg).to(x.device)).contiguous()


def make_inputs(cfg: MoeConfig, device="cpu", weights: bool = True) -> dict:
    x = make_x(cfg, device)
    out = {"x": x, "logits": make_logits(cfg, x)}
    if weights:
        out["W_gate_up"] = make_w_gate_up(cfg, device)
        out["W_down"] = make_w_down(cfg, device)
    if cfg.bwd:
        out["dout"] = make_dout(cfg, device)
    return out

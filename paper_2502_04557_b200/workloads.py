"""Seeded synthetic workloads (input tensors only).

This module draws random tensors with the shapes and value distributions of the five
benchmark configurations.  It contains none of the verification arithmetic and imports
neither the CUDA library nor the CPU oracle; both are fed from here.

All draws come from one ``torch.Generator`` seeded with ``20250204 + 1000*index + sweep``;
values are drawn in float32 and rounded once to the configuration's element type.  The
realised tensors are the inputs (a CPU and a CUDA generator give different streams).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch

BASE_SEED = 20250204


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    index: int
    B: int
    K: int
    V: int
    d: int
    h: int
    dtype: torch.dtype
    logits: str                  # "normal" | "zipf"
    q_std: float = 3.0           # draft logits ~ N(0, q_std^2) ("normal")
    noise_std: float = 1.0       # target = rho * draft + noise_std * N(0,1)
    rho: float = 1.0
    threshold: float = 0.5
    reject_fraction: Optional[float] = None   # choose b2 so roughly this share of scores < 0.5


CONFIGS: Dict[str, Config] = {
    "tiny": Config("tiny", 0, B=1, K=4, V=1000, d=256, h=64, dtype=torch.float32,
                   logits="normal", q_std=2.0, noise_std=0.5),
    "gpt2": Config("gpt2", 1, B=32, K=8, V=50257, d=768, h=256, dtype=torch.bfloat16,
                   logits="normal", q_std=3.0, noise_std=1.0),
    "llama2": Config("llama2", 2, B=128, K=8, V=32000, d=2048, h=512, dtype=torch.bfloat16,
                     logits="zipf", noise_std=0.75),
    "llama3": Config("llama3", 3, B=256, K=16, V=128256, d=2048, h=512, dtype=torch.bfloat16,
                     logits="normal", q_std=3.0, rho=0.9, noise_std=3.0 * math.sqrt(1.0 - 0.81)),
    "sequential": Config("sequential", 4, B=1024, K=1, V=128256, d=4096, h=1024,
                         dtype=torch.bfloat16, logits="normal", q_std=3.0, rho=0.9,
                         noise_std=3.0 * math.sqrt(1.0 - 0.81), reject_fraction=0.2),
}
SEQUENTIAL_BATCHES = (1, 8, 64, 256, 1024)


@dataclasses.dataclass
class Workload:
    cfg: Config
    B: int
    K: int
    Kp: int
    V: int
    ldv: int
    hidden: torch.Tensor        # [B,K,d]
    W1: torch.Tensor            # [h,d]
    b1: torch.Tensor            # [h] f32
    W2: torch.Tensor            # [h]
    b2: torch.Tensor            # [1] f32
    q_logits: torch.Tensor      # [B,K,ldv]
    p_logits: torch.Tensor      # [B,Kp,ldv]
    draft_tokens: torch.Tensor  # [B,K] int32
    uniforms: torch.Tensor      # [B,K+1] f32: accept tests, then the correction draw
    u_replace: torch.Tensor     # [B] f32: replacement draw of the SPRINTER step
    seed: int

    def logits_bytes(self) -> int:
        es = self.q_logits.element_size()
        return (self.B * self.K * 2) * self.V * es


def _gumbel(shape, gen, device):
    u = torch.rand(shape, generator=gen, device=device, dtype=torch.float32)
    u = u.clamp_(min=1e-20, max=1.0 - 6e-8)
    return -torch.log(-torch.log(u))


def make(name: str, device="cpu", B: Optional[int] = None, sweep: int = 0, bonus_row: bool = True,
         ldv: Optional[int] = None, seq_slice: int = 8) -> Workload:
    """Draws the tensors of one configuration.

    B overrides the batch (the sequential configuration is swept over B); ``ldv`` pads the
    logits rows (padding columns hold large values that must be ignored); ``bonus_row``
    adds the (K+1)-th target row used when every draft token is accepted."""
    cfg = CONFIGS[name]
    B = cfg.B if B is None else B
    K, V, d, h = cfg.K, cfg.V, cfg.d, cfg.h
    Kp = K + 1 if bonus_row else K
    ldv = V if ldv is None else ldv
    assert ldv >= V
    seed = BASE_SEED + 1000 * cfg.index + sweep
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)

    def randn(*shape):
        return torch.randn(shape, generator=gen, device=dev, dtype=torch.float32)

    hidden = randn(B, K, d).to(cfg.dtype)
    W1 = (randn(h, d) / math.sqrt(d)).to(cfg.dtype)
    b1 = randn(h) / math.sqrt(d)
    W2 = (randn(h) / math.sqrt(h)).to(cfg.dtype)
    b2 = torch.zeros(1, dtype=torch.float32, device=dev)
    if cfg.reject_fraction is not None:
        # z - b2 = sum_j W2_j relu(g_j), g_j ~ N(0,1) nearly independent: a normal with the
        # moments below; shift so the requested share of z lands below 0 (score < 1/2).
        w2 = W2.float()
        mean = float(w2.sum()) / math.sqrt(2.0 * math.pi)
        std = math.sqrt(float((w2 * w2).sum()) * (0.5 - 0.5 / math.pi))
        quant = torch.distributions.Normal(0.0, 1.0).icdf(torch.tensor(cfg.reject_fraction)).item()
        b2 = torch.tensor([-(mean + quant * std)], dtype=torch.float32, device=dev)

    q_logits = torch.empty((B, K, ldv), dtype=cfg.dtype, device=dev)
    p_logits = torch.empty((B, Kp, ldv), dtype=cfg.dtype, device=dev)
    draft_tokens = torch.empty((B, K), dtype=torch.int32, device=dev)
    if ldv > V:
        q_logits[..., V:] = 60.0
        p_logits[..., V:] = -60.0
    zipf_base = None
    if cfg.logits == "zipf":
        perm = torch.randperm(V, generator=gen, device=dev)
        zipf_base = torch.empty(V, dtype=torch.float32, device=dev)
        zipf_base[perm] = -1.1 * torch.log(torch.arange(1, V + 1, device=dev, dtype=torch.float32))

    for b0 in range(0, B, seq_slice):
        nb = min(seq_slice, B - b0)
        if cfg.logits == "zipf":
            lq = zipf_base + _gumbel((nb, Kp, V), gen, dev)
        else:
            lq = randn(nb, Kp, V) * cfg.q_std
        lp = cfg.rho * lq + cfg.noise_std * randn(nb, Kp, V)
        lq_r = lq[:, :K].to(cfg.dtype)
        q_logits[b0:b0 + nb, :, :V] = lq_r
        p_logits[b0:b0 + nb, :, :V] = lp.to(cfg.dtype)
        # draft tokens distributed as softmax(draft logits): arg-max of logits + Gumbel noise
        g = _gumbel((nb, K, V), gen, dev)
        draft_tokens[b0:b0 + nb] = (lq_r.float() + g).argmax(-1).to(torch.int32)
        del lq, lp, lq_r, g

    uniforms = torch.rand((B, K + 1), generator=gen, device=dev, dtype=torch.float32)
    u_replace = torch.rand((B,), generator=gen, device=dev, dtype=torch.float32)
    return Workload(cfg, B, K, Kp, V, ldv, hidden, W1, b1, W2, b2, q_logits, p_logits, draft_tokens,
                    uniforms, u_replace, seed)


def shard_batch(B: int, rank: int, world: int):
    """Contiguous split of B sequences over `world` ranks: (first, count) of rank `rank`."""
    base, rem = divmod(B, world)
    first = rank * base + min(rank, rem)
    return first, base + (1 if rank < rem else 0)

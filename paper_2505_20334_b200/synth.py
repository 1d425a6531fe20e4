"""Seeded synthetic inputs shaped like the paper's workloads (Section 5.1: Llama-3 / Mistral class
GQA models, 4K-64K prompts, budgets 128-2048, a window of a few lookahead queries).

This module only draws random tensors and plants structure in them (outlier channels, an
attention sink, needle keys, a correlated key sequence). It contains none of the eviction
method's arithmetic and is the one module that both the CUDA tests/benchmark and the CPU oracle's
tests may share. The paper's own evaluation data (LongBench, Needle-in-a-Haystack, RULER) and
model weights are not reproduced; these tensors stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch

BASE_SEED = 20250520


@dataclasses.dataclass(frozen=True)
class EvictConfig:
    """One eviction workload: geometry, budgets and the recipe that fills K."""

    name: str
    cfg_id: int
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prompt_len: int
    window_len: int
    pool_kernel: int
    budgets: Tuple[int, ...]
    recipe: str  # "plain" | "outlier" | "ar1"
    n_needles: int = 0
    sink: bool = False
    planted_one: bool = False

    @property
    def keep_tail(self) -> int:
        return self.window_len

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def units(self) -> int:
        return self.n_layers * self.batch * self.n_kv_heads

    @property
    def rows(self) -> int:
        return self.group * self.window_len

    def scaled(self, **kw) -> "EvictConfig":
        """A copy with some fields replaced (used for oracle-sized test cases)."""
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[int, EvictConfig] = {
    1: EvictConfig("tiny-gqa4-L1024", 1, 1, 1, 4, 1, 128, 1024, 8, 7, (128,), "plain",
                   planted_one=True),
    2: EvictConfig("llama3-8b-L4096", 2, 32, 1, 32, 8, 128, 4096, 16, 7, (128, 512, 1024),
                   "outlier", sink=True),
    3: EvictConfig("llama3-8b-b4-L32768", 3, 32, 4, 32, 8, 128, 32768, 32, 7,
                   (128, 256, 512, 1024, 2048), "outlier", n_needles=16, sink=True),
    4: EvictConfig("mistral-7b-b8-L16384", 4, 32, 8, 32, 8, 128, 16384, 16, 5, (512,), "ar1"),
    5: EvictConfig("llama3-70b-L65536", 5, 80, 1, 64, 8, 128, 65536, 32, 7, (256, 2048),
                   "outlier", sink=True),
}

N_OUTLIER_CHANNELS = 4
OUTLIER_GAIN = 8.0
AR1_RHO = 0.9


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _ar1(eps: torch.Tensor, rho: float) -> torch.Tensor:
    """AR(1) along dim -2 with unit stationary variance: x_j = rho*x_{j-1} + sqrt(1-rho^2)*eps_j,
    evaluated as a 256-tap truncated filter by shift doubling (rho^256 ~ 2e-12)."""
    x = eps * math.sqrt(1.0 - rho * rho)
    s = 1
    while s < 256 and s < x.shape[-2]:
        shifted = torch.zeros_like(x)
        shifted[..., s:, :] = x[..., :-s, :]
        x = x + (rho ** s) * shifted
        s *= 2
    return x


def make_inputs(cfg: EvictConfig, device="cpu", with_v: bool = True) -> Dict[str, object]:
    """Draws Q [NL,Bt,Hq,W,D], K and V [NL,Bt,Hkv,L,D] in bf16 on `device`, layer by layer.

    Returns {'q','k','v','planted'}: `planted` maps 'sink' / 'needles' / 'one' to int64 tensors of
    planted key positions per unit ([NL,Bt,Hkv] or [NL,Bt,Hkv,n]). Values depend on the device
    type (CPU and CUDA generators differ) but are reproducible on each.
    """
    NL, Bt, Hq, Hkv = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    D, L, W, G = cfg.head_dim, cfg.prompt_len, cfg.window_len, cfg.group
    Ls = L - cfg.keep_tail
    seed = (BASE_SEED + cfg.cfg_id) * 1000
    dev = torch.device(device)
    q = torch.empty((NL, Bt, Hq, W, D), dtype=torch.bfloat16, device=dev)
    k = torch.empty((NL, Bt, Hkv, L, D), dtype=torch.bfloat16, device=dev)
    v = torch.empty((NL, Bt, Hkv, L, D), dtype=torch.bfloat16, device=dev) if with_v else None
    planted: Dict[str, torch.Tensor] = {}
    if cfg.sink:
        planted["sink"] = torch.zeros((NL, Bt, Hkv), dtype=torch.int64)
    if cfg.n_needles:
        planted["needles"] = torch.zeros((NL, Bt, Hkv, cfg.n_needles), dtype=torch.int64)
    if cfg.planted_one:
        planted["one"] = torch.zeros((NL, Bt, Hkv), dtype=torch.int64)
    sigma_hat = 1.0
    if cfg.recipe == "outlier":
        sigma_hat = math.sqrt((D - N_OUTLIER_CHANNELS + N_OUTLIER_CHANNELS * OUTLIER_GAIN ** 2) / D)

    for layer in range(NL):
        gq = _gen(dev, seed + 10 * layer + 1)
        gk = _gen(dev, seed + 10 * layer + 2)
        gv = _gen(dev, seed + 10 * layer + 3)
        gp = _gen("cpu", seed + 10 * layer + 4)  # positions / channels / scales: always on CPU
        ql = torch.randn((Bt, Hq, W, D), generator=gq, device=dev, dtype=torch.float32)
        ql = ql.to(torch.bfloat16)
        q[layer] = ql
        kl = torch.randn((Bt, Hkv, L, D), generator=gk, device=dev, dtype=torch.float32)
        if cfg.recipe == "outlier":
            for h in range(Hkv):
                ch = torch.randperm(D, generator=gp)[:N_OUTLIER_CHANNELS].to(dev)
                kl[:, h, :, ch] *= OUTLIER_GAIN
        elif cfg.recipe == "ar1":
            kl = _ar1(kl, AR1_RHO)
            scale = (0.5 + 1.5 * torch.rand((Hkv,), generator=gp)).to(dev)
            kl = kl * scale.view(1, Hkv, 1, 1)
        # planted keys: beta * mean query of the unit, so that the mean logit over the unit's
        # G*W rows equals tau (with the 1/sqrt(D) scale).
        if cfg.sink or cfg.n_needles or cfg.planted_one:
            qbar = ql.float().view(Bt, Hkv, G * W, D).mean(dim=2)  # [Bt,Hkv,D]
            beta = math.sqrt(D) / (qbar * qbar).sum(-1, keepdim=True)  # tau = 1
            unit_key = qbar * beta
            if cfg.planted_one:
                pos = torch.randint(0, Ls, (Bt, Hkv), generator=gp)
                planted["one"][layer] = pos
                for b in range(Bt):
                    for h in range(Hkv):
                        kl[b, h, int(pos[b, h])] = 8.0 * unit_key[b, h]
            if cfg.sink:
                kl[:, :, 0, :] = (8.0 * sigma_hat) * unit_key
            if cfg.n_needles:
                for b in range(Bt):
                    for h in range(Hkv):
                        pos = (torch.randperm(Ls - 1, generator=gp)[:cfg.n_needles] + 1)
                        planted["needles"][layer, b, h] = pos
                        kl[b, h, pos.to(dev)] = (6.0 * sigma_hat) * unit_key[b, h]
        k[layer] = kl.to(torch.bfloat16)
        del kl
        if with_v:
            v[layer] = torch.randn((Bt, Hkv, L, D), generator=gv, device=dev,
                                   dtype=torch.float32).to(torch.bfloat16)
    return {"q": q, "k": k, "v": v, "planted": planted}


def unit_slices(cfg: EvictConfig, inputs: Dict[str, object], u: int):
    """Host copies of one unit's tensors, shaped as a 1-layer/1-batch/1-KV-head problem:
    q [1,1,G,W,D], k and v [1,1,1,L,D]."""
    Hkv, Bt, G = cfg.n_kv_heads, cfg.batch, cfg.group
    h = u % Hkv
    b = (u // Hkv) % Bt
    layer = u // (Hkv * Bt)
    q = inputs["q"][layer, b, h * G:(h + 1) * G].cpu()[None, None]
    k = inputs["k"][layer, b, h].cpu()[None, None, None]
    v = inputs["v"]
    v = None if v is None else v[layer, b, h].cpu()[None, None, None]
    return q, k, v


def sample_units(cfg: EvictConfig, n_random: int, seed: int = 7) -> List[int]:
    """First and last layer's units of batch 0 plus `n_random` seeded random units, sorted unique."""
    Hkv, Bt, NL = cfg.n_kv_heads, cfg.batch, cfg.n_layers
    first = list(range(Hkv))
    last = [((NL - 1) * Bt) * Hkv + h for h in range(Hkv)]
    g = torch.Generator().manual_seed(BASE_SEED + seed)
    rnd = torch.randint(0, cfg.units, (n_random,), generator=g).tolist()
    return sorted(set(first + last + rnd))

"""Seeded synthetic inputs for the split-FFN library and for its CPU oracle.

This module only draws random tensors; it holds none of the method's
arithmetic (no activation, score, selection, factorisation or FFN code) and is
the one module both the CUDA side and the oracle side may consume.

The tensors stand in for the paper's BERT / OPT feed-forward layers (Section 5)
which are not available offline.  The long-tailed neuron-norm distribution of
Figure 1 is imitated by *planting* heavy hitters: a seed-chosen set of neurons
gets +1.0 on its first-layer bias and a 10x larger second-layer row.

Recipe (per layer): generator seed = 20240104 + 1000*config + layer; draws, in
this fixed order and in float32: W1 [d,m], (W1u [d,m] for SwiGLU), W2 [m,d],
the planting permutation, X_cal [T_cal,d], X_fwd [T,d].  Weights ~ N(0, 0.02^2)
(0.02 is the standard deviation), tokens ~ N(0,1), biases zero before
planting.  Each tensor is cast once to the storage dtype; the cast tensors are
the ground-truth inputs of both sides.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch

BASE_SEED = 20240104


@dataclass(frozen=True)
class FFNConfig:
    name: str
    cid: int
    d: int
    m: int
    k: int
    r: int
    act: str            # "gelu_erf" | "gelu_tanh" | "swiglu"
    dtype: str          # "f32" | "bf16"
    layers: int
    t_cal: int
    t_fwd: tuple
    n_plant: int
    note: str = ""

    @property
    def n_in(self) -> int:
        return 2 if self.act == "swiglu" else 1

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


def _ceil_frac(frac_percent: int, m: int) -> int:
    return -(-frac_percent * m // 100)


CONFIGS = {
    1: FFNConfig("single_gelu_fp32", 1, 256, 1024, 32, 64, "gelu_erf", "f32", 1, 512, (128,), 32),
    2: FFNConfig("bert_base_prefill", 2, 768, 3072, 154, 192, "gelu_erf", "bf16", 12, 4096, (4096,), 154),
    3: FFNConfig("gpt2_medium_decode", 3, 1024, 4096, 205, 256, "gelu_erf", "bf16", 24, 4096, (1, 4, 16, 64), 205),
    4: FFNConfig("llama2_7b_swiglu", 4, 4096, 11008, 551, 1024, "swiglu", "bf16", 32, 8192, (2048, 1, 8, 32), 551),
    5: FFNConfig("opt_13b_gelu", 5, 5120, 20480, 1024, 512, "gelu_erf", "bf16", 40, 65536, (1, 32, 4096), 1024),
}

# config 5 sweep axes (heavy fraction in percent, light rank, tokens)
CFG5_HEAVY_PERCENT = (1, 5, 10)
CFG5_RANKS = (256, 512, 1280)
CFG5_TOKENS = (1, 32, 4096)


def cfg5_point(heavy_percent: int, r: int) -> FFNConfig:
    base = CONFIGS[5]
    k = _ceil_frac(heavy_percent, base.m)
    return FFNConfig(f"opt_13b_h{heavy_percent}_r{r}", 5, base.d, base.m, k, r, base.act, base.dtype,
                     base.layers, base.t_cal, base.t_fwd, k)


def custom_config(d, m, k, r, act="gelu_erf", dtype="bf16", n_plant=None, t_cal=256, cid=9) -> FFNConfig:
    return FFNConfig(f"custom_d{d}_m{m}_k{k}_r{r}_{act}_{dtype}", cid, d, m, k, r, act, dtype, 1, t_cal, (0,),
                     k if n_plant is None else n_plant)


def layer_seed(cfg: FFNConfig, layer: int) -> int:
    return BASE_SEED + 1000 * cfg.cid + layer


@dataclass
class LayerInputs:
    cfg: FFNConfig
    layer: int
    W1: torch.Tensor
    W1u: Optional[torch.Tensor]
    b1: Optional[torch.Tensor]
    W2: torch.Tensor
    b2: Optional[torch.Tensor]
    planted: torch.Tensor          # int64 indices, ascending
    gen: torch.Generator = field(repr=False, default=None)

    def tokens(self, T: int) -> torch.Tensor:
        """Next T tokens ~ N(0,1) from this layer's generator, in the storage dtype."""
        x = torch.randn(T, self.cfg.d, generator=self.gen, dtype=torch.float32, device=self.W1.device)
        return x.to(self.cfg.torch_dtype)


def make_layer(cfg: FFNConfig, layer: int = 0, device: str = "cpu", plant: bool = True,
               extra_seed: int = 0) -> LayerInputs:
    """Draw one FFN layer.  device='cuda' uses the CUDA generator (values differ
    from the CPU stream; same distribution), for shapes too large to ship."""
    gen = torch.Generator(device=device)
    gen.manual_seed(layer_seed(cfg, layer) + 7919 * extra_seed)
    d, m = cfg.d, cfg.m
    kw = dict(generator=gen, dtype=torch.float32, device=device)
    W1 = torch.randn(d, m, **kw) * 0.02
    W1u = torch.randn(d, m, **kw) * 0.02 if cfg.act == "swiglu" else None
    W2 = torch.randn(m, d, **kw) * 0.02
    perm = torch.randperm(m, generator=gen, device=device)
    n_plant = cfg.n_plant if plant else 0
    planted = torch.sort(perm[:n_plant]).values
    if cfg.act == "swiglu":
        b1 = None
        b2 = None
    else:
        b1 = torch.zeros(m, dtype=torch.float32, device=device)
        b2 = torch.zeros(d, dtype=torch.float32, device=device)
        if n_plant:
            b1[planted] += 1.0
    if n_plant:
        W2[planted, :] *= 10.0
    dt = cfg.torch_dtype
    cast = lambda t: None if t is None else t.to(dt).contiguous()
    return LayerInputs(cfg, layer, cast(W1), cast(W1u), cast(b1), cast(W2), cast(b2), planted, gen)


def random_scores(m: int, seed: int, ties: int = 0, device: str = "cpu") -> torch.Tensor:
    """Non-negative float32 keys for selection tests; ties>0 draws from only
    that many distinct values so that equal keys are common."""
    gen = torch.Generator(device=device)
    gen.manual_seed(BASE_SEED + 31 * seed + m)
    if ties > 0:
        levels = torch.rand(ties, generator=gen, dtype=torch.float32, device=device)
        pick = torch.randint(0, ties, (m,), generator=gen, device=device)
        return levels[pick].contiguous()
    return (torch.rand(m, generator=gen, dtype=torch.float32, device=device) ** 4 * 1e3).contiguous()

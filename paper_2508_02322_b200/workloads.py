"""Seeded synthetic MoE layers and calibration tokens.

This module only *draws inputs*: layer shapes of the model families the paper
evaluates, random weights and hidden states with a stated distribution.  It
holds none of the method's arithmetic and is the one module both the CUDA
path's callers and the CPU oracle's callers may share.

Every tensor is drawn from its own `torch.Generator` seeded with
(seed, layer_id, tensor_id), in float32, transformed, then cast to the storage
dtype.  The oracle is handed the same storage values widened to float64.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    d_model: int
    n_routed: int
    top_k: int
    d_ff_routed: int
    d_ff_shared: Tuple[int, ...] = ()
    shared_gate_sigmoid: bool = False
    n_tokens: int = 512
    dtype: str = "bf16"                 # "bf16" | "f32"
    x_dist: str = "normal"              # "normal" | "normal_rms1" | "student_t4_outliers"
    router_bias_std: float = 0.0
    weight_std: float = 0.02
    n_layers: int = 1
    norm_topk: bool = True

    @property
    def d_ff(self) -> List[int]:
        return [self.d_ff_routed] * self.n_routed + list(self.d_ff_shared)

    @property
    def n_shared(self) -> int:
        return len(self.d_ff_shared)

    @property
    def n_micro_experts(self) -> int:
        return sum(self.d_ff)

    @property
    def pairs(self) -> int:
        """Token-expert pairs per layer: T*k routed plus T per shared expert."""
        return self.n_tokens * (self.top_k + self.n_shared)

    @property
    def gate_up_flop(self) -> float:
        """4 * d_model * sum_e M_e * d_ff_e with exact routed counts (sum_e M_e = T*k)."""
        return 4.0 * self.d_model * self.n_tokens * (
            self.top_k * self.d_ff_routed + sum(self.d_ff_shared))


CONFIGS: Dict[str, LayerConfig] = {
    # Tiny single layer, fp32.
    "tiny_fp32": LayerConfig("tiny_fp32", 256, 8, 2, 512, (), False, 512, "f32", "normal"),
    # Mixtral-8x7B-shaped.
    "mixtral_8x7b": LayerConfig("mixtral_8x7b", 4096, 8, 2, 14336, (), False, 4096, "bf16", "normal_rms1"),
    # Qwen1.5-MoE-A2.7B-shaped: skewed expert load through a router bias.
    "qwen15_moe_a27b": LayerConfig("qwen15_moe_a27b", 2048, 60, 4, 1408, (5632,), True, 16384, "bf16",
                                   "normal", router_bias_std=0.5),
    # DeepSeek-MoE-16B-shaped: heavy-tailed hidden states with outlier channels.
    "deepseek_moe_16b": LayerConfig("deepseek_moe_16b", 2048, 64, 6, 1408, (1408, 1408), False, 32768,
                                    "bf16", "student_t4_outliers"),
    # Qwen2-57B-A14B-shaped: 28 layers, 128 x 2048 calibration tokens per layer.
    "qwen2_57b_a14b": LayerConfig("qwen2_57b_a14b", 3584, 64, 8, 2560, (20480,), True, 262144, "bf16",
                                  "normal_rms1", n_layers=28),
}

N_OUTLIER_CHANNELS = 8
OUTLIER_SCALE = 20.0

_TENSOR_IDS = {"x": 1, "w_router": 2, "router_bias": 3, "w_shared_gate": 4,
               "w_gate": 5, "w_up": 6, "w_down": 7, "outliers": 8}


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


def _gen(device, seed: int, layer_id: int, tensor: str, sub: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(((seed * 1000003 + layer_id) * 1009 + _TENSOR_IDS[tensor]) * 4099 + sub)
    return g


def _randn(shape, device, g, chunk_rows: int = 1 << 16) -> torch.Tensor:
    return torch.randn(shape, device=device, dtype=torch.float32, generator=g)


def make_tokens(cfg: LayerConfig, seed: int = 0, layer_id: int = 0, device="cpu",
                n_tokens: Optional[int] = None) -> torch.Tensor:
    """Calibration hidden states X [T, d_model] in the storage dtype."""
    T = cfg.n_tokens if n_tokens is None else n_tokens
    dt = torch_dtype(cfg.dtype)
    out = torch.empty((T, cfg.d_model), device=device, dtype=dt)
    g = _gen(device, seed, layer_id, "x")
    outl = None
    if cfg.x_dist == "student_t4_outliers":
        go = _gen("cpu", seed, layer_id, "outliers")
        outl = torch.randperm(cfg.d_model, generator=go)[:N_OUTLIER_CHANNELS].to(device)
    step = 1 << 15
    for r0 in range(0, T, step):
        r1 = min(T, r0 + step)
        x = _randn((r1 - r0, cfg.d_model), device, g)
        if cfg.x_dist == "normal_rms1":
            x = x / x.pow(2).mean(dim=1, keepdim=True).sqrt()
        elif cfg.x_dist == "student_t4_outliers":
            chi = torch.zeros_like(x)
            for _ in range(4):
                chi += _randn(x.shape, device, g).pow(2)
            x = x / (chi / 4.0).sqrt()
            x[:, outl] *= OUTLIER_SCALE
        out[r0:r1] = x.to(dt)
    return out


def outlier_channels(cfg: LayerConfig, seed: int = 0, layer_id: int = 0) -> List[int]:
    if cfg.x_dist != "student_t4_outliers":
        return []
    go = _gen("cpu", seed, layer_id, "outliers")
    return torch.randperm(cfg.d_model, generator=go)[:N_OUTLIER_CHANNELS].tolist()


def make_layer(cfg: LayerConfig, seed: int = 0, layer_id: int = 0, device="cpu",
               down_layout: str = "hf") -> Dict[str, object]:
    """Random weights of one MoE layer.

    Returns a dict with w_router [E_r,d], router_bias [E_r] fp32 or None,
    w_shared_gate [E_s,d] or None, and lists w_gate / w_up ([f_e,d]) and
    w_down ([d,f_e] for down_layout "hf", [f_e,d] for "me_major").
    """
    dt = torch_dtype(cfg.dtype)
    d = cfg.d_model
    std = cfg.weight_std
    L: Dict[str, object] = {"cfg": cfg, "down_layout": down_layout}
    L["w_router"] = (_randn((cfg.n_routed, d), device, _gen(device, seed, layer_id, "w_router")) * std).to(dt)
    if cfg.router_bias_std > 0:
        L["router_bias"] = _randn((cfg.n_routed,), device, _gen(device, seed, layer_id, "router_bias")) \
            * cfg.router_bias_std
    else:
        L["router_bias"] = None
    if cfg.n_shared and cfg.shared_gate_sigmoid:
        L["w_shared_gate"] = (_randn((cfg.n_shared, d), device,
                                     _gen(device, seed, layer_id, "w_shared_gate")) * std).to(dt)
    else:
        L["w_shared_gate"] = None
    wg, wu, wd = [], [], []
    for e, f in enumerate(cfg.d_ff):
        wg.append((_randn((f, d), device, _gen(device, seed, layer_id, "w_gate", e)) * std).to(dt))
        wu.append((_randn((f, d), device, _gen(device, seed, layer_id, "w_up", e)) * std).to(dt))
        shape = (d, f) if down_layout == "hf" else (f, d)
        wd.append((_randn(shape, device, _gen(device, seed, layer_id, "w_down", e)) * std).to(dt))
    L["w_gate"], L["w_up"], L["w_down"] = wg, wu, wd
    return L


def scaled(cfg: LayerConfig, **kw) -> LayerConfig:
    """A copy of a config with some fields replaced (smaller token counts, ...)."""
    return replace(cfg, **kw)

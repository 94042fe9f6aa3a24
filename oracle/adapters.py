"""Hands the synthetic workloads to the oracle: widens stored tensors (bf16 / fp32, any device)
to float64 numpy arrays and arranges a generated layer as an `OracleLayer`.

TEST INFRASTRUCTURE ONLY, like the rest of this package.  No arithmetic of the method lives here:
every value is converted exactly (float64 holds every bf16 and fp32 value), and the only layout
change is the transpose that brings a `W_down` stored one micro-expert per row into the paper's
[d_model, d_ff] form (Eq. 3: micro-expert i owns column i of W_down).
"""
from __future__ import annotations

import numpy as np

from .camera_oracle import OracleLayer

__all__ = ["f64", "to_oracle_layer"]


def f64(t):
    """A tensor-like object (anything with detach / cpu / double / numpy) as a float64 array; None stays None."""
    return None if t is None else t.detach().cpu().double().numpy()


def to_oracle_layer(L) -> OracleLayer:
    """`L` is the dict a workload generator returns: cfg, down_layout, w_router, router_bias,
    w_shared_gate and the per-expert lists w_gate, w_up, w_down."""
    cfg = L["cfg"]
    if L["down_layout"] == "hf":
        w_down = [f64(w) for w in L["w_down"]]
    else:
        w_down = [np.ascontiguousarray(f64(w).T) for w in L["w_down"]]
    return OracleLayer(
        w_router=f64(L["w_router"]), top_k=cfg.top_k,
        w_gate=[f64(w) for w in L["w_gate"]], w_up=[f64(w) for w in L["w_up"]], w_down=w_down,
        router_bias=f64(L["router_bias"]), norm_topk=cfg.norm_topk, n_shared=cfg.n_shared,
        w_shared_gate=f64(L["w_shared_gate"]))

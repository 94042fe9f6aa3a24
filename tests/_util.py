"""Test helpers: turn a generated layer (torch tensors in storage dtype) into
the oracle's float64 layer, and small random layers for the pins."""
import numpy as np
import torch

from oracle import OracleLayer


def f64(t):
    return None if t is None else t.detach().to("cpu").to(torch.float64).numpy()


def to_oracle_layer(L) -> OracleLayer:
    """`L` is the dict returned by workloads.make_layer."""
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


def random_layer(rng, d=6, d_ff=(3, 3, 3), n_shared=0, top_k=2, shared_gate=False, bias=False,
                 norm_topk=True, scale=1.0) -> OracleLayer:
    n_routed = len(d_ff) - n_shared
    return OracleLayer(
        w_router=rng.standard_normal((max(n_routed, 0), d)),
        top_k=top_k,
        w_gate=[rng.standard_normal((f, d)) * scale for f in d_ff],
        w_up=[rng.standard_normal((f, d)) * scale for f in d_ff],
        w_down=[rng.standard_normal((d, f)) * scale for f in d_ff],
        router_bias=rng.standard_normal(n_routed) if bias else None,
        norm_topk=norm_topk, n_shared=n_shared,
        w_shared_gate=rng.standard_normal((n_shared, d)) if (shared_gate and n_shared) else None)

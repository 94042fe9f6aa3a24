"""Test helpers: the oracle's adapters for generated layers (re-exported) and small random layers for the pins."""
import numpy as np

from oracle import OracleLayer, f64, to_oracle_layer  # noqa: F401


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

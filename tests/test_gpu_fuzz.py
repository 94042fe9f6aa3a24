"""Seeded random layer shapes through every kernel variant, against the oracle: odd expert counts, d_ff values
that leave partial channel tiles, token counts around the tile sizes, gated / ungated shared experts, biased routers."""
import numpy as np
import pytest
import torch

import oracle as O
from _gpu import run_and_compare
from _util import f64, to_oracle_layer

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
FUZZ_FLOOR_RESCUES = 4


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def random_cfg(r):
    from paper_2508_02322_b200 import workloads as W
    n_routed = int(r.integers(0, 40))
    n_shared = int(r.integers(0 if n_routed else 1, 3))
    top_k = int(r.integers(1, min(n_routed, 8) + 1)) if n_routed else 1
    return W.LayerConfig(
        name="fuzz", d_model=int(r.choice([64, 128, 192, 320, 512])), n_routed=n_routed, top_k=top_k,
        d_ff_routed=int(r.choice([8, 64, 72, 128, 200, 264, 384])),
        d_ff_shared=tuple(int(r.choice([16, 128, 136, 448])) for _ in range(n_shared)),
        shared_gate_sigmoid=bool(r.integers(0, 2)) and n_shared > 0, n_tokens=int(r.choice([1, 31, 257, 600, 1500, 4100])),
        dtype="bf16", x_dist=str(r.choice(["normal", "normal_rms1", "student_t4_outliers"])),
        router_bias_std=float(r.choice([0.0, 0.5, 2.0])), weight_std=0.05, norm_topk=bool(r.integers(0, 2)))


@pytest.mark.parametrize("seed", range(14))
def test_random_layers(P, seed):
    from paper_2508_02322_b200 import workloads as W
    r = np.random.default_rng(1000 + seed)
    cfg = random_cfg(r)
    L = W.make_layer(cfg, seed=seed, device=DEV, down_layout=str(r.choice(["hf", "me_major"])))
    X = W.make_tokens(cfg, seed=seed, device=DEV)
    alpha = float(r.choice([0.0, 0.5, 0.95, 1.0]))
    kernel = ["umma", "umma_pair", "simt", "auto"][seed % 4]
    # random shapes starve experts (one or two tokens, nearly cancelled dot products): up to FUZZ_FLOOR_RESCUES scores
    # per compared array may miss 1e-3 of their own value while a million times below the layer's largest
    out, _ = run_and_compare(P, L, X, alpha=alpha, force_simt=kernel == "simt",
                              cta_pair={"umma": False, "umma_pair": True}.get(kernel), max_floor_rescues=FUZZ_FLOOR_RESCUES)
    # selections on these scores, and the weights they select
    E = out["energy"]
    ratio = float(r.choice([0.0, 0.3, 0.7]))
    keep = P.camera_select_prune(E, ratio)
    assert np.array_equal(keep.cpu().numpy(), O.select_prune(E.cpu().numpy(), ratio))
    layer = P.Layer.from_workload(L)
    off = P.expert_offsets_tensor(layer)
    sub, counts = P.camera_sub_index(keep, off, [1])
    lists, ref_counts = O.sub_index_lists(keep.cpu().numpy(), off.cpu().numpy(), [1])
    assert np.array_equal(counts.cpu().numpy(), ref_counts)
    outw = P.camera_compact_weights(layer, sub, counts, 1)
    ref = O.slice_layer(to_oracle_layer(L), lists)
    for e in range(layer.n_experts):
        m = len(lists[e])
        assert np.array_equal(f64(outw["w_gate"][e][:m]), ref.w_gate[e])
        got = f64(outw["w_down"][e][:, :m]) if L["down_layout"] == "hf" else f64(outw["w_down"][e][:m]).T
        assert np.array_equal(got, ref.w_down[e])
    # the layer output, where the forward path takes the layout
    if L["down_layout"] == "hf":
        from test_gpu_forward import assert_output_close, oracle_forward
        y, routing = P.camera_layer_forward(layer, X, want_routing=True, **[dict(), dict(cta_pair=False), dict(cta_pair=True), dict(token_rows=True)][(seed // 2) % 4])
        gi, gw = routing
        ref_y = oracle_forward(to_oracle_layer(L), f64(X), (gi.cpu().numpy().astype(np.int64), gw.cpu().numpy().astype(np.float64)))
        assert_output_close(f"fuzz {seed} layer output", y.cpu().numpy(), ref_y)
        # scores and output from one pass, then the retained micro-experts' output from the h it leaves behind
        from _gpu import assert_close
        T = int(X.shape[0])
        ws = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, T), DEV)
        E1, y1 = P.camera_score_forward_layer(layer, X, alpha, routing_in=routing, workspace=ws)
        assert P.camera_read_status(ws) == 0
        rt = (gi.cpu().numpy().astype(np.int64), gw.cpu().numpy().astype(np.float64))
        p2, pinf, w2 = O.camera_components(to_oracle_layer(L), f64(X), routing=rt)
        assert_close(f"fuzz {seed} one-pass energy", E1.cpu().numpy(), O.energy(p2, pinf, w2, float(np.float32(alpha))),
                     max_floor_rescues=FUZZ_FLOOR_RESCUES)
        assert_output_close(f"fuzz {seed} one-pass output", y1.cpu().numpy(), ref_y)
        y_hat = P.camera_pruned_output(layer, P.camera_mask_down_columns(layer, keep), T, ws)
        ref_hat = oracle_forward(ref, f64(X), (gi.cpu().numpy().astype(np.int64), gw.cpu().numpy().astype(np.float64)))
        assert_output_close(f"fuzz {seed} pruned output", y_hat.cpu().numpy(), ref_hat)

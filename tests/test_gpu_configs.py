"""GPU parity at the full sizes of the five workload configs, in the launch configuration the
benchmark times.

The float64 oracle cannot score 10^5 micro-experts over 10^5 tokens in a test, so it scores a seeded
sample of micro-experts exactly: micro-experts do not interact once the routing is fixed, hence the
scores of a layer that keeps only the sampled rows of W_gate / W_up and columns of W_down are the
scores of those micro-experts in the full layer.  The oracle routes *all* tokens, and the selections
are checked bit for bit on the full GPU score vector.
"""
import numpy as np
import pytest
import torch

import oracle as O
from _gpu import W_TOL, assert_close, check_routing
from _util import f64

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def W():
    from paper_2508_02322_b200 import workloads
    return workloads


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def sampled_layer(L, channels):
    """The oracle's view of the layer restricted to `channels` = {expert: channel indices}.  Experts
    outside the sample keep one (never visited) row so that expert numbering is unchanged."""
    cfg = L["cfg"]
    wg, wu, wd = [], [], []
    for e in range(len(L["w_gate"])):
        ch = torch.as_tensor(channels.get(e, [0]), device=L["w_gate"][e].device)
        wg.append(f64(L["w_gate"][e][ch]))
        wu.append(f64(L["w_up"][e][ch]))
        wd.append(f64(L["w_down"][e][:, ch]) if L["down_layout"] == "hf" else f64(L["w_down"][e][ch]).T.copy())
    return O.OracleLayer(w_router=f64(L["w_router"]), top_k=cfg.top_k, w_gate=wg, w_up=wu, w_down=wd,
                         router_bias=f64(L["router_bias"]), norm_topk=cfg.norm_topk, n_shared=cfg.n_shared,
                         w_shared_gate=f64(L["w_shared_gate"]))


def pick_channels(cfg, experts, per_expert, seed):
    r = np.random.default_rng(seed)
    out = {}
    for e in experts:
        f = cfg.d_ff[e]
        must = {0, 127, 128, f - 1}
        out[e] = sorted(must | set(r.choice(f, size=per_expert, replace=False).tolist()))
    return out


def run_config(P, name, n_routed_sampled, per_expert, alpha, prune_ratios, bit_scheme, inject_oracle_routing):
    cfg = W().CONFIGS[name]
    L = W().make_layer(cfg, seed=0, device=DEV)
    X = W().make_tokens(cfg, seed=0, device=DEV)
    T = cfg.n_tokens
    layer = P.Layer.from_workload(L)
    # the first call scores all tokens in one pass (what the benchmark's step times); the call under the oracle's
    # routing below takes the default, which walks more than 65536 tokens in batches
    ws = P.alloc_workspace(P.camera_score_workspace_bytes_single_pass(layer, T), DEV)
    out = P.camera_score_layer(layer, X, alpha, details=True, workspace=ws, single_pass=True)
    assert P.camera_read_status(ws) == 0
    counts = out["expert_token_counts"].cpu().numpy()
    gi = out["topk_idx"].cpu().numpy().astype(np.int64)
    gw = out["topk_w"].cpu().numpy().astype(np.float64)
    assert np.array_equal(counts[:cfg.n_routed], np.bincount(gi.reshape(-1), minlength=cfg.n_routed))
    assert (counts[cfg.n_routed:] == T).all()

    # the sample: most and least loaded routed expert, first, last, a few seeded ones; every shared expert
    r = np.random.default_rng(1)
    routed = {0, cfg.n_routed - 1, int(counts[:cfg.n_routed].argmax()), int(counts[:cfg.n_routed].argmin())}
    routed |= set(r.choice(cfg.n_routed, size=min(n_routed_sampled, cfg.n_routed), replace=False).tolist())
    experts = sorted(routed) + list(range(cfg.n_routed, cfg.n_routed + cfg.n_shared))
    channels = pick_channels(cfg, experts, per_expert, seed=2)
    red = sampled_layer(L, channels)
    Xd = f64(X)

    # routing of all tokens against the oracle (in blocks of tokens, to bound the oracle's memory)
    flips = 0
    idx_o, w_o = [], []
    for t0 in range(0, T, 65536):
        t1 = min(T, t0 + 65536)
        flips += check_routing(red, Xd[t0:t1], out["topk_idx"][t0:t1], out["topk_w"][t0:t1])
        if inject_oracle_routing:
            i, w = O.top_and_norm(O.router_probs(red, Xd[t0:t1]), red.top_k, red.norm_topk)
            idx_o.append(i); w_o.append(w)
    assert flips <= 2 + T // 5000, f"{flips} near-tie tokens routed differently"

    off_full = np.concatenate([[0], np.cumsum(cfg.d_ff)])
    off_red = O.me_offsets(red)
    full_index = np.concatenate([off_full[e] + np.asarray(channels[e]) for e in experts])
    red_index = np.concatenate([off_red[e] + np.arange(len(channels[e])) for e in experts])
    red_channels = {e: list(range(len(channels[e]))) for e in experts}

    def compare(o, routing, tag):
        p2, pinf, w2 = O.camera_components(red, Xd, channels=red_channels, routing=routing)
        assert_close(f"{name} omega2 {tag}", o["omega2"].cpu().numpy()[full_index], w2[red_index])
        assert_close(f"{name} phi2 {tag}", o["phi2"].cpu().numpy()[full_index], p2[red_index])
        assert_close(f"{name} phi_inf_sq {tag}", o["phi_inf_sq"].cpu().numpy()[full_index], pinf[red_index])
        E = O.energy(p2, pinf, w2, float(np.float32(alpha)))
        assert_close(f"{name} energy {tag}", o["energy"].cpu().numpy()[full_index], E[red_index])

    compare(out, (gi, gw), "(GPU routing)")
    if cfg.n_shared:
        assert_close(f"{name} shared_w", out["shared_w"].cpu().numpy().astype(np.float64).T, O.shared_coeff(red, Xd),
                     rel=W_TOL)

    # the selections, bit for bit, on the full GPU score vector
    E_gpu = out["energy"]
    E_np = E_gpu.cpu().numpy()
    assert np.isfinite(E_np).all() and (E_np >= 0).all()
    for ratio in prune_ratios:
        keep = P.camera_select_prune(E_gpu, ratio)
        assert np.array_equal(keep.cpu().numpy(), O.select_prune(E_np, ratio)), f"{name} mask at {ratio}"
    ratios, bits = bit_scheme
    got = P.camera_alloc_bits(E_gpu, ratios, bits)
    assert np.array_equal(got.cpu().numpy(), O.alloc_bits(E_np, ratios, bits)[0]), f"{name} bit allocation"

    if inject_oracle_routing:
        idx_o = np.concatenate(idx_o); w32 = np.concatenate(w_o).astype(np.float32)
        out2 = P.camera_score_layer(layer, X, alpha, details=True, workspace=ws,
                                    routing_in=(torch.from_numpy(idx_o.astype(np.int32)), torch.from_numpy(w32)))
        assert P.camera_read_status(ws) == 0
        compare(out2, (idx_o, w32.astype(np.float64)), "(oracle routing)")
    return out, counts


def test_mixtral_8x7b_shape(P):
    run_config(P, "mixtral_8x7b", 8, 12, 0.95, (0.2, 0.4, 0.6), ([0.2, 0.6, 0.2], [3, 2, 1]), True)


def test_qwen15_moe_shape_skewed_load(P):
    _, counts = run_config(P, "qwen15_moe_a27b", 8, 12, 0.95, (0.2, 0.4, 0.6), ([0.2, 0.6, 0.2], [3, 2, 1]), True)
    routed = counts[:60]
    assert routed.max() > 4 * max(1, routed.min())     # the router bias really skews the load


def test_deepseek_moe_shape_heavy_tails_bit_budget(P):
    # CAMERA-Q at b = 2, r = 0.2: widths (3, 2, 1), 2 bits of payload + 0.25 of group overhead
    out, _ = run_config(P, "deepseek_moe_16b", 8, 12, 1.0, (0.2, 0.6), ([0.2, 0.6, 0.2], [3, 2, 1]), True)
    bits = P.camera_alloc_bits(out["energy"], [0.2, 0.6, 0.2], [3, 2, 1])
    assert abs(float(bits.float().mean()) - 2.0) < 1e-4      # floor(0.2 n) top and bottom differ by at most one
    assert abs(O.average_bits([3, 2, 1], [0.2, 0.6, 0.2], 128, 32) - 2.25) < 1e-12


def test_qwen2_57b_shape_one_full_layer(P):
    # the configuration the benchmark's headline is quoted on: sampled like the others, and scored a second time
    # under the oracle's routing of all 262144 tokens, so that no token is left out of the comparison
    run_config(P, "qwen2_57b_a14b", 8, 12, 0.95, (0.2, 0.4, 0.6), ([0.2, 0.6, 0.2], [3, 2, 1]), True)


def test_qwen15_moe_shape_layer_output_on_sampled_tokens(P):
    """The layer output at a full-size config: the oracle computes Eq. 1-2 for a sample of tokens under the GPU's
    routing of those tokens (every expert's full weights take part)."""
    from test_gpu_forward import assert_output_close, oracle_forward
    from _util import to_oracle_layer
    cfg = W().CONFIGS["qwen15_moe_a27b"]
    L = W().make_layer(cfg, seed=0, device=DEV)
    X = W().make_tokens(cfg, seed=0, device=DEV)
    y, (gi, gw) = P.camera_layer_forward(P.Layer.from_workload(L), X, want_routing=True)
    tok = np.sort(np.random.default_rng(3).choice(cfg.n_tokens, size=48, replace=False))
    tok[0], tok[-1] = 0, cfg.n_tokens - 1
    ol = to_oracle_layer(L)
    ref = oracle_forward(ol, f64(X[torch.from_numpy(tok).to(DEV)]),
                         (gi.cpu().numpy().astype(np.int64)[tok], gw.cpu().numpy().astype(np.float64)[tok]))
    assert_output_close("qwen15 layer output", y.cpu().numpy()[tok], ref)


def test_qwen2_57b_shape_layer_output_on_sampled_tokens(P):
    """The same at the Qwen2-57B-A14B shape, on one 65536-token batch (the size the benchmark's forward leg uses)."""
    from test_gpu_forward import assert_output_close, oracle_forward
    from _util import to_oracle_layer
    cfg = W().scaled(W().CONFIGS["qwen2_57b_a14b"], n_tokens=65536)
    L = W().make_layer(cfg, seed=0, device=DEV)
    X = W().make_tokens(cfg, seed=0, device=DEV)
    y, (gi, gw) = P.camera_layer_forward(P.Layer.from_workload(L), X, want_routing=True)
    tok = np.sort(np.random.default_rng(4).choice(cfg.n_tokens, size=24, replace=False))
    tok[0], tok[-1] = 0, cfg.n_tokens - 1
    ref = oracle_forward(to_oracle_layer(L), f64(X[torch.from_numpy(tok).to(DEV)]),
                         (gi.cpu().numpy().astype(np.int64)[tok], gw.cpu().numpy().astype(np.float64)[tok]))
    assert_output_close("qwen2 layer output", y.cpu().numpy()[tok], ref)


def test_qwen2_57b_shape_one_pass_scores_output_and_pruned_output(P):
    """The calls of the Algorithm 2 loop on one 65536-token batch of the Qwen2-57B-A14B shape: the one-pass call gives
    camera_score_layer's energies bit for bit and the layer output within the forward tolerance on sampled tokens; the
    retained micro-experts' output from the stored h agrees with the oracle's sliced layer on those tokens."""
    from test_gpu_forward import assert_output_close, oracle_forward
    from _util import to_oracle_layer
    cfg = W().scaled(W().CONFIGS["qwen2_57b_a14b"], n_tokens=65536)
    L = W().make_layer(cfg, seed=0, device=DEV)
    X = W().make_tokens(cfg, seed=0, device=DEV)
    layer = P.Layer.from_workload(L)
    ws = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, cfg.n_tokens), DEV)
    ref = P.camera_score_layer(layer, X, 0.95, details=True)
    E, y = P.camera_score_forward_layer(layer, X, 0.95, workspace=ws,
                                        routing_in=(ref["topk_idx"], ref["topk_w"]))
    assert P.camera_read_status(ws) == 0
    assert torch.equal(E, ref["energy"])
    tok = np.sort(np.random.default_rng(5).choice(cfg.n_tokens, size=16, replace=False))
    tok[0], tok[-1] = 0, cfg.n_tokens - 1
    ol = to_oracle_layer(L)
    Xs = f64(X[torch.from_numpy(tok).to(DEV)])
    routing = (ref["topk_idx"].cpu().numpy().astype(np.int64)[tok], ref["topk_w"].cpu().numpy().astype(np.float64)[tok])
    assert_output_close("qwen2 one-pass output", y.cpu().numpy()[tok], oracle_forward(ol, Xs, routing))
    keep = P.camera_select_prune(E, 0.4)
    y_hat = P.camera_pruned_output(layer, P.camera_mask_down_columns(layer, keep), cfg.n_tokens, ws)
    assert P.camera_read_status(ws) == 0
    lists, _ = O.sub_index_lists(keep.cpu().numpy(), O.me_offsets(ol), [1])
    assert_output_close("qwen2 pruned output", y_hat.cpu().numpy()[tok], oracle_forward(O.slice_layer(ol, lists), Xs, routing))

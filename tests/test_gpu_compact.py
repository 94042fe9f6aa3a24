"""GPU parity of the selection's application to the weights: GetSubIndex (Algorithm 3, Algorithm 2) and the gathers W_up[S,:], W_gate[S,:], W_down[:,S] (Algorithm 2, the slicing step), bit for bit against
the oracle's index lists and slices."""
import numpy as np
import pytest
import torch

import oracle as O
from _util import f64, to_oracle_layer

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def W():
    from paper_2508_02322_b200 import workloads
    return workloads


def layer_cfg(**kw):
    base = dict(name="compact", d_model=256, n_routed=5, top_k=2, d_ff_routed=200, d_ff_shared=(72,),
                shared_gate_sigmoid=False, n_tokens=64, dtype="bf16", x_dist="normal")
    base.update(kw)
    return W().LayerConfig(**base)


def check_against_oracle(P, L, labels_np, order, n_take, down_ld=None):
    layer = P.Layer.from_workload(L)
    off = P.expert_offsets_tensor(layer)
    labels = torch.from_numpy(labels_np).to(DEV)
    sub, counts = P.camera_sub_index(labels, off, order)
    lists, ref_counts = O.sub_index_lists(labels_np, off.cpu().numpy(), order)
    assert np.array_equal(counts.cpu().numpy(), ref_counts)
    sub_np, off_np = sub.cpu().numpy(), off.cpu().numpy()
    for e in range(layer.n_experts):
        assert np.array_equal(sub_np[off_np[e]:off_np[e] + len(lists[e])], lists[e]), f"index list of expert {e}"
    out = None
    if down_ld is not None:
        t = layer.tensors
        out = {"w_gate": [torch.empty_like(w) for w in t["w_gate"]], "w_up": [torch.empty_like(w) for w in t["w_up"]],
               "w_down": [torch.empty((layer.d_model, ld), dtype=layer.dtype, device=DEV) for ld in down_ld]}
    out = P.camera_compact_weights(layer, sub, counts, n_take, out=out, down_ld=down_ld)
    taken = [np.concatenate([[], lists[e][:int(ref_counts[e, :n_take].sum())]]).astype(np.int64) for e in range(layer.n_experts)]
    ref = O.slice_layer(to_oracle_layer(L), taken)
    hf = L["down_layout"] == "hf"
    for e in range(layer.n_experts):
        m = len(taken[e])
        assert np.array_equal(f64(out["w_gate"][e][:m]), ref.w_gate[e]), f"W_gate of expert {e}"
        assert np.array_equal(f64(out["w_up"][e][:m]), ref.w_up[e]), f"W_up of expert {e}"
        got = f64(out["w_down"][e][:, :m]) if hf else f64(out["w_down"][e][:m]).T
        assert np.array_equal(got, ref.w_down[e]), f"W_down of expert {e}"
    return out, counts


@pytest.mark.parametrize("down_layout", ["hf", "me_major"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_prune_mask_to_sliced_weights(P, down_layout, dtype):
    cfg = layer_cfg(dtype=dtype)
    L = W().make_layer(cfg, seed=20, device=DEV, down_layout=down_layout)
    r = np.random.default_rng(20)
    keep = (r.random(sum(cfg.d_ff)) > 0.4).astype(np.uint8)
    keep[200:400] = 0          # an expert that loses every micro-expert
    keep[400:600] = 1          # one that keeps all
    check_against_oracle(P, L, keep, [1], 1)


def test_reorder_by_precision_class(P):
    cfg = layer_cfg()
    L = W().make_layer(cfg, seed=21, device=DEV)
    r = np.random.default_rng(21)
    bits = r.choice(np.array([3, 2, 1], dtype=np.uint8), size=sum(cfg.d_ff), p=[0.2, 0.6, 0.2])
    out, counts = check_against_oracle(P, L, bits, [3, 2, 1], 3)
    assert (counts.sum(dim=1).cpu().numpy() == np.array(cfg.d_ff)).all()
    check_against_oracle(P, L, bits, [3, 2, 1], 2)       # only the two wider classes are copied


def test_exact_size_outputs_for_w_down(P):
    cfg = layer_cfg()
    L = W().make_layer(cfg, seed=22, device=DEV)
    r = np.random.default_rng(22)
    keep = (r.random(sum(cfg.d_ff)) > 0.5).astype(np.uint8)
    off = np.concatenate([[0], np.cumsum(cfg.d_ff)])
    ld = [max(1, int(keep[off[e]:off[e + 1]].sum())) for e in range(len(cfg.d_ff))]
    check_against_oracle(P, L, keep, [1], 1, down_ld=ld)


def test_scores_to_pruned_layer_end_to_end(P):
    """Score, select, slice: the sliced layer's output equals the oracle's Phi[:,S] W[S,:] of the GPU's mask."""
    cfg = layer_cfg(n_tokens=300, d_ff_routed=256, d_ff_shared=(128,))
    L = W().make_layer(cfg, seed=23, device=DEV)
    X = W().make_tokens(cfg, seed=23, device=DEV)
    layer = P.Layer.from_workload(L)
    E = P.camera_score_layer(layer, X, 0.95)
    keep = P.camera_select_prune(E, 0.4)
    sub, counts = P.camera_sub_index(keep, P.expert_offsets_tensor(layer), [1])
    out = P.camera_compact_weights(layer, sub, counts, 1)
    m = counts[:, 0].cpu().numpy()
    ol = to_oracle_layer(L)
    pruned = O.OracleLayer(w_router=ol.w_router, top_k=ol.top_k,
                           w_gate=[f64(out["w_gate"][e][:m[e]]) for e in range(layer.n_experts)],
                           w_up=[f64(out["w_up"][e][:m[e]]) for e in range(layer.n_experts)],
                           w_down=[f64(out["w_down"][e][:, :m[e]]) for e in range(layer.n_experts)],
                           router_bias=ol.router_bias, norm_topk=ol.norm_topk, n_shared=ol.n_shared,
                           w_shared_gate=ol.w_shared_gate)
    S = np.nonzero(keep.cpu().numpy())[0]
    Xd = f64(X)
    Y_hat = O.phi_matrix(ol, Xd)[:, S] @ O.basis(ol)[S, :]
    assert np.allclose(O.forward(pruned, Xd), Y_hat, rtol=1e-12, atol=1e-12)
    assert int(m.sum()) == int(keep.sum()) == layer.n_me - int(0.4 * layer.n_me)


def test_compact_argument_errors(P):
    cfg = layer_cfg()
    L = W().make_layer(cfg, seed=24, device=DEV)
    layer = P.Layer.from_workload(L)
    off = P.expert_offsets_tensor(layer)
    labels = torch.ones(layer.n_me, dtype=torch.uint8, device=DEV)
    with pytest.raises(P.CameraError):
        P.camera_sub_index(labels, off, [1, 1])
    sub, counts = P.camera_sub_index(labels, off, [1])
    with pytest.raises(P.CameraError):
        P.camera_compact_weights(layer, sub, counts, 2)

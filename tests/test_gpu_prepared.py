"""camera_layer_prepare: with a handle a call must give exactly what it gives without one (which the other files
compare with the oracle), whether the per-call parts are rebuilt (first call, other tokens, other workspace, other
count) or reused (the same call again)."""
import numpy as np
import pytest
import torch

import oracle as O
from _gpu import assert_close
from _util import f64, to_oracle_layer

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def make(T=900, seed=60, **kw):
    from paper_2508_02322_b200 import workloads as W
    base = dict(name="prep", d_model=256, n_routed=6, top_k=2, d_ff_routed=256, d_ff_shared=(192,), shared_gate_sigmoid=True,
                n_tokens=T, dtype="bf16", x_dist="normal_rms1", router_bias_std=0.3, weight_std=0.05)
    base.update(kw)
    cfg = W.LayerConfig(**base)
    return cfg, W.make_layer(cfg, seed=seed, device=DEV), W.make_tokens(cfg, seed=seed, device=DEV)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_scores_with_a_handle_are_those_without(P, dtype):
    cfg, L, X = make(dtype=dtype)
    plain = P.Layer.from_workload(L)
    prepared = P.camera_layer_prepare(P.Layer.from_workload(L))
    ws = P.alloc_workspace(P.camera_score_workspace_bytes(plain, cfg.n_tokens), DEV)
    ref = P.camera_score_layer(plain, X, 0.95, details=True)
    for _ in range(3):                                   # built, then reused twice
        got = P.camera_score_layer(prepared, X, 0.95, details=True, workspace=ws)
        assert P.camera_read_status(ws) == 0
        for k in ("energy", "phi2", "phi_inf_sq", "omega2", "topk_idx", "topk_w", "shared_w", "expert_token_counts"):
            assert torch.equal(got[k], ref[k]), k
    # other tokens at another address, fewer of them, another workspace: the per-call parts follow
    X2 = X[100:700].clone()
    ws2 = P.alloc_workspace(P.camera_score_workspace_bytes(plain, cfg.n_tokens), DEV)
    for x, w in ((X2, ws), (X2, ws2), (X, ws2), (X, ws)):
        got = P.camera_score_layer(prepared, x, 0.95, workspace=w).clone()
        assert P.camera_read_status(w) == 0
        assert torch.equal(got, P.camera_score_layer(plain, x, 0.95))
    # and against the oracle directly
    ol, Xd = to_oracle_layer(L), f64(X)
    got = P.camera_score_layer(prepared, X, 0.95, details=True, workspace=ws)
    routing = (got["topk_idx"].cpu().numpy().astype(np.int64), got["topk_w"].cpu().numpy().astype(np.float64))
    E = O.energy(*O.camera_components(ol, Xd, routing=routing), float(np.float32(0.95)))
    assert_close("energy through a prepared layer", got["energy"].cpu().numpy(), E)


@pytest.mark.parametrize("T", [64, 1500])
def test_forward_calls_with_a_handle(P, T):
    cfg, L, X = make(T=T, seed=61)
    plain = P.Layer.from_workload(L)
    prepared = P.camera_layer_prepare(P.Layer.from_workload(L))
    ws = P.alloc_workspace(P.camera_forward_workspace_bytes(plain, T), DEV)
    y_ref = P.camera_layer_forward(plain, X)
    for _ in range(3):
        y = P.camera_layer_forward(prepared, X, workspace=ws)
        assert P.camera_read_status(ws) == 0
        assert torch.equal(y, y_ref)
    E_ref, y2_ref = P.camera_score_forward_layer(plain, X, 0.95)
    E, y2 = P.camera_score_forward_layer(prepared, X, 0.95, workspace=ws)
    assert torch.equal(E, E_ref) and torch.equal(y2, y2_ref)
    # scoring alone on the same handle in between, then the pruned output from the h of a fresh forward call
    assert torch.equal(P.camera_score_layer(prepared, X, 0.95), E_ref)
    E, y2 = P.camera_score_forward_layer(prepared, X, 0.95, workspace=ws)
    keep = P.camera_select_prune(E, 0.4)
    masked = P.camera_mask_down_columns(plain, keep)
    ws_plain = P.alloc_workspace(P.camera_forward_workspace_bytes(plain, T), DEV)
    P.camera_score_forward_layer(plain, X, 0.95, workspace=ws_plain)
    ref_hat = P.camera_pruned_output(plain, masked, T, ws_plain)
    for _ in range(2):
        assert torch.equal(P.camera_pruned_output(prepared, masked, T, ws), ref_hat)
    assert P.camera_read_status(ws) == 0
    # the layer's own W_down again after the masked one
    assert torch.equal(P.camera_layer_forward(prepared, X, workspace=ws), y_ref)


def test_a_handle_is_tied_to_its_layer(P):
    cfg, L, X = make(T=200, seed=62)
    prepared = P.camera_layer_prepare(P.Layer.from_workload(L))
    other = P.Layer.from_workload(L)
    other.c.prepared = prepared.c.prepared
    other.c.top_k = 3                                    # not the layer the handle was made for
    with pytest.raises(P.CameraError) as e:
        P.camera_score_layer(other, X, 0.95)
    assert e.value.status == -1
    other.c.prepared = None
    P.camera_layer_release(prepared)
    assert prepared.c.prepared is None
    E = P.camera_score_layer(prepared, X, 0.95)          # without a handle again
    assert torch.equal(E, P.camera_score_layer(P.Layer.from_workload(L), X, 0.95))


def test_a_repeated_decode_step_can_be_replayed_from_a_cuda_graph(P):
    """What the handle is for: a repeated call consists of memsets and kernel launches only, so a stream capture
    takes it as it is.  The replayed step gives the eager step's output."""
    cfg, L, X = make(T=64, seed=63)
    prepared = P.camera_layer_prepare(P.Layer.from_workload(L))
    ws = P.alloc_workspace(P.camera_forward_workspace_bytes(prepared, 64), DEV)
    y = torch.empty((64, cfg.d_model), dtype=torch.float32, device=DEV)
    y_ref = P.camera_layer_forward(prepared, X, y=y, workspace=ws).clone()     # builds the per-call parts
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        P.camera_layer_forward(prepared, X, y=y, workspace=ws)
        with torch.cuda.graph(graph, stream=side):
            P.camera_layer_forward(prepared, X, y=y, workspace=ws)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(y, y_ref)
    assert P.camera_read_status(ws) == 0

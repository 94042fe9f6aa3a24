"""Inputs and situations the kernels must turn into a status word instead of a fault or a hang: tokens whose routing
cannot be used (NaN / infinite hidden states, a prescribed expert out of range or named twice), and a wait inside a
kernel that runs out.  Every case here returns normally by construction: bad tokens get coefficient 0 and indices in
range, and the probe's wait is bounded by the limit the test passes."""
import time

import numpy as np
import pytest
import torch

import oracle as O
from _gpu import assert_close
from _util import f64, to_oracle_layer

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
INVALID_ARG, DEVICE_TIMEOUT = -1, -6


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def small_layer(dtype="bf16", T=300, seed=50):
    from paper_2508_02322_b200 import workloads as W
    cfg = W.LayerConfig("guards", 128, 6, 3, 128, (64,), True, T, dtype, "normal_rms1", router_bias_std=0.2, weight_std=0.05)
    return cfg, W.make_layer(cfg, seed=seed, device=DEV), W.make_tokens(cfg, seed=seed, device=DEV)


@pytest.mark.parametrize("T", [300, 90])       # 90 tokens: the front end for decode-sized batches
@pytest.mark.parametrize("router", ["tensor_core", "fma_bf16", "fma_fp32"])
def test_non_finite_tokens_set_the_status_word_and_nothing_faults(P, router, T):
    cfg, L, X = small_layer("f32" if router == "fma_fp32" else "bf16", T=T)
    layer = P.Layer.from_workload(L)
    bad_tokens = [5, 70, T - 1]
    Xb = X.clone()
    Xb[5, 17] = float("nan")
    Xb[70, :] = float("inf")
    Xb[T - 1, 3] = float("-inf")
    ws = P.alloc_workspace(P.camera_score_workspace_bytes(layer, cfg.n_tokens), DEV)
    out = P.camera_score_layer(layer, Xb, 0.95, details=True, workspace=ws, force_simt=router != "tensor_core")
    assert P.camera_read_status(ws) == INVALID_ARG
    idx = out["topk_idx"].cpu().numpy()
    w = out["topk_w"].cpu().numpy()
    assert idx.min() >= 0 and idx.max() < cfg.n_routed
    assert (np.sort(idx, axis=1)[:, 1:] != np.sort(idx, axis=1)[:, :-1]).all()      # k distinct experts per token
    assert (w[bad_tokens] == 0).all()
    good = np.setdiff1d(np.arange(cfg.n_tokens), bad_tokens)
    assert np.isfinite(w[good]).all() and (w[good] > 0).all()
    counts = out["expert_token_counts"].cpu().numpy()
    assert counts[:cfg.n_routed].sum() == cfg.n_tokens * cfg.top_k
    # the same workspace serves a clean call afterwards, with the result of a fresh one
    clean = P.camera_score_layer(layer, X, 0.95, details=True, workspace=ws, force_simt=router != "tensor_core")
    assert P.camera_read_status(ws) == 0
    fresh = P.camera_score_layer(layer, X, 0.95, details=True, force_simt=router != "tensor_core")
    assert torch.equal(clean["energy"], fresh["energy"]) and torch.equal(clean["topk_idx"], fresh["topk_idx"])


@pytest.mark.parametrize("T", [300, 120])
@pytest.mark.parametrize("router", ["tensor_core", "fma_bf16"])
def test_prescribed_routing_out_of_range_or_repeated(P, router, T):
    cfg, L, X = small_layer(T=T)
    layer = P.Layer.from_workload(L)
    ol, Xd = to_oracle_layer(L), f64(X)
    idx, w = O.top_and_norm(O.router_probs(ol, Xd), ol.top_k, ol.norm_topk)
    w32 = w.astype(np.float32)
    bad = idx.copy()
    bad[3, 1] = bad[3, 0]           # an expert named twice by one token
    bad[9, 2] = 99                  # past the last expert
    bad[T - 100, 0] = -1
    ws = P.alloc_workspace(P.camera_score_workspace_bytes(layer, cfg.n_tokens), DEV)
    out = P.camera_score_layer(layer, X, 0.95, details=True, workspace=ws, force_simt=router != "tensor_core",
                               routing_in=(torch.from_numpy(bad.astype(np.int32)), torch.from_numpy(w32)))
    assert P.camera_read_status(ws) == INVALID_ARG
    gi = out["topk_idx"].cpu().numpy()
    assert gi.min() >= 0 and gi.max() < cfg.n_routed
    # the three tokens count for nothing among the routed experts; everything else is scored as prescribed
    w_fixed = w32.astype(np.float64)
    w_fixed[[3, 9, T - 100]] = 0.0
    p2, pinf, w2 = O.camera_components(ol, Xd, routing=(idx, w_fixed))
    E = O.energy(p2, pinf, w2, float(np.float32(0.95)))
    assert_close("energy with three tokens dropped", out["energy"].cpu().numpy(), E)
    # a correct prescription on the same workspace
    ok = P.camera_score_layer(layer, X, 0.95, details=True, workspace=ws, force_simt=router != "tensor_core",
                              routing_in=(torch.from_numpy(idx.astype(np.int32)), torch.from_numpy(w32)))
    assert P.camera_read_status(ws) == 0
    p2, pinf, w2 = O.camera_components(ol, Xd, routing=(idx, w32.astype(np.float64)))
    assert_close("energy as prescribed", ok["energy"].cpu().numpy(), O.energy(p2, pinf, w2, float(np.float32(0.95))))


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(P):
    """The convention of every tensor-core kernel, exercised where nothing else is at stake: one CTA waits on a barrier
    nothing arrives on, with a limit of 1 ms; the launch returns, the status word says so, and ordinary work follows."""
    ws = P.alloc_workspace(4096, DEV)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    P.camera_wait_probe(ws, 1_000_000)
    assert P.camera_read_status(ws) == DEVICE_TIMEOUT           # synchronises the stream
    assert time.perf_counter() - t0 < 1.0
    # a longer limit is honoured too (the wait ends after it, not before)
    t0 = time.perf_counter()
    P.camera_wait_probe(ws, 50_000_000)
    assert P.camera_read_status(ws) == DEVICE_TIMEOUT
    dt = time.perf_counter() - t0
    assert 0.045 <= dt < 1.0
    with pytest.raises(P.CameraError):
        P.camera_wait_probe(ws, 5_000_000_000)                  # more than a second is refused
    # the next ordinary call, on a fresh workspace, is correct
    cfg, L, X = small_layer()
    layer = P.Layer.from_workload(L)
    ws2 = P.alloc_workspace(P.camera_score_workspace_bytes(layer, cfg.n_tokens), DEV)
    out = P.camera_score_layer(layer, X, 0.95, details=True, workspace=ws2)
    assert P.camera_read_status(ws2) == 0
    ol, Xd = to_oracle_layer(L), f64(X)
    routing = (out["topk_idx"].cpu().numpy().astype(np.int64), out["topk_w"].cpu().numpy().astype(np.float64))
    E = O.energy(*O.camera_components(ol, Xd, routing=routing), float(np.float32(0.95)))
    assert_close("energy after the probe", out["energy"].cpu().numpy(), E)


def test_wait_limit_is_a_runtime_setting(P):
    default = P.camera_get_wait_limit_ns()
    assert default == 4_000_000_000
    try:
        P.camera_set_wait_limit_ns(250_000_000)
        assert P.camera_get_wait_limit_ns() == 250_000_000
        # kernels take the limit in force when they are launched; a healthy call never comes near it
        cfg, L, X = small_layer(T=2000)
        layer = P.Layer.from_workload(L)
        ws = P.alloc_workspace(P.camera_score_workspace_bytes(layer, cfg.n_tokens), DEV)
        a = P.camera_score_layer(layer, X, 0.95, workspace=ws).clone()
        assert P.camera_read_status(ws) == 0
        with pytest.raises(P.CameraError):
            P.camera_set_wait_limit_ns(10)
        assert P.camera_get_wait_limit_ns() == 250_000_000
    finally:
        P.camera_set_wait_limit_ns(default)
    b = P.camera_score_layer(layer, X, 0.95, workspace=ws)
    assert torch.equal(a, b)

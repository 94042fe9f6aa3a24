"""Shared pieces of the GPU parity tests: run the CUDA path through the C ABI binding, run the
float64 oracle on the same stored values, and compare under the stated tolerances."""
import numpy as np
import torch

import oracle as O
from _util import to_oracle_layer, f64

REL_TOL = 1e-3          # scores: fp32 accumulation of bf16/fp32 products against float64
FLOOR = 1e-6            # ... relative to max(|ref_i|, FLOOR * max|ref|): a micro-expert a million times below the
                        # layer's largest score is dominated by the absolute rounding error of its fp32 dot products
TIE_TOL = 1e-5          # routing: relative gap of the k-th and (k+1)-th probability below which either is right
W_TOL = 1e-4            # router / shared-gate coefficients: a logit is an fp32 sum of d_model products of size ~1
                        # (absolute error up to ~d_model * 2^-24 = 2e-4 at d_model 3584, observed 3e-5), and softmax and
                        # sigmoid pass an absolute logit error on as a relative error of at most the same size


UNDERFLOW = 1e-30       # scores below this are squares of numbers fp32 cannot hold to 1e-3 (its normal range ends at
                        # 1.2e-38, and lambda^2 is formed in fp32): they are judged on the floored scale and not counted
FLOOR_LOG = []          # (name, elements compared, elements below the floor, of those: passing only thanks to it)


def assert_close(name, got, ref, rel=REL_TOL, max_floor_rescues=0):
    """Element by element within `rel` of max(|ref_i|, FLOOR * max|ref|).  Counts the elements that pass only thanks
    to the floor (beyond `rel` of their own value, and not in fp32's underflow range) and fails when there are more
    than `max_floor_rescues`: the floor exists for the rare micro-expert seen by one or two tokens whose fp32 dot
    product nearly cancels, not to hide a population of small scores.  Prints how many elements sat below the floor."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    floor = max(FLOOR * float(np.abs(ref).max(initial=0.0)), 1e-30)
    scale = np.maximum(np.abs(ref), floor)
    err = np.abs(got - ref) / scale
    # values that are exactly zero in the oracle must be exactly zero on the GPU
    zero = ref == 0
    assert (got[zero] == 0).all(), f"{name}: non-zero where the oracle is exactly zero"
    bad = err[~zero] > rel
    assert not bad.any(), f"{name}: {bad.sum()} of {bad.size} beyond {rel}, worst {err[~zero].max():.3e}"
    under = ~zero & (np.abs(ref) < floor)
    rescued = under & (np.abs(got - ref) > rel * np.abs(ref)) & (np.abs(ref) >= UNDERFLOW)
    FLOOR_LOG.append((name, int(ref.size), int(under.sum()), int(rescued.sum())))
    if under.any():
        print(f"[floor] {name}: {int(under.sum())} of {ref.size} elements below {FLOOR} of the maximum, "
              f"{int(rescued.sum())} pass only thanks to the floor")
    assert rescued.sum() <= max_floor_rescues, \
        f"{name}: {int(rescued.sum())} elements beyond {rel} of their own value pass only on the floored scale (allowed {max_floor_rescues})"
    return int(rescued.sum())


def check_routing(olayer, Xd, topk_idx, topk_w):
    """GPU routing against the oracle's.  Returns the number of near-tie tokens whose expert set differs."""
    if olayer.n_routed == 0:
        return 0
    p = O.router_probs(olayer, Xd)
    idx_o, w_o = O.top_and_norm(p, olayer.top_k, olayer.norm_topk)
    gi = topk_idx.cpu().numpy().astype(np.int64)
    gw = topk_w.cpu().numpy().astype(np.float64)
    same = (np.sort(gi, axis=1) == np.sort(idx_o, axis=1)).all(axis=1)
    k = olayer.top_k
    if not same.all():
        ps = -np.sort(-p, axis=1)
        if k < p.shape[1]:
            gap = (ps[:, k - 1] - ps[:, k]) / ps[:, k - 1]
            assert (gap[~same] < TIE_TOL).all(), "expert sets differ on tokens that are not near-ties"
        else:
            raise AssertionError("expert sets differ with k == n_routed")
    # weights of the tokens that agree, matched by expert
    order_g, order_o = np.argsort(gi, axis=1), np.argsort(idx_o, axis=1)
    wg = np.take_along_axis(gw, order_g, axis=1)[same]
    wo = np.take_along_axis(w_o, order_o, axis=1)[same]
    assert np.abs(wg - wo).max() <= W_TOL * max(1.0, np.abs(wo).max()), "router weights differ"
    # order of the exported slots: decreasing probability
    assert (np.diff(gw, axis=1) <= 1e-6).all()
    return int((~same).sum())


def run_and_compare(P, L, X, alpha=0.95, channels=None, force_simt=False, check_dense=False, cta_pair=None,
                    max_floor_rescues=0):
    """Scores one layer on the GPU (own routing, then the oracle's routing injected) and checks
    every component against the oracle.  `channels` restricts the oracle to sampled micro-experts."""
    layer = P.Layer.from_workload(L)
    olayer = to_oracle_layer(L)
    Xd = f64(X)
    ws = P.alloc_workspace(P.camera_score_workspace_bytes(layer, X.shape[0]), X.device)
    out = P.camera_score_layer(layer, X, alpha, details=True, workspace=ws, force_simt=force_simt, cta_pair=cta_pair)
    assert P.camera_read_status(ws) == 0
    flips = check_routing(olayer, Xd, out["topk_idx"], out["topk_w"])

    # (1) scoring under the GPU's own routing: the oracle is given that routing
    routing = None
    if olayer.n_routed:
        routing = (out["topk_idx"].cpu().numpy().astype(np.int64), out["topk_w"].cpu().numpy().astype(np.float64))
    shared_w = out["shared_w"].cpu().numpy().astype(np.float64).T
    if olayer.n_shared:
        assert_close("shared_w", shared_w, O.shared_coeff(olayer, Xd), rel=W_TOL)
    phi2, phi_inf, omega2 = O.camera_components(olayer, Xd, channels=channels, routing=routing)
    sel = ~np.isnan(phi2)
    assert_close("omega2", out["omega2"].cpu().numpy(), omega2, max_floor_rescues=max_floor_rescues)
    assert_close("phi2", out["phi2"].cpu().numpy()[sel], phi2[sel], max_floor_rescues=max_floor_rescues)
    assert_close("phi_inf_sq", out["phi_inf_sq"].cpu().numpy()[sel], phi_inf[sel], max_floor_rescues=max_floor_rescues)
    E = O.energy(phi2, phi_inf, omega2, float(np.float32(alpha)))
    assert_close("energy", out["energy"].cpu().numpy()[sel], E[sel], max_floor_rescues=max_floor_rescues)
    counts = out["expert_token_counts"].cpu().numpy()
    if olayer.n_routed:
        assert np.array_equal(counts[:olayer.n_routed], np.bincount(routing[0].reshape(-1), minlength=olayer.n_routed))
    assert (counts[olayer.n_routed:] == X.shape[0]).all()

    # (2) the oracle's routing injected into the GPU path: no token is excluded
    if olayer.n_routed:
        idx_o, w_o = O.top_and_norm(O.router_probs(olayer, Xd), olayer.top_k, olayer.norm_topk)
        w32 = w_o.astype(np.float32)
        out2 = P.camera_score_layer(layer, X, alpha, details=True, workspace=ws, force_simt=force_simt, cta_pair=cta_pair,
                                    routing_in=(torch.from_numpy(idx_o.astype(np.int32)), torch.from_numpy(w32)))
        assert P.camera_read_status(ws) == 0
        p2, pi, w2 = O.camera_components(olayer, Xd, channels=channels, routing=(idx_o, w32.astype(np.float64)))
        assert_close("phi2 (oracle routing)", out2["phi2"].cpu().numpy()[sel], p2[sel], max_floor_rescues=max_floor_rescues)
        assert_close("phi_inf_sq (oracle routing)", out2["phi_inf_sq"].cpu().numpy()[sel], pi[sel], max_floor_rescues=max_floor_rescues)
        assert_close("energy (oracle routing)", out2["energy"].cpu().numpy()[sel],
                     O.energy(p2, pi, w2, float(np.float32(alpha)))[sel], max_floor_rescues=max_floor_rescues)
    if check_dense:
        d2, dinf, dw = O.camera_components_dense(olayer, Xd)
        if flips == 0:
            assert_close("phi2 vs literal Algorithm 1", out["phi2"].cpu().numpy(), d2, max_floor_rescues=max_floor_rescues)
            assert_close("phi_inf_sq vs literal Algorithm 1", out["phi_inf_sq"].cpu().numpy(), dinf, max_floor_rescues=max_floor_rescues)
    return out, flips


def sample_channels(d_ff, per_expert, seed=0):
    """A seeded sample of micro-experts per expert that always holds the first and last channel
    and a channel on either side of a 64-channel tile edge."""
    r = np.random.default_rng(seed)
    ch = {}
    for e, f in enumerate(d_ff):
        must = {0, f - 1, min(63, f - 1), min(64, f - 1)}
        extra = set(r.choice(f, size=min(per_expert, f), replace=False).tolist())
        ch[e] = sorted(must | extra)
    return ch

"""GPU parity of the layer output (Eq. 1-2) and of the output of a sliced layer (Y_hat = Phi[:,S] W[S,:], Eq. 7)
against the float64 oracle, and of the error metrics against their definitions.

Tolerance, derived from the arithmetic and evaluated by the oracle per output element (it has Phi and W):
the GPU forms g = w_gate.x and u = w_up.x as fp32 sums of d_model bf16 products, rounds phi = a SiLU(g) u to bf16
(h, the operand of the second GEMM) and adds the d_ff products phi_i w_i[c] in fp32.  With u16 = 2^-8 (half an ulp of
bf16's 8-bit significand) and u32 = 2^-23 (one ulp of fp32: the tensor cores may truncate their sums),

  hard bound   |y_gpu - y|[t,c] <= sum_i (u16 |phi_ti| + dphi_ti) |w_i[c]| + f u32 sum_i |phi_ti| |w_i[c]|
               with dphi = a (1.1 dg |u| + |SiLU(g)| du + 1.1 dg du) + 4e-6 |phi|,  dg = d u32 (|x| . |w_gate|),
               du likewise (|SiLU'| <= 1.1; 4e-6 covers the fast exp / divide of the epilogue): every rounding error
               at its largest and all of one sign.  No element may pass it.
  statistics   the roundings of different micro-experts are independent, a bf16 rounding error is uniform within
               +-u16 |phi| (variance u16^2 phi^2 / 3) and an fp32 sum of n terms strays by about sqrt(n) u32 times
               its terms' size, so  sigma^2[t,c] = sum_i (u16^2 phi_ti^2 / 3 + dphi'_ti^2) w_i[c]^2  with dphi' as
               above under dg = sqrt(d) u32 (|x| . |w_gate|).  No element may pass 8 sigma (plus the fp32 part of the
               hard bound's last term taken at sqrt(f)), and the whole error is at most 1.5 sqrt(sum sigma^2) in
               Frobenius norm (a sum of 10^5 and more independent squares sits within a few per cent of its mean).
"""
import numpy as np
import pytest
import torch

import oracle as O
from _util import f64, to_oracle_layer

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
U16, U32 = 2.0 ** -8, 2.0 ** -23
SIGMAS, FRO_FACTOR = 8.0, 1.5


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def W():
    from paper_2508_02322_b200 import workloads
    return workloads


def cfg_of(**kw):
    base = dict(name="fwd", d_model=256, n_routed=6, top_k=2, d_ff_routed=256, d_ff_shared=(192,),
                shared_gate_sigmoid=True, n_tokens=700, dtype="bf16", x_dist="normal_rms1", router_bias_std=0.3,
                weight_std=0.05)
    base.update(kw)
    return W().LayerConfig(**base)


class OutputRef:
    """The oracle's layer output with, per element, the hard error bound and the variance of the header."""

    def __init__(self, y, hard, var):
        self.y, self.hard, self.var = y, hard, var


def oracle_forward(ol, Xd, routing):
    """Eq. 1-2 with the routed coefficients prescribed (the ones handed to the GPU), and the error model of the
    header evaluated on the same Phi and W."""
    A = O.coefficients(ol, Xd, routing=routing)
    d = Xd.shape[1]
    T, dm = Xd.shape[0], ol.w_down[0].shape[0]
    Y, hard, var = np.zeros((T, dm)), np.zeros((T, dm)), np.zeros((T, dm))
    absX = np.abs(Xd)
    for e in range(ol.n_experts):
        a = np.abs(A[:, e:e + 1])
        tok = np.nonzero(a[:, 0])[0]
        if tok.size == 0 or ol.d_ff[e] == 0:
            continue
        wg, wu, wd = ol.w_gate[e], ol.w_up[e], ol.w_down[e]
        G, U = Xd[tok] @ wg.T, Xd[tok] @ wu.T
        sil = O.silu(G)
        phi = A[tok, e:e + 1] * sil * U
        Ye = phi @ wd.T
        Y[tok] += Ye
        if e >= ol.n_routed and ol.w_shared_gate is not None:
            # the coefficient of a gated shared expert is the sigmoid of an fp32 logit: one relative error for the
            # whole expert (the routed coefficients are handed over as fp32 values, exactly)
            hard[tok] += d * U32 * np.abs(Ye)
            var[tok] += (np.sqrt(d) * U32 * Ye) ** 2
        Gabs, Uabs = absX[tok] @ np.abs(wg).T, absX[tok] @ np.abs(wu).T
        f = ol.d_ff[e]

        def dphi(scale):     # error of phi from errors dg = scale * Gabs, du = scale * Uabs of the two fp32 sums
            dg, du = scale * Gabs, scale * Uabs
            return a[tok] * (1.1 * dg * np.abs(U) + np.abs(sil) * du + 1.1 * dg * du) + 4e-6 * np.abs(phi)

        absW = np.abs(wd).T
        pw = np.abs(phi) @ absW
        hard[tok] += (U16 * np.abs(phi) + dphi(d * U32)) @ absW + f * U32 * pw
        var[tok] += (U16 ** 2 / 3.0 * phi ** 2 + dphi(np.sqrt(d) * U32) ** 2) @ (absW ** 2) + (np.sqrt(f) * U32 * pw) ** 2
    n_terms = A.shape[1]
    hard += n_terms * 2.0 ** -24 * np.abs(Y) + 1e-30       # the fp32 sum over a token's experts
    return OutputRef(Y, hard, var)


def assert_output_close(name, got, ref):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref.y)
    over = err > ref.hard
    assert not over.any(), f"{name}: {over.sum()} of {err.size} elements beyond the hard bound, worst {np.max(err / ref.hard):.3f} of it"
    sigma = np.sqrt(ref.var)
    stat = SIGMAS * sigma + 8 * 2.0 ** -24 * np.abs(ref.y) + 1e-30       # ... and the fp32 sum over a token's experts
    over = err > stat
    assert not over.any(), f"{name}: {over.sum()} of {err.size} elements beyond {SIGMAS} sigma, worst {np.max(err / np.maximum(sigma, 1e-300)):.2f} sigma"
    fro, fro_model = np.sqrt((err ** 2).sum()), np.sqrt(ref.var.sum())
    assert fro <= FRO_FACTOR * fro_model + 1e-30, f"{name}: Frobenius error {fro:.3e} against a model of {fro_model:.3e}"
    assert (got[(ref.y == 0).all(axis=1)] == 0).all()
    return float(np.max(err / np.maximum(sigma, 1e-300))), float(fro / max(fro_model, 1e-300))


def oracle_routing(ol, Xd):
    idx, w = O.top_and_norm(O.router_probs(ol, Xd), ol.top_k, ol.norm_topk)
    w32 = w.astype(np.float32)
    return (torch.from_numpy(idx.astype(np.int32)), torch.from_numpy(w32)), (idx, w32.astype(np.float64))


KERNELS = {"single": dict(cta_pair=False), "pair": dict(cta_pair=True), "token_rows": dict(token_rows=True)}


@pytest.mark.parametrize("kernel", list(KERNELS))
@pytest.mark.parametrize("T", [1, 255, 700, 5000])
def test_layer_output(P, T, kernel):
    cfg = cfg_of(n_tokens=T)
    L = W().make_layer(cfg, seed=30, device=DEV)
    X = W().make_tokens(cfg, seed=30, device=DEV)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    y = P.camera_layer_forward(P.Layer.from_workload(L), X, routing_in=rin, **KERNELS[kernel])
    ref = oracle_forward(ol, Xd, rout)
    assert np.allclose(ref.y, O.forward(ol, Xd), rtol=1e-5, atol=1e-6)       # the helper above is Eq. 1-2 (coefficients rounded to fp32)
    assert_output_close("layer output", y.cpu().numpy(), ref)


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_layer_output_own_routing_and_no_shared(P, kernel):
    # d_ff 320 = 2.5 tiles of 128: a pair's second CTA has a half tile, then none, of h's 384 padded columns; with the
    # tokens on the accumulator rows the second unit of an expert is 64 micro-experts wide
    cfg = cfg_of(n_tokens=900, d_ff_shared=(), shared_gate_sigmoid=False, n_routed=5, top_k=3, d_ff_routed=320)
    L = W().make_layer(cfg, seed=31, device=DEV)
    X = W().make_tokens(cfg, seed=31, device=DEV)
    ol, Xd = to_oracle_layer(L), f64(X)
    y, (gi, gw) = P.camera_layer_forward(P.Layer.from_workload(L), X, want_routing=True, **KERNELS[kernel])
    ref = oracle_forward(ol, Xd, (gi.cpu().numpy().astype(np.int64), gw.cpu().numpy().astype(np.float64)))
    assert_output_close("layer output under the GPU's routing", y.cpu().numpy(), ref)


@pytest.mark.parametrize("d_ff", [8, 72, 200, 264, 648])
def test_token_rows_kernel_ragged_widths(P, d_ff):
    """Widths that leave the last unit 64, 128 or 192 micro-experts wide, or the only unit narrower than a k-block."""
    cfg = cfg_of(n_tokens=1500, n_routed=3, top_k=2, d_ff_routed=d_ff, d_ff_shared=(d_ff + 64,))
    L = W().make_layer(cfg, seed=35, device=DEV)
    X = W().make_tokens(cfg, seed=35, device=DEV)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    y = P.camera_layer_forward(P.Layer.from_workload(L), X, routing_in=rin, token_rows=True)
    assert_output_close(f"token rows, d_ff {d_ff}", y.cpu().numpy(), oracle_forward(ol, Xd, rout))


@pytest.mark.parametrize("cta_pair", [False, True])
def test_scores_and_output_from_one_pass(P, cta_pair):
    """camera_score_forward_layer: the energies against the oracle's (Algorithm 1) and bit for bit against
    camera_score_layer's, the output bit for bit against camera_layer_forward's, also when the tokens come in two
    batches that accumulate."""
    from _gpu import assert_close
    cfg = cfg_of(n_tokens=1300, d_ff_routed=320)
    L = W().make_layer(cfg, seed=36, device=DEV)
    X = W().make_tokens(cfg, seed=36, device=DEV)
    layer = P.Layer.from_workload(L)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    E, y = P.camera_score_forward_layer(layer, X, 0.95, routing_in=rin, cta_pair=cta_pair)
    E_ref = P.camera_score_layer(layer, X, 0.95, routing_in=rin, cta_pair=cta_pair)
    y_ref = P.camera_layer_forward(layer, X, routing_in=rin, cta_pair=cta_pair)
    assert torch.equal(E, E_ref) and torch.equal(y, y_ref)
    p2, pinf, w2 = O.camera_components(ol, Xd, routing=rout)
    assert_close("energy from the one-pass call", E.cpu().numpy(), O.energy(p2, pinf, w2, float(np.float32(0.95))))
    assert_output_close("output from the one-pass call", y.cpu().numpy(), oracle_forward(ol, Xd, rout))
    # two batches: the components accumulate, the outputs are the batches' rows
    phi2 = torch.empty(layer.n_me, dtype=torch.float32, device=DEV)
    pinf_t = torch.empty_like(phi2)
    E2 = torch.empty_like(phi2)
    om = torch.empty_like(phi2)             # the W_down norms: computed with the first batch, given to the second
    y2 = torch.empty_like(y)
    ws = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, 800), DEV)
    for i, (t0, t1) in enumerate([(0, 800), (800, 1300)]):
        P.camera_score_forward_layer(layer, X[t0:t1], 0.95, energy=E2, y=y2[t0:t1], workspace=ws, phi2=phi2,
                                     phi_inf_sq=pinf_t, accumulate=i > 0, cta_pair=cta_pair, omega2=om, omega_given=i > 0,
                                     routing_in=(rin[0][t0:t1], rin[1][t0:t1]))
    assert P.camera_read_status(ws) == 0
    assert_close("energy accumulated over two batches", E2.cpu().numpy(), O.energy(p2, pinf, w2, float(np.float32(0.95))))
    assert_output_close("output in two batches", y2.cpu().numpy(), oracle_forward(ol, Xd, rout))


@pytest.mark.parametrize("T,ratio", [(1300, 0.4), (5000, 0.7), (70, 0.2)])
def test_pruned_output_from_stored_h(P, T, ratio):
    """Phi[:,S] W[S,:] of Eq. 7 from the h the one-pass call left in its workspace and W_down with the pruned columns
    zeroed: against the oracle's sliced layer, and against the sliced layer run through camera_layer_forward (the same
    products, another order of the fp32 sums over d_ff)."""
    cfg = cfg_of(n_tokens=T, d_ff_routed=320, d_ff_shared=(192,))
    L = W().make_layer(cfg, seed=38, device=DEV)
    X = W().make_tokens(cfg, seed=38, device=DEV)
    layer = P.Layer.from_workload(L)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    ws = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, T), DEV)
    E, y = P.camera_score_forward_layer(layer, X, 0.95, routing_in=rin, workspace=ws)
    keep = P.camera_select_prune(E, ratio)
    keep[320:640] = 0                       # one routed expert loses every micro-expert
    masked = P.camera_mask_down_columns(layer, keep)
    off = O.me_offsets(ol)
    for e in range(layer.n_experts):        # the masking itself, bit for bit
        k = keep[off[e]:off[e + 1]].bool()
        assert torch.equal(masked[e], torch.where(k[None, :], L["w_down"][e], torch.zeros_like(L["w_down"][e])))
    y_hat = P.camera_pruned_output(layer, masked, T, ws)
    y_hat2 = P.camera_pruned_output(layer, masked, T, ws)          # the call leaves the workspace reusable
    assert torch.equal(y_hat, y_hat2)
    assert P.camera_read_status(ws) == 0
    lists, _ = O.sub_index_lists(keep.cpu().numpy(), off, [1])
    ref_hat = oracle_forward(O.slice_layer(ol, lists), Xd, rout)
    assert_output_close("pruned output from stored h", y_hat.cpu().numpy(), ref_hat)
    # the sliced layer through the forward call
    sub, counts = P.camera_sub_index(keep, P.expert_offsets_tensor(layer), [1])
    out = P.camera_compact_weights(layer, sub, counts, 1)
    m = counts[:, 0].cpu().numpy()
    sliced = P.Layer(L["w_router"], [out["w_gate"][e][:m[e]] for e in range(layer.n_experts)],
                     [out["w_up"][e][:m[e]] for e in range(layer.n_experts)], out["w_down"], cfg.top_k, cfg.n_shared,
                     L["router_bias"], L["w_shared_gate"], cfg.norm_topk, "hf", down_ld=layer.d_ff)
    y_sl = P.camera_layer_forward(sliced, X, routing_in=rin).cpu().numpy().astype(np.float64)
    got = y_hat.cpu().numpy().astype(np.float64)
    rms = np.sqrt((y_sl ** 2).mean(axis=1, keepdims=True))
    assert (np.abs(got - y_sl) <= 1e-5 * np.maximum(rms, 1e-30)).all()
    # and the full mask gives back the layer's own output
    full = P.camera_mask_down_columns(layer, torch.ones_like(keep))
    assert torch.equal(P.camera_pruned_output(layer, full, T, ws), y)
    # the h that camera_layer_forward leaves behind serves as well
    y_fw = P.camera_layer_forward(layer, X, routing_in=rin, workspace=ws)
    assert torch.equal(P.camera_pruned_output(layer, full, T, ws), y_fw)
    assert torch.equal(P.camera_pruned_output(layer, masked, T, ws), y_hat)


def test_one_pass_call_without_tokens(P):
    cfg = cfg_of(n_tokens=0)
    L = W().make_layer(cfg, seed=37, device=DEV)
    layer = P.Layer.from_workload(L)
    X = torch.empty((0, cfg.d_model), dtype=torch.bfloat16, device=DEV)
    E, y = P.camera_score_forward_layer(layer, X, 0.95)
    assert y.shape == (0, cfg.d_model) and float(E.abs().max()) == 0.0


def test_dense_layer_is_a_gated_ffn(P):
    cfg = cfg_of(n_tokens=400, n_routed=0, top_k=1, d_ff_shared=(384,), shared_gate_sigmoid=False, router_bias_std=0.0)
    L = W().make_layer(cfg, seed=32, device=DEV)
    X = W().make_tokens(cfg, seed=32, device=DEV)
    y = P.camera_layer_forward(P.Layer.from_workload(L), X)
    Xd = f64(X)
    ref = oracle_forward(to_oracle_layer(L), Xd, None)
    assert np.allclose(ref.y, O.expert_hidden(Xd, f64(L["w_gate"][0]), f64(L["w_up"][0])) @ f64(L["w_down"][0]).T,
                       rtol=1e-12, atol=1e-12)              # one expert, coefficient 1: a plain gated FFN
    assert_output_close("dense FFN", y.cpu().numpy(), ref)


@pytest.mark.parametrize("ratio", [0.2, 0.6])
def test_sliced_layer_output_and_error_metrics(P, ratio):
    """Score, select, slice, run the sliced layer: its output is Phi[:,S] W[S,:] of the GPU's own mask, and the
    reported error is the objective of Eq. 7 for that mask."""
    cfg = cfg_of(n_tokens=1200)
    L = W().make_layer(cfg, seed=33, device=DEV)
    X = W().make_tokens(cfg, seed=33, device=DEV)
    layer = P.Layer.from_workload(L)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    E = P.camera_score_layer(layer, X, 0.95, routing_in=rin)
    keep = P.camera_select_prune(E, ratio)
    keep[256:512] = 0                       # one routed expert loses every micro-expert
    sub, counts = P.camera_sub_index(keep, P.expert_offsets_tensor(layer), [1])
    out = P.camera_compact_weights(layer, sub, counts, 1)
    m = counts[:, 0].cpu().numpy()
    assert m[1] == 0
    sliced = P.Layer(L["w_router"], [out["w_gate"][e][:m[e]] for e in range(layer.n_experts)],
                     [out["w_up"][e][:m[e]] for e in range(layer.n_experts)], out["w_down"], cfg.top_k, cfg.n_shared,
                     L["router_bias"], L["w_shared_gate"], cfg.norm_topk, "hf", down_ld=layer.d_ff)
    y = P.camera_layer_forward(layer, X, routing_in=rin)
    y_hat = P.camera_layer_forward(sliced, X, routing_in=rin, token_rows=ratio > 0.5)
    lists, _ = O.sub_index_lists(keep.cpu().numpy(), O.me_offsets(ol), [1])
    ref_hat = oracle_forward(O.slice_layer(ol, lists), Xd, rout)
    assert_output_close("sliced layer output", y_hat.cpu().numpy(), ref_hat)
    # the metrics against their definitions on the same two fp32 arrays
    got = P.camera_output_error(y, y_hat).cpu().numpy()
    a, b = y.cpu().numpy().astype(np.float64), y_hat.cpu().numpy().astype(np.float64)
    cos = (a * b).sum(1) / np.sqrt((a * a).sum(1) * (b * b).sum(1))
    assert np.allclose(got, [((a - b) ** 2).sum(), (a * a).sum(), cos.mean()], rtol=1e-12)
    # and against the oracle's decoding error of the pruned set (Eq. 7), which the bf16 rounding of h perturbs a little
    ref_err = ((oracle_forward(ol, Xd, rout).y - ref_hat.y) ** 2).sum()
    assert abs(got[0] - ref_err) <= 0.02 * ref_err


def test_forward_argument_errors(P):
    cfg = cfg_of(dtype="f32", n_tokens=64)
    L = W().make_layer(cfg, seed=34, device=DEV)
    X = W().make_tokens(cfg, seed=34, device=DEV)
    with pytest.raises(P.CameraError) as e:
        P.camera_layer_forward(P.Layer.from_workload(L), X)
    assert e.value.status == -2


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_residual_norm(P, dtype):
    g = torch.Generator(device="cpu").manual_seed(3)
    x = (torch.randn(1001, 256, generator=g) * 2).to(dtype).to(DEV)
    y = (torch.randn(1001, 256, generator=g) * 0.5).to(DEV)
    out = P.camera_residual_norm(x, y, eps=1e-6)
    ref = O.next_layer_input(f64(x), f64(y), eps=1e-6)
    tol = 2.0 ** -8 if dtype == torch.bfloat16 else 1e-6       # one rounding to the output dtype
    assert np.abs(f64(out) - ref).max() <= tol * np.abs(ref).max()
    assert out.dtype == dtype


@pytest.mark.parametrize("shape", ["gated_shared", "many_small_experts"])
def test_decode_batch_full_and_sliced_layers(P, shape):
    """A decode step: 64 tokens through the full layer and through the layer sliced at 40 % by CAMERA-P masks taken
    on calibration tokens, each against the oracle (Eq. 1-2 on the full and on the sliced weights), with and without a
    prepared layer."""
    kw = dict(d_model=256, n_routed=6, top_k=2, d_ff_routed=256, d_ff_shared=(192,), shared_gate_sigmoid=True) \
        if shape == "gated_shared" else \
        dict(d_model=128, n_routed=16, top_k=6, d_ff_routed=64, d_ff_shared=(64, 64), shared_gate_sigmoid=False)
    cfg = cfg_of(n_tokens=2000, **kw)
    L = W().make_layer(cfg, seed=40, device=DEV)
    Xcal = W().make_tokens(cfg, seed=40, device=DEV)
    layer = P.Layer.from_workload(L)
    keep = P.camera_select_prune(P.camera_score_layer(layer, Xcal, 0.95), 0.4)
    X = W().make_tokens(W().scaled(cfg, n_tokens=64), seed=41, device=DEV)
    ol, Xd = to_oracle_layer(L), f64(X)
    rin, rout = oracle_routing(ol, Xd)
    ref = oracle_forward(ol, Xd, rout)
    for lay in (layer, P.camera_layer_prepare(P.Layer.from_workload(L))):
        assert_output_close("decode batch, full layer", P.camera_layer_forward(lay, X, routing_in=rin).cpu().numpy(), ref)
        y, (gi, gw) = P.camera_layer_forward(lay, X, want_routing=True)              # the layer's own router
        ref_own = oracle_forward(ol, Xd, (gi.cpu().numpy().astype(np.int64), gw.cpu().numpy().astype(np.float64)))
        assert_output_close("decode batch, own routing", y.cpu().numpy(), ref_own)
    from _gpu import check_routing
    check_routing(ol, Xd, gi, gw)
    sub, counts = P.camera_sub_index(keep, P.expert_offsets_tensor(layer), [1])
    out = P.camera_compact_weights(layer, sub, counts, 1)
    m = counts[:, 0].cpu().numpy()
    def sliced():
        return P.Layer(L["w_router"], [out["w_gate"][e][:m[e]] for e in range(layer.n_experts)],
                       [out["w_up"][e][:m[e]] for e in range(layer.n_experts)], out["w_down"], cfg.top_k, cfg.n_shared,
                       L["router_bias"], L["w_shared_gate"], cfg.norm_topk, "hf", down_ld=layer.d_ff)
    lists, _ = O.sub_index_lists(keep.cpu().numpy(), O.me_offsets(ol), [1])
    ref_hat = oracle_forward(O.slice_layer(ol, lists), Xd, rout)
    for lay in (sliced(), P.camera_layer_prepare(sliced())):
        assert_output_close("decode batch, sliced layer", P.camera_layer_forward(lay, X, routing_in=rin).cpu().numpy(), ref_hat)

"""GPU parity: the CUDA path, called through the C ABI binding, against the float64 oracle on the
same seeded inputs.  Scores within 1e-3 relative (fp32 accumulation), routing / masks / bit-widths
bit-exact (routing: except near-ties, which are reported)."""
import numpy as np
import pytest
import torch

import oracle as O
from _gpu import REL_TOL, assert_close, run_and_compare, sample_channels
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


def small_cfg(**kw):
    base = dict(name="small", d_model=256, n_routed=6, top_k=2, d_ff_routed=128, d_ff_shared=(192,),
                shared_gate_sigmoid=True, n_tokens=700, dtype="bf16", x_dist="normal_rms1", router_bias_std=0.3)
    base.update(kw)
    return W().LayerConfig(**base)


# ------------------------------------------------------------------ config 1: tiny fp32, everything
def test_tiny_fp32_full(P):
    cfg = W().CONFIGS["tiny_fp32"]
    L = W().make_layer(cfg, seed=0, device=DEV)
    X = W().make_tokens(cfg, seed=0, device=DEV)
    out, flips = run_and_compare(P, L, X, alpha=0.95, check_dense=True)
    E = out["energy"]
    E_np = E.cpu().numpy()
    keep = P.camera_select_prune(E, 0.40)
    assert np.array_equal(keep.cpu().numpy(), O.select_prune(E_np, 0.40))
    assert int((keep == 0).sum()) == int(0.4 * 4096)
    bits = P.camera_alloc_bits(E, [0.2, 0.6, 0.2], [4, 3, 2])
    assert np.array_equal(bits.cpu().numpy(), O.alloc_bits(E_np, [0.2, 0.6, 0.2], [4, 3, 2])[0])
    # mask from GPU scores against mask from oracle scores: may differ only inside the tolerance band
    olayer = to_oracle_layer(L)
    Eo = O.energy(*O.camera_components(olayer, f64(X)), float(np.float32(0.95)))
    keep_o = O.select_prune(Eo, 0.40)
    diff = np.nonzero(keep.cpu().numpy() != keep_o)[0]
    tau = np.sort(Eo)[int(0.4 * 4096)]
    assert (np.abs(Eo[diff] - tau) <= REL_TOL * tau).all()
    assert int(keep.sum()) == int(keep_o.sum())


@pytest.mark.parametrize("alpha", [0.0, 0.5, 1.0])
def test_tiny_fp32_alpha_sweep(P, alpha):
    cfg = W().scaled(W().CONFIGS["tiny_fp32"], n_tokens=200)
    L = W().make_layer(cfg, seed=1, device=DEV)
    X = W().make_tokens(cfg, seed=1, device=DEV)
    run_and_compare(P, L, X, alpha=alpha)


# ------------------------------------------------------------------ bf16: tensor-core kernel and the FMA kernel
@pytest.mark.parametrize("kernel", ["umma", "umma_pair", "simt"])
@pytest.mark.parametrize("down_layout", ["hf", "me_major"])
def test_small_bf16(P, kernel, down_layout):
    cfg = small_cfg()
    L = W().make_layer(cfg, seed=2, device=DEV, down_layout=down_layout)
    X = W().make_tokens(cfg, seed=2, device=DEV)
    run_and_compare(P, L, X, alpha=0.95, force_simt=kernel == "simt", cta_pair=kernel == "umma_pair" if kernel != "simt" else None,
                    check_dense=True)


@pytest.mark.parametrize("cta_pair", [False, True])
@pytest.mark.parametrize("T", [1, 15, 16, 17, 255, 256, 257, 1030])
def test_ragged_token_counts(P, T, cta_pair):
    cfg = small_cfg(n_tokens=T, n_routed=4, d_ff_routed=64, d_ff_shared=(64,))
    L = W().make_layer(cfg, seed=3, device=DEV)
    X = W().make_tokens(cfg, seed=3, device=DEV)
    run_and_compare(P, L, X, alpha=0.5, cta_pair=cta_pair)


def test_zero_tokens(P):
    cfg = small_cfg(n_tokens=0)
    L = W().make_layer(cfg, seed=4, device=DEV)
    X = W().make_tokens(cfg, seed=4, device=DEV)
    layer = P.Layer.from_workload(L)
    out = P.camera_score_layer(layer, X, 0.95, details=True)
    assert (out["energy"] == 0).all() and (out["phi2"] == 0).all()
    assert_close("omega2", out["omega2"].cpu().numpy(), O.camera_components(to_oracle_layer(L), f64(X))[2])


def test_starved_and_flooded_experts(P):
    """One expert no token reaches, one expert that takes a slot of every token."""
    cfg = small_cfg(n_tokens=600, n_routed=5, top_k=2, d_ff_shared=())
    L = W().make_layer(cfg, seed=5, device=DEV)
    L["router_bias"] = torch.tensor([0.0, -50.0, 0.0, 50.0, 0.0], device=DEV)
    X = W().make_tokens(cfg, seed=5, device=DEV)
    out, _ = run_and_compare(P, L, X, alpha=0.95)
    counts = out["expert_token_counts"].cpu().numpy()
    assert counts[1] == 0 and counts[3] == 600
    assert (out["energy"][128:256] == 0).all()


def test_dense_model_as_single_expert(P):
    """N_E = 1: the paper's dense-model case, as one routed expert and as one shared expert."""
    for n_routed, shared in ((1, ()), (0, (128,))):
        cfg = small_cfg(n_tokens=300, n_routed=n_routed, top_k=1, d_ff_routed=128, d_ff_shared=shared,
                        shared_gate_sigmoid=False, router_bias_std=0.0)
        L = W().make_layer(cfg, seed=6, device=DEV)
        X = W().make_tokens(cfg, seed=6, device=DEV)
        out, _ = run_and_compare(P, L, X, alpha=0.95)
        if n_routed:
            assert (out["topk_w"] == 1).all()


def test_unnormalised_router_and_many_experts(P):
    cfg = small_cfg(n_tokens=500, n_routed=70, top_k=6, d_ff_routed=64, d_ff_shared=(64, 64),
                    shared_gate_sigmoid=False, norm_topk=False)
    L = W().make_layer(cfg, seed=7, device=DEV)
    X = W().make_tokens(cfg, seed=7, device=DEV)
    # 43 tokens per expert on average, raw softmax weights of 70 experts: a score or two, a million times below the
    # largest, may miss 1e-3 of its own value
    run_and_compare(P, L, X, alpha=0.95, max_floor_rescues=2)


def test_fma_kernel_takes_odd_shapes(P):
    """bf16 shapes the tensor-core kernel does not take (d_model, d_ff not multiples of 64)."""
    cfg = small_cfg(d_model=136, d_ff_routed=72, d_ff_shared=(40,), n_tokens=333)
    L = W().make_layer(cfg, seed=8, device=DEV)
    X = W().make_tokens(cfg, seed=8, device=DEV)
    run_and_compare(P, L, X, alpha=0.95)


def test_heavy_tailed_inputs(P):
    cfg = small_cfg(x_dist="student_t4_outliers", n_tokens=900, shared_gate_sigmoid=False)
    L = W().make_layer(cfg, seed=9, device=DEV)
    X = W().make_tokens(cfg, seed=9, device=DEV)
    run_and_compare(P, L, X, alpha=1.0)


def test_bit_reproducible(P):
    cfg = small_cfg(n_tokens=2000)
    L = W().make_layer(cfg, seed=10, device=DEV)
    X = W().make_tokens(cfg, seed=10, device=DEV)
    layer = P.Layer.from_workload(L)
    a = P.camera_score_layer(layer, X, 0.95).clone()
    b = P.camera_score_layer(layer, X, 0.95)
    assert torch.equal(a, b)


@pytest.mark.parametrize("cta_pair", [False, True])
def test_multi_chunk_units(P, cta_pair):
    """Enough tokens per expert that a work unit spans several token tiles and chunks; d_ff values that
    leave a channel tile partly (320 = 2 * 128 + 64) or, for the second CTA of a pair, wholly empty."""
    cfg = small_cfg(n_tokens=6000, n_routed=2, top_k=1, d_ff_routed=320, d_ff_shared=(64,))
    L = W().make_layer(cfg, seed=11, device=DEV)
    X = W().make_tokens(cfg, seed=11, device=DEV)
    run_and_compare(P, L, X, alpha=0.95, cta_pair=cta_pair)


# ------------------------------------------------------------------ argument checks need no kernel to run
def test_argument_errors(P):
    cfg = small_cfg(n_tokens=64)
    L = W().make_layer(cfg, seed=12, device=DEV)
    X = W().make_tokens(cfg, seed=12, device=DEV)
    layer = P.Layer.from_workload(L)
    with pytest.raises(P.CameraError) as e:
        P.camera_score_layer(layer, X, 1.5)
    assert e.value.status == -1
    with pytest.raises(P.CameraError) as e:
        P.camera_score_layer(layer, X, 0.5, workspace=P.alloc_workspace(1024, DEV))
    assert e.value.status == -3
    with pytest.raises(P.CameraError):
        P.camera_select_prune(torch.zeros(10, device=DEV), 1.0)
    with pytest.raises(P.CameraError):
        P.camera_alloc_bits(torch.zeros(10, device=DEV), [0.5, 0.4], [2, 1])


# ------------------------------------------------------------------ selection kernels on their own
def _energies(n, seed, ties=True):
    g = torch.Generator(device="cpu").manual_seed(seed)
    E = torch.rand(n, generator=g) ** 4
    if ties and n > 50:
        E[n // 10: n // 10 + n // 20] = 0.0
        E[n // 2: n // 2 + 7] = E[n // 2]
        E[-3:] = E[0]
    return E


@pytest.mark.parametrize("n", [1, 2, 37, 1000, 4096, 184320])
@pytest.mark.parametrize("ratio", [0.0, 0.2, 0.4, 0.6, 0.97])
def test_select_prune_bit_exact(P, n, ratio):
    E = _energies(n, n)
    keep, thr = P.camera_select_prune(E.to(DEV), ratio, want_threshold=True)
    ref = O.select_prune(E.numpy(), ratio)
    assert np.array_equal(keep.cpu().numpy(), ref)
    assert float(thr[0]) == E.numpy()[ref == 1].min()


def test_select_prune_all_equal(P):
    E = torch.full((5000,), 0.125)
    keep = P.camera_select_prune(E.to(DEV), 0.3)
    assert np.array_equal(keep.cpu().numpy(), O.select_prune(E.numpy(), 0.3))
    assert (keep[:1500] == 0).all() and (keep[1500:] == 1).all()


def test_select_segments_and_expert_counts(P):
    sizes = [4096, 1000, 0, 7777, 3]
    seg = np.concatenate([[0], np.cumsum(sizes)])
    E = _energies(int(seg[-1]), 99)
    exp_off = np.unique(np.concatenate([seg, np.arange(0, seg[-1], 512)]))
    keep, kept = P.camera_select_prune(E.to(DEV), 0.4, seg_offsets=seg.tolist(),
                                       expert_offsets=torch.from_numpy(exp_off).to(DEV))
    ref = np.concatenate([O.select_prune(E.numpy()[seg[s]:seg[s + 1]], 0.4) for s in range(len(sizes))])
    assert np.array_equal(keep.cpu().numpy(), ref)
    assert np.array_equal(kept.cpu().numpy(), [ref[exp_off[i]:exp_off[i + 1]].sum() for i in range(len(exp_off) - 1)])


@pytest.mark.parametrize("n", [5, 1003, 92928])
@pytest.mark.parametrize("scheme", [([0.2, 0.6, 0.2], [3, 2, 1]), ([0.1, 0.8, 0.1], [4, 3, 2]),
                                    ([0.5, 0.0, 0.5], [3, 2, 1]), ([0.25, 0.25, 0.25, 0.25], [8, 4, 3, 2]),
                                    ([1.0, 0.0], [4, 2]), ([0.0, 1.0], [4, 2])])
def test_alloc_bits_bit_exact(P, n, scheme):
    ratios, bits = scheme
    E = _energies(n, 7 * n)
    off = np.unique(np.concatenate([[0, n], np.arange(0, n, 1408)]))
    out, counts = P.camera_alloc_bits(E.to(DEV), ratios, bits, expert_offsets=torch.from_numpy(off).to(DEV))
    ref_bits, ref_cls = O.alloc_bits(E.numpy(), ratios, bits)
    assert np.array_equal(out.cpu().numpy(), ref_bits)
    assert np.array_equal(counts.cpu().numpy(), O.sub_index(ref_cls, off, len(ratios)))


@pytest.mark.parametrize("n", [1, 37, 5000, 184320])
def test_select_all_equals_the_separate_selections(P, n):
    """Several masks and the bit-widths from one set of radix passes: the oracle's results bit for bit (with ties),
    also over segments of unequal length, and with the bit-widths left out."""
    E = _energies(n, 3 * n + 1)
    prune = [0.2, 0.4, 0.6]
    keep, bits = P.camera_select_all(E.to(DEV), prune, [0.2, 0.6, 0.2], [3, 2, 1])
    for j, r in enumerate(prune):
        assert np.array_equal(keep[j].cpu().numpy(), O.select_prune(E.numpy(), r)), f"mask at {r}"
    assert np.array_equal(bits.cpu().numpy(), O.alloc_bits(E.numpy(), [0.2, 0.6, 0.2], [3, 2, 1])[0])
    # four classes and four masks: seven thresholds, the most one call takes; an eighth is refused
    keep4, bits4 = P.camera_select_all(E.to(DEV), [0.0, 0.3, 0.5, 0.97], [0.25, 0.25, 0.25, 0.25], [8, 4, 3, 2])
    for j, r in enumerate([0.0, 0.3, 0.5, 0.97]):
        assert np.array_equal(keep4[j].cpu().numpy(), O.select_prune(E.numpy(), r))
    assert np.array_equal(bits4.cpu().numpy(), O.alloc_bits(E.numpy(), [0.25, 0.25, 0.25, 0.25], [8, 4, 3, 2])[0])
    with pytest.raises(P.CameraError):
        P.camera_select_all(E.to(DEV), [0.1, 0.2, 0.3, 0.4, 0.5], [0.25, 0.25, 0.25, 0.25], [8, 4, 3, 2])
    only, none = P.camera_select_all(E.to(DEV), [0.4])
    assert none is None and np.array_equal(only[0].cpu().numpy(), O.select_prune(E.numpy(), 0.4))


def test_select_all_over_segments(P):
    sizes = [4096, 1000, 0, 7777, 3]
    seg = np.concatenate([[0], np.cumsum(sizes)])
    E = _energies(int(seg[-1]), 98)
    keep, bits = P.camera_select_all(E.to(DEV), [0.2, 0.6], [0.1, 0.8, 0.1], [4, 3, 2], seg_offsets=seg.tolist())
    for j, r in enumerate([0.2, 0.6]):
        ref = np.concatenate([O.select_prune(E.numpy()[seg[s]:seg[s + 1]], r) for s in range(len(sizes))])
        assert np.array_equal(keep[j].cpu().numpy(), ref)
    ref_bits = np.concatenate([O.alloc_bits(E.numpy()[seg[s]:seg[s + 1]], [0.1, 0.8, 0.1], [4, 3, 2])[0] for s in range(len(sizes))])
    assert np.array_equal(bits.cpu().numpy(), ref_bits)


def test_bit_budget_on_gpu(P):
    """The appendix' worked example realised by the allocation: [3,2,1] x [0.1,0.8,0.1] averages 2 bits."""
    E = _energies(12800, 5, ties=False)
    out = P.camera_alloc_bits(E.to(DEV), [0.1, 0.8, 0.1], [3, 2, 1])
    assert float(out.float().mean()) == 2.0
    assert abs(O.average_bits([3, 2, 1], [0.1, 0.8, 0.1], 128, 32) - 2.25) < 1e-12


# ------------------------------------------------------------------ the host-buffer entry point
def test_analyze_layer_host(P):
    cfg = small_cfg(n_tokens=900)
    L = W().make_layer(cfg, seed=13, device=DEV)
    X = W().make_tokens(cfg, seed=13, device=DEV)
    layer = P.Layer.from_workload(L)
    E = P.camera_score_layer(layer, X, 0.95)
    keep = torch.stack([P.camera_select_prune(E, r) for r in (0.2, 0.6)])
    bits = P.camera_alloc_bits(E, [0.2, 0.6, 0.2], [3, 2, 1])
    xh = X.cpu().pin_memory()
    eh = torch.empty(layer.n_me, dtype=torch.float32).pin_memory()
    kh = torch.empty((2, layer.n_me), dtype=torch.uint8).pin_memory()
    bh = torch.empty(layer.n_me, dtype=torch.uint8).pin_memory()
    ws = P.alloc_workspace(P.camera_analyze_workspace_bytes(layer, 900, 3), DEV)
    P.camera_analyze_layer_host(layer, xh, 0.95, [0.2, 0.6], [0.2, 0.6, 0.2], [3, 2, 1], energy_host=eh, keep_host=kh,
                                bits_host=bh, workspace=ws)
    assert torch.equal(eh, E.cpu()) and torch.equal(kh, keep.cpu()) and torch.equal(bh, bits.cpu())


# ------------------------------------------------------------------ the calibration set fed in batches
@pytest.mark.parametrize("kernel", ["umma", "simt"])
def test_accumulate_over_token_batches(P, kernel):
    """Column sums add up and column maxima take the maximum over batches of tokens (Algorithm 1's ColumnSum and ColumnMax):
    three uneven batches must give the scores of the whole set."""
    cfg = small_cfg(n_tokens=2500)
    L = W().make_layer(cfg, seed=14, device=DEV)
    X = W().make_tokens(cfg, seed=14, device=DEV)
    layer = P.Layer.from_workload(L)
    ws = P.alloc_workspace(P.camera_score_workspace_bytes(layer, 1499), DEV)
    phi2 = torch.empty(layer.n_me, dtype=torch.float32, device=DEV)
    phi_inf = torch.empty_like(phi2)
    om = torch.empty_like(phi2)             # the W_down norms: computed with the first batch, given to the later ones
    idx, w = [], []
    out = None
    for b, (t0, t1) in enumerate(((0, 1000), (1000, 1001), (1001, 2500))):
        out = P.camera_score_layer(layer, X[t0:t1].contiguous(), 0.95, details=True, workspace=ws, phi2=phi2,
                                   phi_inf_sq=phi_inf, accumulate=b > 0, omega2=om, omega_given=b > 0,
                                   force_simt=kernel == "simt")
        idx.append(out["topk_idx"].cpu().numpy().astype(np.int64))
        w.append(out["topk_w"].cpu().numpy().astype(np.float64))
    assert P.camera_read_status(ws) == 0
    p2, pinf, w2 = O.camera_components(to_oracle_layer(L), f64(X), routing=(np.concatenate(idx), np.concatenate(w)))
    assert_close("phi2 over batches", phi2.cpu().numpy(), p2)
    assert_close("phi_inf_sq over batches", phi_inf.cpu().numpy(), pinf)
    assert_close("energy over batches", out["energy"].cpu().numpy(), O.energy(p2, pinf, w2, float(np.float32(0.95))))
    whole = P.camera_score_layer(layer, X, 0.95, force_simt=kernel == "simt")
    assert_close("batches vs one call", out["energy"].cpu().numpy(), whole.cpu().numpy(), rel=1e-5)
    with pytest.raises(P.CameraError):      # accumulating needs the running components
        P.camera_score_layer(layer, X[:10].contiguous(), 0.95, accumulate=True)


def test_analyze_layer_host_in_batches(P):
    """More tokens than one host-to-device batch (65536): batches are copied on a second stream while the
    previous one is scored; the result must be that of one call over all tokens."""
    cfg = small_cfg(n_tokens=150001, d_model=128, n_routed=4, d_ff_routed=128, d_ff_shared=(64,))
    L = W().make_layer(cfg, seed=15, device=DEV)
    X = W().make_tokens(cfg, seed=15, device=DEV)
    layer = P.Layer.from_workload(L)
    E = P.camera_score_layer(layer, X, 0.95)
    xh = X.cpu().pin_memory()
    eh = torch.empty(layer.n_me, dtype=torch.float32).pin_memory()
    kh = torch.empty((2, layer.n_me), dtype=torch.uint8).pin_memory()
    bh = torch.empty(layer.n_me, dtype=torch.uint8).pin_memory()
    ws = P.alloc_workspace(P.camera_analyze_workspace_bytes(layer, cfg.n_tokens, 3), DEV)
    first = None
    for _ in range(2):      # the second call reuses the workspace the first one left behind
        eh.zero_()
        P.camera_analyze_layer_host(layer, xh, 0.95, [0.2, 0.6], [0.2, 0.6, 0.2], [3, 2, 1], energy_host=eh,
                                    keep_host=kh, bits_host=bh, workspace=ws)
        assert_close("energy in batches", eh.numpy(), E.cpu().numpy(), rel=1e-5)
        for j, r in enumerate((0.2, 0.6)):
            assert np.array_equal(kh[j].numpy(), O.select_prune(eh.numpy(), r))
        assert np.array_equal(bh.numpy(), O.alloc_bits(eh.numpy(), [0.2, 0.6, 0.2], [3, 2, 1])[0])
        # the batch schedule depends on the sizes alone: every run gives the same bits
        if first is None:
            first = eh.numpy().copy()
        assert np.array_equal(first, eh.numpy())


def test_token_shards_reduced_then_finalised(P):
    """Token-sharded scoring as a multi-GPU run does it: every shard gives its components, sums add and maxima take
    the maximum (the all-reduce), and a call with no tokens and CAMERA_SCORE_ACCUMULATE turns them into energies."""
    cfg = small_cfg(n_tokens=3000)
    L = W().make_layer(cfg, seed=16, device=DEV)
    X = W().make_tokens(cfg, seed=16, device=DEV)
    layer = P.Layer.from_workload(L)
    parts = []
    for t0, t1 in ((0, 1400), (1400, 3000)):
        o = P.camera_score_layer(layer, X[t0:t1].contiguous(), 0.95, details=True)
        parts.append((o["phi2"], o["phi_inf_sq"]))
    phi2 = parts[0][0] + parts[1][0]
    phi_inf = torch.maximum(parts[0][1], parts[1][1])
    E = P.camera_score_layer(layer, X[:0], 0.95, phi2=phi2, phi_inf_sq=phi_inf, accumulate=True)
    whole = P.camera_score_layer(layer, X, 0.95)
    assert_close("sharded vs one call", E.cpu().numpy(), whole.cpu().numpy(), rel=1e-5)


def test_limits_of_the_router(P):
    """The largest expert count and top-k the library takes (256 routed experts, top-16): more logit columns than
    the tensor-core router holds, so the fp32 router runs next to the tensor-core scoring kernel."""
    cfg = small_cfg(n_tokens=300, d_model=128, n_routed=256, top_k=16, d_ff_routed=64, d_ff_shared=(), shared_gate_sigmoid=False,
                    router_bias_std=1.0)
    L = W().make_layer(cfg, seed=17, device=DEV)
    X = W().make_tokens(cfg, seed=17, device=DEV)
    out, _ = run_and_compare(P, L, X, alpha=0.95)
    assert int(out["expert_token_counts"].sum()) == 300 * 16


def test_many_logit_columns_on_the_tensor_core_router(P):
    """112 routed experts + 3 gated shared experts = 128 logit columns, the most the tensor-core router takes."""
    cfg = small_cfg(n_tokens=1000, d_model=192, n_routed=112, top_k=5, d_ff_routed=64, d_ff_shared=(64, 64, 64),
                    shared_gate_sigmoid=True)
    L = W().make_layer(cfg, seed=18, device=DEV)
    X = W().make_tokens(cfg, seed=18, device=DEV)
    # 45 tokens per expert on average: a score or two, a million times below the largest, may miss 1e-3 of its own value
    run_and_compare(P, L, X, alpha=0.95, max_floor_rescues=2)


def test_selection_over_28_layers_at_once(P):
    """All layers of a model as segments of one call: every layer gets its own threshold."""
    n, layers = 184320, 28
    g = torch.Generator(device="cpu").manual_seed(5)
    E = torch.rand(n * layers, generator=g) ** 3 * (1 + torch.arange(n * layers) // n).float()
    seg = [i * n for i in range(layers + 1)]
    keep, thr = P.camera_select_prune(E.to(DEV), 0.4, seg_offsets=seg, want_threshold=True)
    ref = np.concatenate([O.select_prune(E.numpy()[seg[i]:seg[i + 1]], 0.4) for i in range(layers)])
    assert np.array_equal(keep.cpu().numpy(), ref)
    bits = P.camera_alloc_bits(E.to(DEV), [0.2, 0.6, 0.2], [3, 2, 1], seg_offsets=seg)
    refb = np.concatenate([O.alloc_bits(E.numpy()[seg[i]:seg[i + 1]], [0.2, 0.6, 0.2], [3, 2, 1])[0] for i in range(layers)])
    assert np.array_equal(bits.cpu().numpy(), refb)


@pytest.mark.parametrize("prepared", [False, True])
def test_long_token_sets_are_walked_in_batches(P, prepared):
    """More than 65536 tokens in one call: the default walks them in batches of 65536 through the scratch of one batch.
    The result is, bit for bit, that of accumulating calls over the same batches; the routing, the shared-expert
    coefficients and the token counts are those of the single pass; the energies agree with the single pass to the
    rounding of the batches' fp32 sums and with the oracle within the usual tolerance."""
    T = 65536 + 4500
    cfg = small_cfg(n_tokens=T, d_model=128, n_routed=5, top_k=2, d_ff_routed=128, d_ff_shared=(64,))
    L = W().make_layer(cfg, seed=21, device=DEV)
    X = W().make_tokens(cfg, seed=21, device=DEV)
    layer = P.Layer.from_workload(L)
    if prepared:
        P.camera_layer_prepare(layer)
    small, big = P.camera_score_workspace_bytes(layer, T), P.camera_score_workspace_bytes_single_pass(layer, T)
    assert small < big and small == P.camera_score_workspace_bytes(layer, 10 * T)      # stops growing at one batch
    ws = P.alloc_workspace(small, DEV)
    got = P.camera_score_layer(layer, X, 0.95, details=True, workspace=ws)
    assert P.camera_read_status(ws) == 0
    one = P.camera_score_layer(layer, X, 0.95, details=True, single_pass=True)
    for k in ("topk_idx", "topk_w", "shared_w", "expert_token_counts", "omega2"):
        assert torch.equal(got[k], one[k]), k
    assert torch.equal(got["phi_inf_sq"], one["phi_inf_sq"])                            # maxima do not round
    rel = ((got["energy"] - one["energy"]).abs() / one["energy"].clamp_min(1e-30)).max()
    assert float(rel) < 1e-5
    # the same batches by hand
    phi2 = torch.empty(layer.n_me, dtype=torch.float32, device=DEV)
    pinf, om, E = torch.empty_like(phi2), torch.empty_like(phi2), torch.empty_like(phi2)
    for i, (t0, t1) in enumerate([(0, 65536), (65536, T)]):
        P.camera_score_layer(layer, X[t0:t1], 0.95, energy=E, phi2=phi2, phi_inf_sq=pinf, omega2=om, accumulate=i > 0,
                             omega_given=i > 0)
    assert torch.equal(E, got["energy"]) and torch.equal(phi2, got["phi2"])
    # too small a workspace for one pass is refused, not walked
    with pytest.raises(P.CameraError) as e:
        P.camera_score_layer(layer, X, 0.95, workspace=ws, single_pass=True)
    assert e.value.status == -3
    # against the oracle
    ol, Xd = to_oracle_layer(L), f64(X)
    routing = (got["topk_idx"].cpu().numpy().astype(np.int64), got["topk_w"].cpu().numpy().astype(np.float64))
    p2, pi, w2 = O.camera_components(ol, Xd, routing=routing)
    assert_close("energy of a batched walk", got["energy"].cpu().numpy(), O.energy(p2, pi, w2, float(np.float32(0.95))))
    assert_close("phi2 of a batched walk", got["phi2"].cpu().numpy(), p2)


@pytest.mark.parametrize("T", [1, 33, 100, 128, 129])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_decode_sized_batches_at_the_front_end_limits(P, T, dtype):
    """Up to 128 tokens and 128 logit columns take the front end made for decode steps: here with the most columns it
    takes (125 routed experts + 3 gated shared experts), top-16, token counts around a counting-sort block and at the
    limit; 129 tokens go the general way.  Routing, token counts and scores against the oracle."""
    cfg = small_cfg(n_tokens=T, d_model=192, n_routed=125, top_k=16, d_ff_routed=64, d_ff_shared=(64, 64, 64),
                    shared_gate_sigmoid=True, router_bias_std=1.0, dtype=dtype)
    L = W().make_layer(cfg, seed=22, device=DEV)
    X = W().make_tokens(cfg, seed=22, device=DEV)
    out, _ = run_and_compare(P, L, X, alpha=0.95, max_floor_rescues=2)      # one or two tokens per expert
    assert int(out["expert_token_counts"][:125].sum()) == T * 16
    # a repeat on the same inputs gives the same bits (fixed summation order in the logit kernel)
    layer = P.Layer.from_workload(L)
    a = P.camera_score_layer(layer, X, 0.95, details=True)
    assert torch.equal(a["energy"], out["energy"]) and torch.equal(a["topk_idx"], out["topk_idx"])

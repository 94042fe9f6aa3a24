"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each one is chosen so that a
plausible slip in the oracle (a dropped router weight, SiLU with the wrong
sign, W_down indexed by rows instead of columns, max taken before the router
weight is applied, a ratio rounded the other way ...) makes it fail.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle as O
from _util import random_layer

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- SiLU (sigma of Eq. 1)
def test_silu_closed_forms_and_library():
    g = np.array([-30.0, -2.0, -0.5, 0.0, 0.5, 1.0, 2.0, 30.0])
    s = O.silu(g)
    assert s[3] == 0.0
    assert abs(s[5] - 0.7310585786300049) < 1e-15            # 1 * logistic(1)
    assert abs(s[-1] - 30.0) < 1e-11 and abs(s[0]) < 1e-11   # limits
    assert np.allclose(O.silu(g) - O.silu(-g), g, atol=1e-14)  # g*s(g) + g*s(-g) = g
    h = 1e-6
    assert abs((O.silu(np.array([h])) - O.silu(np.array([-h])))[0] / (2 * h) - 0.5) < 1e-9
    ref = torch.nn.functional.silu(torch.from_numpy(g)).numpy()
    assert np.allclose(s, ref, rtol=1e-14, atol=1e-300)


# ---------------------------------------------------------------- router (Alg. 1, Top&Norm)
@pytest.mark.parametrize("norm", [True, False])
def test_router_against_library_softmax_topk(norm):
    r = rng(1)
    layer = random_layer(r, d=7, d_ff=(2,) * 9, top_k=3, bias=True, norm_topk=norm)
    X = r.standard_normal((40, 7))
    p = O.router_probs(layer, X)
    z = torch.from_numpy(X) @ torch.from_numpy(layer.w_router).T + torch.from_numpy(layer.router_bias)
    pt = torch.softmax(z, dim=1)
    assert np.allclose(p, pt.numpy(), rtol=1e-13)
    idx, w = O.top_and_norm(p, 3, norm)
    tv, ti = torch.topk(pt, 3, dim=1)
    assert np.array_equal(idx, ti.numpy())
    if norm:
        tv = tv / tv.sum(dim=1, keepdim=True)
        assert np.allclose(w.sum(axis=1), 1.0, atol=1e-14)
    assert np.allclose(w, tv.numpy(), rtol=1e-13)
    assert (w >= 0).all() and (np.diff(w, axis=1) <= 1e-18).all()


def test_router_ties_go_to_lower_index():
    p = np.array([[0.25, 0.25, 0.25, 0.25], [0.1, 0.4, 0.4, 0.1]])
    idx, w = O.top_and_norm(p, 2, True)
    assert idx.tolist() == [[0, 1], [1, 2]]
    assert np.allclose(w, 0.5)


def test_router_full_k_is_softmax_and_single_expert_is_dense_ffn():
    r = rng(2)
    layer = random_layer(r, d=5, d_ff=(3, 3, 3, 3), top_k=4)
    X = r.standard_normal((11, 5))
    A = O.coefficients(layer, X)
    assert np.allclose(A, O.router_probs(layer, X), rtol=1e-13)
    # N_E = 1, k = 1: A == 1 and the layer is a plain gated FFN (the paper's dense-model case).
    dense = random_layer(r, d=5, d_ff=(8,), top_k=1)
    assert np.array_equal(O.coefficients(dense, X), np.ones((11, 1)))
    xt = torch.from_numpy(X)
    ffn = (torch.nn.functional.silu(xt @ torch.from_numpy(dense.w_gate[0]).T)
           * (xt @ torch.from_numpy(dense.w_up[0]).T)) @ torch.from_numpy(dense.w_down[0]).T
    assert np.allclose(O.forward(dense, X), ffn.numpy(), rtol=1e-12, atol=1e-12)


def test_shared_expert_coefficient():
    r = rng(3)
    X = r.standard_normal((9, 6))
    plain = random_layer(r, d=6, d_ff=(2, 2, 2, 4), n_shared=1, top_k=2)
    assert np.array_equal(O.coefficients(plain, X)[:, 3], np.ones(9))
    gated = random_layer(r, d=6, d_ff=(2, 2, 2, 4), n_shared=1, top_k=2, shared_gate=True)
    sg = torch.sigmoid(torch.from_numpy(X) @ torch.from_numpy(gated.w_shared_gate).T).numpy()
    assert np.allclose(O.coefficients(gated, X)[:, 3:], sg, rtol=1e-13)
    # routed columns hold exactly top_k non-zeros per token
    assert ((O.coefficients(gated, X)[:, :3] != 0).sum(axis=1) == 2).all()


# ---------------------------------------------------------------- P1 decomposition invariant (Eq. 2 == Eq. 5)
@pytest.mark.parametrize("n_shared,gate", [(0, False), (1, False), (2, True)])
def test_decomposition_invariant(n_shared, gate):
    r = rng(10 + n_shared)
    layer = random_layer(r, d=6, d_ff=(3, 5, 4, 2, 3)[: 3 + n_shared], n_shared=n_shared, top_k=2,
                         shared_gate=gate, bias=True)
    X = r.standard_normal((13, 6))
    Y = O.forward(layer, X)
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    assert Phi.shape == (13, sum(layer.d_ff)) and W.shape == (sum(layer.d_ff), 6)
    assert np.allclose(Phi @ W, Y, rtol=1e-12, atol=1e-12)
    # and once more, micro-expert by micro-expert with scalar loops (Eq. 3-5)
    A = O.coefficients(layer, X)
    off = O.me_offsets(layer)
    t = 4
    y = np.zeros(6)
    for e in range(layer.n_experts):
        for i in range(layer.d_ff[e]):
            g = sum(layer.w_gate[e][i, c] * X[t, c] for c in range(6))
            u = sum(layer.w_up[e][i, c] * X[t, c] for c in range(6))
            phi = A[t, e] * O.silu(np.array([g]))[0] * u
            assert abs(phi - Phi[t, off[e] + i]) < 1e-12
            y += phi * layer.w_down[e][:, i]
    assert np.allclose(y, Y[t], rtol=1e-12, atol=1e-12)


def test_forward_matches_library_moe():
    """Eq. 1-2 with torch as the library: dense softmax/top-k routing, expert MLPs."""
    r = rng(20)
    layer = random_layer(r, d=8, d_ff=(4, 4, 4, 4), top_k=2)
    X = r.standard_normal((10, 8))
    xt = torch.from_numpy(X)
    p = torch.softmax(xt @ torch.from_numpy(layer.w_router).T, dim=1)
    tv, ti = torch.topk(p, 2, dim=1)
    tv = tv / tv.sum(dim=1, keepdim=True)
    Y = torch.zeros(10, 8, dtype=torch.float64)
    for t in range(10):
        for s in range(2):
            e = int(ti[t, s])
            h = torch.nn.functional.silu(torch.from_numpy(layer.w_gate[e]) @ xt[t]) * \
                (torch.from_numpy(layer.w_up[e]) @ xt[t])
            Y[t] += tv[t, s] * (torch.from_numpy(layer.w_down[e]) @ h)
    assert np.allclose(O.forward(layer, X), Y.numpy(), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- P2 drop-one brute force == closed form (Eq. 9)
def test_drop_one_error_equals_energy_alpha0():
    r = rng(30)
    layer = random_layer(r, d=5, d_ff=(3, 2, 4, 3), n_shared=1, top_k=2, bias=True)
    X = r.standard_normal((17, 5))
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    phi2, phi_inf, omega2 = O.camera_components(layer, X)
    E0 = O.energy(phi2, phi_inf, omega2, 0.0)
    for i in range(Phi.shape[1]):
        assert math.isclose(O.decode_error(Phi, W, [i]), E0[i], rel_tol=1e-10, abs_tol=1e-14)


def test_components_against_phi_by_loops():
    r = rng(31)
    layer = random_layer(r, d=5, d_ff=(3, 2, 4, 3), n_shared=1, top_k=2, shared_gate=True)
    X = r.standard_normal((12, 5))
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    phi2, phi_inf, omega2 = O.camera_components(layer, X)
    d2, dinf, dw = O.camera_components_dense(layer, X)
    assert np.allclose(phi2, d2, rtol=1e-13) and np.allclose(phi_inf, dinf, rtol=1e-13)
    assert np.allclose(omega2, dw, rtol=1e-13)
    for i in range(Phi.shape[1]):
        col = [Phi[t, i] for t in range(12)]
        assert math.isclose(phi2[i], sum(v * v for v in col), rel_tol=1e-12)
        assert math.isclose(phi_inf[i], max(abs(v) for v in col) ** 2, rel_tol=1e-12)
        assert math.isclose(omega2[i], sum(W[i, c] ** 2 for c in range(5)), rel_tol=1e-12)


# ---------------------------------------------------------------- P3 valid multi-drop bounds
def test_multi_drop_bounds():
    r = rng(32)
    layer = random_layer(r, d=5, d_ff=(3, 3, 3), top_k=2)
    X = r.standard_normal((15, 5))
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    phi2, _, omega2 = O.camera_components(layer, X)
    for m in (2, 3, 4):
        for R in itertools.islice(itertools.combinations(range(9), m), 40):
            R = list(R)
            eps = O.decode_error(Phi, W, R)
            assert eps <= phi2[R].sum() * omega2[R].sum() * (1 + 1e-12)
            assert eps <= m * (phi2[R] * omega2[R]).sum() * (1 + 1e-12)
    # two identical micro-experts: eps = 4 phi^2 w^2, twice the sum of the two energies
    Phi2 = np.concatenate([Phi[:, :1], Phi[:, :1]], axis=1)
    W2 = np.concatenate([W[:1], W[:1]], axis=0)
    e1 = (Phi[:, 0] ** 2).sum() * (W[0] ** 2).sum()
    assert math.isclose(O.decode_error(Phi2, W2, [0, 1]), 4 * e1, rel_tol=1e-12)


# ---------------------------------------------------------------- P4 affine in alpha (Eq. 11 vs Eq. 9)
def test_energy_affine_in_alpha():
    r = rng(33)
    p2, pi, w2 = r.random(50), r.random(50), r.random(50)
    E0, E1 = O.energy(p2, pi, w2, 0.0), O.energy(p2, pi, w2, 1.0)
    assert np.array_equal(E0, p2 * w2) and np.array_equal(E1, pi * w2)
    for a in (0.25, 0.5, 0.95):
        assert np.allclose(O.energy(p2, pi, w2, a), (1 - a) * E0 + a * E1, rtol=1e-14)


# ---------------------------------------------------------------- P5 scaling laws and invariances
def test_single_token_energy_is_alpha_free_and_duplication_law():
    r = rng(34)
    layer = random_layer(r, d=6, d_ff=(4, 4, 4, 4), n_shared=1, top_k=2)
    x1 = r.standard_normal((1, 6))
    p2, pi, w2 = O.camera_components(layer, x1)
    assert np.allclose(p2, pi, rtol=1e-14)
    X = r.standard_normal((9, 6))
    a2, ai, _ = O.camera_components(layer, X)
    b2, bi, _ = O.camera_components(layer, np.concatenate([X, X]))
    assert np.allclose(b2, 2 * a2, rtol=1e-13) and np.allclose(bi, ai, rtol=1e-13)
    perm = r.permutation(9)
    c2, ci, _ = O.camera_components(layer, X[perm])
    assert np.allclose(c2, a2, rtol=1e-13) and np.allclose(ci, ai, rtol=1e-13)


def test_expert_permutation_and_scaling():
    r = rng(35)
    layer = random_layer(r, d=6, d_ff=(3, 5, 4), top_k=2, bias=True)
    X = r.standard_normal((14, 6))
    comps = O.camera_components(layer, X)
    E = O.energy(*comps, 0.5)
    off = O.me_offsets(layer)
    order = [2, 0, 1]
    perm = O.OracleLayer(w_router=layer.w_router[order], top_k=2,
                         w_gate=[layer.w_gate[e] for e in order], w_up=[layer.w_up[e] for e in order],
                         w_down=[layer.w_down[e] for e in order], router_bias=layer.router_bias[order])
    Ep = O.energy(*O.camera_components(perm, X), 0.5)
    expect = np.concatenate([E[off[e]:off[e + 1]] for e in order])
    assert np.allclose(Ep, expect, rtol=1e-12)
    # scaling column i of W_down by c scales E_i by c^2 and nothing else
    layer.w_down[1][:, 2] *= 3.0
    Es = O.energy(*O.camera_components(layer, X), 0.5)
    i = off[1] + 2
    assert math.isclose(Es[i], 9.0 * E[i], rel_tol=1e-12)
    assert np.allclose(np.delete(Es, i), np.delete(E, i), rtol=1e-13)
    layer.w_down[1][:, 2] /= 3.0
    # scaling every router weight by c scales every energy by c^2
    idx, w = O.top_and_norm(O.router_probs(layer, X), 2, True)
    Er = O.energy(*O.camera_components(layer, X, routing=(idx, 0.5 * w)), 0.5)
    assert np.allclose(Er, 0.25 * E, rtol=1e-12)


def test_channel_subset_equals_full():
    r = rng(36)
    layer = random_layer(r, d=6, d_ff=(6, 6, 6, 8), n_shared=1, top_k=2, shared_gate=True)
    X = r.standard_normal((21, 6))
    full = O.camera_components(layer, X)
    ch = {0: [0, 5], 2: [1, 2, 3], 3: [0, 7]}
    sub = O.camera_components(layer, X, channels=ch)
    off = O.me_offsets(layer)
    for e, cs in ch.items():
        for c in cs:
            assert sub[0][off[e] + c] == full[0][off[e] + c]
            assert sub[1][off[e] + c] == full[1][off[e] + c]
    assert np.isnan(sub[0][off[1]:off[2]]).all()
    assert np.array_equal(sub[2], full[2])


def test_unrouted_expert_has_zero_energy():
    r = rng(37)
    layer = random_layer(r, d=4, d_ff=(3, 3, 3), top_k=1)
    layer.router_bias = np.array([0.0, -1e3, 0.0])      # expert 1 never chosen
    X = r.standard_normal((10, 4))
    p2, pi, _ = O.camera_components(layer, X)
    assert (p2[3:6] == 0).all() and (pi[3:6] == 0).all()
    assert (p2[:3] > 0).all()


# ---------------------------------------------------------------- P7 exhaustive subset search (Eq. 7)
def test_camera_vs_exhaustive_cssp():
    r = rng(40)
    layer = random_layer(r, d=6, d_ff=(4, 3, 3), top_k=2)
    X = r.standard_normal((16, 6))
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    E0 = O.energy(*O.camera_components(layer, X), 0.0)
    n = Phi.shape[1]
    for ratio in (0.2, 0.5):
        keep = O.select_prune(E0, ratio)
        removed = [i for i in range(n) if keep[i] == 0]
        assert len(removed) == int(ratio * n)
        best, _ = O.best_subset_error(Phi, W, n - len(removed))
        assert O.decode_error(Phi, W, removed) >= best * (1 - 1e-12)


def test_camera_is_optimal_for_orthogonal_basis():
    r = rng(41)
    d, n = 8, 8
    Q, _ = np.linalg.qr(r.standard_normal((d, d)))
    scale = r.uniform(0.5, 2.0, size=n)
    layer = O.OracleLayer(w_router=r.standard_normal((2, d)), top_k=1,
                          w_gate=[r.standard_normal((4, d)) for _ in range(2)],
                          w_up=[r.standard_normal((4, d)) for _ in range(2)],
                          w_down=[Q[:, :4] * scale[:4], Q[:, 4:] * scale[4:]])
    X = r.standard_normal((30, d))
    Phi, W = O.phi_matrix(layer, X), O.basis(layer)
    E0 = O.energy(*O.camera_components(layer, X), 0.0)
    for m in (3, 5, 6):
        keep = O.select_prune(E0, (n - m) / n)
        removed = [i for i in range(n) if not keep[i]]
        err = O.decode_error(Phi, W, removed)
        assert math.isclose(err, E0[removed].sum(), rel_tol=1e-10)
        best, _ = O.best_subset_error(Phi, W, m)
        assert math.isclose(err, best, rel_tol=1e-10)


# ---------------------------------------------------------------- P8 selection invariants
def test_select_prune_invariants():
    r = rng(50)
    E = r.random(1000)
    E[100:140] = 0.0                       # a block of exact ties at the bottom
    E[500:520] = E[499]                    # and one in the middle
    prev = None
    for ratio in (0.0, 0.03, 0.2, 0.4, 0.6, 0.999):
        keep = O.select_prune(E, ratio)
        npr = int(math.floor(ratio * 1000 + 1e-9))
        assert int((keep == 0).sum()) == npr
        if 0 < npr < 1000:
            assert E[keep == 1].min() >= E[keep == 0].max()
        ref = sorted(range(1000), key=lambda i: (E[i], i))
        expect = np.ones(1000, dtype=np.uint8)
        expect[ref[:npr]] = 0
        assert np.array_equal(keep, expect)
        if prev is not None:
            assert (keep <= prev).all()    # nested masks
        prev = keep
    # ties are pruned lowest index first
    keep = O.select_prune(E, 0.02)
    assert (keep[100:120] == 0).all() and (keep[120:140] == 1).all()


def test_alloc_bits_classes():
    r = rng(51)
    E = r.random(1003)
    E[10:30] = 0.0
    bits, cls = O.alloc_bits(E, [0.2, 0.6, 0.2], [3, 2, 1])
    c = O.class_boundaries([0.2, 0.6, 0.2], 1003)
    assert c == [0, 200, 802, 1003]
    desc = sorted(range(1003), key=lambda i: (E[i], i), reverse=True)
    for j in range(3):
        for i in desc[c[j]:c[j + 1]]:
            assert cls[i] == j and bits[i] == [3, 2, 1][j]
    assert E[cls == 0].min() >= E[cls == 1].max() >= E[cls == 1].min() >= E[cls == 2].max()
    # symmetric scheme: equal top and bottom counts give exactly the middle width on average
    bits2, cls2 = O.alloc_bits(r.random(1000), [0.2, 0.6, 0.2], [4, 3, 2])
    assert (cls2 == 0).sum() == (cls2 == 2).sum() == 200 and bits2.mean() == 3.0
    counts = O.sub_index(cls, np.array([0, 400, 1003]), 3)
    assert counts.sum() == 1003 and counts[0].sum() == 400


# ---------------------------------------------------------------- P9 printed worked example
def test_bit_budget_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "bit_budget_example.txt")) if not l.startswith("#")]
    v = [float(x) for x in rows[0]]
    bits, ratios, group, meta = v[0:3], v[3:6], int(v[6]), int(v[7])
    assert math.isclose(O.average_bits(bits, ratios), v[8], abs_tol=1e-12)
    assert math.isclose(meta / group, v[9])
    assert math.isclose(O.average_bits(bits, ratios, group, meta), v[10], abs_tol=1e-12)
    # the allocation realises that payload on a layer whose size the ratios divide
    b, _ = O.alloc_bits(rng(52).random(1280), ratios, [int(x) for x in bits])
    assert math.isclose(b.mean(), v[8], abs_tol=1e-12)


# ---------------------------------------------------------------- P10 float32 arithmetic stays far inside 1e-3
def test_float32_rerun_within_tolerance():
    r = rng(60)
    d, f, T = 256, 64, 512
    Wg = (r.standard_normal((f, d)) * 0.02).astype(np.float32)
    Wu = (r.standard_normal((f, d)) * 0.02).astype(np.float32)
    X = r.standard_normal((T, d)).astype(np.float32)
    a = r.random(T).astype(np.float32)
    g, u = X @ Wg.T, X @ Wu.T
    lam32 = a[:, None] * (g / (1 + np.exp(-g))) * u
    s32, m32 = (lam32 * lam32).sum(axis=0, dtype=np.float32), np.abs(lam32).max(axis=0) ** 2
    lam64 = a.astype(np.float64)[:, None] * O.expert_hidden(X.astype(np.float64), Wg.astype(np.float64),
                                                          Wu.astype(np.float64))
    s64, m64 = (lam64 * lam64).sum(axis=0), np.abs(lam64).max(axis=0) ** 2
    assert np.abs(s32 / s64 - 1).max() < 1e-4 and np.abs(m32 / m64 - 1).max() < 1e-4


# ---------------------------------------------------------------- GetSubIndex and weight slicing (Alg. 2, Alg. 3)
def test_sliced_layer_decodes_like_the_retained_micro_experts():
    """Slicing W_up[S,:], W_gate[S,:], W_down[:,S] (Alg. 2, the slicing step) must give the layer whose output is
    Phi[:,S] W[S,:], the Y-hat of Eq. 7 -- computed here from the full Phi and W, never from the slices."""
    r = rng(40)
    layer = random_layer(r, d=7, d_ff=(5, 4, 6, 3), n_shared=1, top_k=2, shared_gate=True, bias=True)
    X = r.standard_normal((23, 7))
    off = O.me_offsets(layer)
    E = O.energy(*O.camera_components(layer, X), 0.5)
    keep = O.select_prune(E, 0.4)
    lists, counts = O.sub_index_lists(keep, off, [1])
    assert counts.sum() == keep.sum() and [len(l) for l in lists] == counts[:, 0].tolist()
    S = np.nonzero(keep)[0]
    assert np.array_equal(np.concatenate([off[e] + lists[e] for e in range(4)]), S)       # ascending inside an expert
    Y_hat = O.phi_matrix(layer, X)[:, S] @ O.basis(layer)[S, :]
    assert np.allclose(O.forward(O.slice_layer(layer, lists), X), Y_hat, rtol=1e-12, atol=1e-12)
    # and the error of that layer is the decoding error of the pruned set
    err = ((O.forward(layer, X) - O.forward(O.slice_layer(layer, lists), X)) ** 2).sum()
    assert abs(err - O.decode_error(O.phi_matrix(layer, X), O.basis(layer), np.nonzero(keep == 0)[0])) <= 1e-10 * max(err, 1)


def test_zeroing_pruned_columns_of_w_down_equals_slicing():
    """Phi[:,S] W[S,:] is also Phi times W with the rows outside S set to zero: the full layer with the pruned columns
    of W_down zeroed (gate and up untouched) gives the sliced layer's output.  The GPU's pruned-output call rests on it."""
    import copy
    r = rng(42)
    layer = random_layer(r, d=6, d_ff=(5, 7, 4), n_shared=1, top_k=2, shared_gate=True)
    X = r.standard_normal((19, 6))
    off = O.me_offsets(layer)
    keep = O.select_prune(O.energy(*O.camera_components(layer, X), 0.95), 0.5)
    keep[off[1]:off[2]] = 0                                   # an expert that loses everything
    lists, _ = O.sub_index_lists(keep, off, [1])
    masked = copy.deepcopy(layer)
    masked.w_down = [layer.w_down[e] * keep[off[e]:off[e + 1]][None, :] for e in range(len(layer.w_down))]
    assert np.allclose(O.forward(masked, X), O.forward(O.slice_layer(layer, lists), X), rtol=1e-12, atol=1e-12)
    S = np.nonzero(keep)[0]
    assert np.allclose(O.forward(masked, X), O.phi_matrix(layer, X)[:, S] @ O.basis(layer)[S, :], rtol=1e-12, atol=1e-12)


def test_reordering_by_class_keeps_the_layer_and_colocates_classes():
    r = rng(41)
    layer = random_layer(r, d=6, d_ff=(8, 5, 7), n_shared=0, top_k=2)
    X = r.standard_normal((17, 6))
    off = O.me_offsets(layer)
    E = O.energy(*O.camera_components(layer, X), 0.95)
    _, cls = O.alloc_bits(E, [0.25, 0.5, 0.25], [4, 3, 2])
    lists, counts = O.sub_index_lists(cls, off, [0, 1, 2])
    assert np.array_equal(counts, O.sub_index(cls, off, 3))
    for e in range(3):
        assert sorted(lists[e].tolist()) == list(range(layer.d_ff[e]))                     # a permutation
        seg = cls[off[e]:off[e + 1]][lists[e]]
        assert (np.diff(seg.astype(int)) >= 0).all()                                       # classes contiguous, in order
        for j in range(3):                                                                 # stable inside a class
            part = lists[e][seg == j]
            assert (np.diff(part) > 0).all()
    assert np.allclose(O.forward(O.slice_layer(layer, lists), X), O.forward(layer, X), rtol=1e-12, atol=1e-12)
    # brute force: the same lists from a stable sort by (class, channel)
    for e in range(3):
        seg = cls[off[e]:off[e + 1]]
        assert lists[e].tolist() == sorted(range(len(seg)), key=lambda i: (int(seg[i]), i))


def test_sub_index_leaves_out_other_labels_and_handles_empty_experts():
    labels = np.array([1, 0, 1, 1, 0, 0, 0, 1, 0], dtype=np.uint8)
    lists, counts = O.sub_index_lists(labels, np.array([0, 4, 4, 7, 9]), [1])
    assert [l.tolist() for l in lists] == [[0, 2, 3], [], [], [0]]
    assert counts[:, 0].tolist() == [3, 0, 0, 1]


def test_next_layer_input_is_the_unit_rms_residual():
    r = rng(42)
    X, Y = r.standard_normal((9, 16)), r.standard_normal((9, 16)) * 3
    Z = O.next_layer_input(X, Y, eps=0.0)
    assert np.allclose((Z * Z).mean(axis=1), 1.0, atol=1e-12)                  # RMS 1 per token
    assert np.allclose(Z * np.sqrt(((X + Y) ** 2).mean(axis=1, keepdims=True)), X + Y, atol=1e-12)   # same direction as x + y
    assert np.allclose(O.next_layer_input(2 * X, 2 * Y, eps=0.0), Z, atol=1e-12)   # scale invariant
    ref = torch.nn.functional.rms_norm(torch.from_numpy(X + Y), (16,), eps=1e-6).numpy()
    assert np.allclose(O.next_layer_input(X, Y, eps=1e-6), ref, rtol=1e-12)

"""CAMERA micro-expert redundancy analysis, written out in float64 numpy.

TEST INFRASTRUCTURE ONLY: a slow, plain, obviously-correct statement of what
the paper's Algorithm 1 (micro-expert ranking), the selection step of
Algorithm 2 (CAMERA-P) and the split step of Algorithm 3 (CAMERA-Q) compute.
Nothing here is blocked, fused or reordered beyond what the paper states, and
nothing here is shared with the CUDA path.

Conventions (paper, Section "From Expert to Micro-Expert"):
  * an expert is  E(x) = W_down [ SiLU(W_gate x) * (W_up x) ]           (Eq. 1)
    with W_gate, W_up of shape [d_ff, d_model] and W_down of shape
    [d_model, d_ff];
  * micro-expert i of that expert is row i of W_gate and W_up together with
    column i of W_down                                                   (Eq. 3);
  * experts are ordered routed[0..n_routed) then shared[0..n_shared); the
    global micro-expert index is offset[e] + i with offset the prefix sum of
    the experts' d_ff (Algorithm 1's global index, generalised to unequal d_ff).

Every input array is float64 and holds the *storage-rounded* values (a bf16
tensor widened exactly), so the only difference to the CUDA path is the
arithmetic itself.

Pinning status: every function below is pinned by the CPU test-suite
(decomposition invariant, drop-one closed form, brute-force subset search on
tiny layers, affine-in-alpha and scaling laws, the paper's printed bit-budget
example).  The one thing with no pin is absolute scores / rankings / masks on
the paper's trained models, which the paper never prints: parity unpinned
for those, and they are not computed here.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

__all__ = [
    "OracleLayer", "silu", "router_probs", "top_and_norm", "shared_coeff",
    "coefficients", "expert_hidden", "forward", "phi_matrix", "basis",
    "me_offsets", "camera_components_dense", "camera_components", "energy",
    "camera_rank", "n_pruned", "select_prune", "class_boundaries",
    "alloc_bits", "sub_index", "sub_index_lists", "slice_layer", "next_layer_input", "decode_error", "best_subset_error",
    "average_bits",
]


@dataclass
class OracleLayer:
    """One MoE layer in the paper's layout, all arrays float64.

    w_router      [n_routed, d_model]   router R (Algorithm 1 input)
    router_bias   [n_routed] or None    added to the logits before softmax
    top_k         number of routed experts per token
    norm_topk     divide the k kept probabilities by their sum ("Top&Norm")
    w_gate, w_up  lists over experts of [d_ff_e, d_model]
    w_down        list over experts of [d_model, d_ff_e] (column i = w_i)
    n_shared      the last n_shared experts see every token
    w_shared_gate [n_shared, d_model] or None; None means coefficient 1,
                  otherwise the coefficient is sigmoid(x . w_shared_gate[s])
    """
    w_router: np.ndarray
    top_k: int
    w_gate: List[np.ndarray]
    w_up: List[np.ndarray]
    w_down: List[np.ndarray]
    router_bias: Optional[np.ndarray] = None
    norm_topk: bool = True
    n_shared: int = 0
    w_shared_gate: Optional[np.ndarray] = None

    @property
    def n_experts(self) -> int:
        return len(self.w_gate)

    @property
    def n_routed(self) -> int:
        return self.n_experts - self.n_shared

    @property
    def d_ff(self) -> List[int]:
        return [int(w.shape[0]) for w in self.w_gate]


def silu(g: np.ndarray) -> np.ndarray:
    """sigma in Eq. 1: SiLU(g) = g / (1 + exp(-g))."""
    return g / (1.0 + np.exp(-g))


def me_offsets(layer: OracleLayer) -> np.ndarray:
    """Start of each expert's micro-experts in the global index (the global index of Alg. 1)."""
    return np.concatenate([[0], np.cumsum(layer.d_ff)]).astype(np.int64)


# ----------------------------------------------------------------------------
# Router: A <- Top&Norm(R X)                                   (Alg. 1, Top&Norm)
# ----------------------------------------------------------------------------
def router_probs(layer: OracleLayer, X: np.ndarray) -> np.ndarray:
    """softmax over the routed experts of z = X R^T (+ bias); shape [T, n_routed]."""
    z = X @ layer.w_router.T
    if layer.router_bias is not None:
        z = z + layer.router_bias[None, :]
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=1, keepdims=True)


def top_and_norm(p: np.ndarray, k: int, norm: bool) -> Tuple[np.ndarray, np.ndarray]:
    """Keep the k largest probabilities of every row (ties: lower index first).

    Returns (idx [T,k] int64 in order of decreasing probability, w [T,k]).
    With norm the kept weights are divided by their sum.
    """
    idx = np.argsort(-p, axis=1, kind="stable")[:, :k]
    w = np.take_along_axis(p, idx, axis=1)
    if norm:
        w = w / w.sum(axis=1, keepdims=True)
    return idx.astype(np.int64), w


def shared_coeff(layer: OracleLayer, X: np.ndarray) -> np.ndarray:
    """Coefficient of the shared experts: 1, or sigmoid(x . w_sg); shape [T, n_shared]."""
    T = X.shape[0]
    if layer.n_shared == 0:
        return np.zeros((T, 0))
    if layer.w_shared_gate is None:
        return np.ones((T, layer.n_shared))
    return 1.0 / (1.0 + np.exp(-(X @ layer.w_shared_gate.T)))


def coefficients(layer: OracleLayer, X: np.ndarray,
                 routing: Optional[Tuple[np.ndarray, np.ndarray]] = None) -> np.ndarray:
    """The router matrix A of Eq. 2 as a dense [T, n_experts] array (zeros where
    a token is not routed to an expert).  `routing` = (idx, w) overrides the
    routed part (used to score under a prescribed routing)."""
    T = X.shape[0]
    A = np.zeros((T, layer.n_experts))
    if layer.n_routed > 0:
        if routing is None:
            idx, w = top_and_norm(router_probs(layer, X), layer.top_k, layer.norm_topk)
        else:
            idx, w = routing
        rows = np.repeat(np.arange(T), idx.shape[1])
        A[rows, np.asarray(idx).reshape(-1)] = np.asarray(w, dtype=np.float64).reshape(-1)
    if layer.n_shared:
        A[:, layer.n_routed:] = shared_coeff(layer, X)
    return A


# ----------------------------------------------------------------------------
# Experts, the ordinary forward (Eq. 1-2) and the micro-expert form (Eq. 4-5)
# ----------------------------------------------------------------------------
def expert_hidden(X: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray) -> np.ndarray:
    """SiLU(W_gate x) * (W_up x) for every row x of X; shape [T, d_ff]."""
    return silu(X @ w_gate.T) * (X @ w_up.T)


def forward(layer: OracleLayer, X: np.ndarray) -> np.ndarray:
    """y = sum_e A_e(x) W_down_e [SiLU(W_gate_e x) * W_up_e x]   (Eq. 1-2), the
    ordinary expert-by-expert evaluation.  Shape [T, d_model]."""
    A = coefficients(layer, X)
    Y = np.zeros((X.shape[0], X.shape[1]))
    for e in range(layer.n_experts):
        Y += A[:, e:e + 1] * (expert_hidden(X, layer.w_gate[e], layer.w_up[e]) @ layer.w_down[e].T)
    return Y


def phi_matrix(layer: OracleLayer, X: np.ndarray) -> np.ndarray:
    """Activation-coefficient matrix Phi [T, N_e]: phi_{t,i} = a_i(x_t) SiLU(w_i^gate x_t) w_i^up x_t
    (Eq. 4).  Only for small layers: the method itself never forms Phi."""
    A = coefficients(layer, X)
    cols = [A[:, e:e + 1] * expert_hidden(X, layer.w_gate[e], layer.w_up[e])
            for e in range(layer.n_experts)]
    return np.concatenate(cols, axis=1)


def basis(layer: OracleLayer) -> np.ndarray:
    """Basis-vector matrix W [N_e, d_model]: row i is w_i, column i of its W_down."""
    return np.concatenate([w.T for w in layer.w_down], axis=0)


# ----------------------------------------------------------------------------
# Algorithm 1: phi^2, phi^inf, omega^2 and the energy (Eq. 11)
# ----------------------------------------------------------------------------
def camera_components_dense(layer: OracleLayer, X: np.ndarray):
    """Algorithm 1 up to the components, taken literally: Lambda is formed over *all* n
    tokens with the dense column A[:, e].  Returns (phi2, phi_inf_sq, omega2),
    each of length N_e."""
    A = coefficients(layer, X)
    phi2, phi_inf, omega2 = [], [], []
    for e in range(layer.n_experts):
        omega2.append((layer.w_down[e] * layer.w_down[e]).sum(axis=0))        # omega
        Lam = A[:, e:e + 1] * expert_hidden(X, layer.w_gate[e], layer.w_up[e])  # Lambda
        phi2.append((Lam * Lam).sum(axis=0))                                   # ColumnSum
        phi_inf.append(np.abs(Lam).max(axis=0) ** 2 if Lam.shape[0] else np.zeros(Lam.shape[1]))  # ColumnMax
    return np.concatenate(phi2), np.concatenate(phi_inf), np.concatenate(omega2)


def camera_components(layer: OracleLayer, X: np.ndarray,
                      channels: Optional[Dict[int, Sequence[int]]] = None,
                      routing: Optional[Tuple[np.ndarray, np.ndarray]] = None):
    """Same quantities as `camera_components_dense`, but each expert only
    visits the tokens whose coefficient is non-zero (rows with A = 0 add 0 to
    a column sum and cannot raise a column max of absolute values).

    `channels` optionally restricts the work to a subset of micro-experts:
    {expert: sorted channel indices}.  The returned arrays then hold NaN for
    phi2 / phi_inf_sq of every micro-expert not listed (omega2 is always full).
    """
    T = X.shape[0]
    off = me_offsets(layer)
    n_e = int(off[-1])
    phi2 = np.full(n_e, np.nan)
    phi_inf = np.full(n_e, np.nan)
    omega2 = np.empty(n_e)
    if layer.n_routed > 0:
        if routing is None:
            idx, w = top_and_norm(router_probs(layer, X), layer.top_k, layer.norm_topk)
        else:
            idx, w = np.asarray(routing[0]), np.asarray(routing[1], dtype=np.float64)
    sc = shared_coeff(layer, X)
    for e in range(layer.n_experts):
        omega2[off[e]:off[e + 1]] = (layer.w_down[e] * layer.w_down[e]).sum(axis=0)
        if channels is not None and e not in channels:
            continue
        ch = np.arange(layer.d_ff[e]) if channels is None else np.asarray(channels[e], dtype=np.int64)
        if e < layer.n_routed:
            hit = (idx == e)
            tok = np.nonzero(hit.any(axis=1))[0]
            a = (w * hit).sum(axis=1)[tok]
        else:
            tok = np.arange(T)
            a = sc[:, e - layer.n_routed]
        nz = a != 0.0
        tok, a = tok[nz], a[nz]
        if tok.size == 0:
            phi2[off[e] + ch] = 0.0
            phi_inf[off[e] + ch] = 0.0
            continue
        w_gate = layer.w_gate[e] if channels is None else layer.w_gate[e][ch]
        w_up = layer.w_up[e] if channels is None else layer.w_up[e][ch]
        Lam = a[:, None] * expert_hidden(X[tok], w_gate, w_up)
        phi2[off[e] + ch] = (Lam * Lam).sum(axis=0)
        phi_inf[off[e] + ch] = np.abs(Lam).max(axis=0) ** 2
    return phi2, phi_inf, omega2


def energy(phi2: np.ndarray, phi_inf_sq: np.ndarray, omega2: np.ndarray, alpha: float) -> np.ndarray:
    """E_i = [(1 - alpha) ||Phi_i||_2^2 + alpha ||Phi_i||_inf^2] ||w_i||_2^2   (Eq. 11, the energy step of Alg. 1)."""
    return ((1.0 - alpha) * phi2 + alpha * phi_inf_sq) * omega2


def camera_rank(E: np.ndarray) -> np.ndarray:
    """The Argsort step of Alg. 1: all micro-experts from least to most important
    (energy ascending, lower index first among equal energies)."""
    return np.argsort(E, kind="stable")


# ----------------------------------------------------------------------------
# Selection: CAMERA-P keep mask (Alg. 2, TopSelect), CAMERA-Q classes (Alg. 3, ListSplitByRatio / GetSubIndex)
# ----------------------------------------------------------------------------
def _floor_count(ratio: float, n: int) -> int:
    return int(math.floor(ratio * float(n) + 1e-9))


def n_pruned(ratio: float, n: int) -> int:
    """Number of micro-experts removed at pruning ratio lambda: floor(lambda * N_e)."""
    return _floor_count(ratio, n)


def select_prune(E: np.ndarray, ratio: float) -> np.ndarray:
    """S <- TopSelect(R, 1 - lambda): uint8 mask, 1 = retained.  The
    floor(lambda N_e) lowest-energy micro-experts of the layer are removed,
    whatever expert they belong to."""
    keep = np.ones(E.shape[0], dtype=np.uint8)
    keep[camera_rank(E)[:n_pruned(ratio, E.shape[0])]] = 0
    return keep


def class_boundaries(ratios: Sequence[float], n: int) -> List[int]:
    """Cumulative class sizes c_0 = 0 <= c_1 <= ... <= c_L = n with
    c_j = floor((r_1 + ... + r_j) n); the last class takes the remainder."""
    c = [0]
    acc = 0.0
    for r in ratios[:-1]:
        acc += r
        c.append(_floor_count(acc, n))
    c.append(n)
    return c


def alloc_bits(E: np.ndarray, ratios: Sequence[float], bits: Sequence[int]):
    """S_1..S_L <- ListSplitByRatio(R, r_1..r_L) with the most important
    micro-experts first, then bit-width b_j for class j.  Returns
    (bits_per_micro_expert uint8 [N_e], class_id uint8 [N_e])."""
    n = E.shape[0]
    desc = camera_rank(E)[::-1]          # most important first
    c = class_boundaries(ratios, n)
    cls = np.empty(n, dtype=np.uint8)
    for j in range(len(ratios)):
        cls[desc[c[j]:c[j + 1]]] = j
    return np.asarray(bits, dtype=np.uint8)[cls], cls


def sub_index(cls_or_mask: np.ndarray, offsets: np.ndarray, n_classes: int) -> np.ndarray:
    """GetSubIndex reduced to counts: how many micro-experts of each expert
    fall into each class; shape [n_experts, n_classes]."""
    out = np.zeros((len(offsets) - 1, n_classes), dtype=np.int64)
    for e in range(len(offsets) - 1):
        seg = cls_or_mask[offsets[e]:offsets[e + 1]]
        for j in range(n_classes):
            out[e, j] = int((seg == j).sum())
    return out


def sub_index_lists(labels: np.ndarray, offsets: np.ndarray, order: Sequence[int]):
    """GetSubIndex (Algorithm 3; the per-expert retained sets of Algorithm 2).

    For every expert, its micro-experts (channel numbers inside the expert)
    listed label by label in the given `order` of label values, ascending
    channel inside a label; micro-experts whose label is not in `order` are
    left out.  Returns (lists, counts): lists[e] is an int64 array, counts is
    [n_experts, len(order)].  With labels = keep mask and order = [1] this is
    the retained set S of each expert; with labels = precision class and
    order = all classes it is the reordering that colocates micro-experts of
    equal precision (Section "CAMERA-Q")."""
    lists, counts = [], np.zeros((len(offsets) - 1, len(order)), dtype=np.int64)
    for e in range(len(offsets) - 1):
        seg = np.asarray(labels[offsets[e]:offsets[e + 1]])
        parts = []
        for j, v in enumerate(order):
            ch = np.nonzero(seg == v)[0]
            counts[e, j] = ch.size
            parts.append(ch)
        lists.append(np.concatenate(parts).astype(np.int64) if parts else np.zeros(0, dtype=np.int64))
    return lists, counts


def slice_layer(layer: OracleLayer, lists: Sequence[np.ndarray]) -> OracleLayer:
    """The slicing step of Algorithm 2: W_up <- W_up[S,:], W_gate <- W_gate[S,:],
    W_down <- W_down[:,S] for every expert, S given as channel lists (any
    order; a permutation of all channels merely reorders the micro-experts)."""
    return OracleLayer(
        w_router=layer.w_router, top_k=layer.top_k,
        w_gate=[w[np.asarray(ix, dtype=np.int64)] for w, ix in zip(layer.w_gate, lists)],
        w_up=[w[np.asarray(ix, dtype=np.int64)] for w, ix in zip(layer.w_up, lists)],
        w_down=[w[:, np.asarray(ix, dtype=np.int64)] for w, ix in zip(layer.w_down, lists)],
        router_bias=layer.router_bias, norm_topk=layer.norm_topk, n_shared=layer.n_shared,
        w_shared_gate=layer.w_shared_gate)


def next_layer_input(X: np.ndarray, Y: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """Glue of the synthetic multi-layer stack (NO counterpart in the paper, whose
    layers are whole decoder layers of a trained model): the next layer's input
    is the residual sum x + y of a token, rescaled to root-mean-square 1.  It
    stands in for "I <- O" of Algorithm 2 where no attention block,
    norm weights or trained model exist."""
    Z = X + Y
    return Z / np.sqrt((Z * Z).mean(axis=1, keepdims=True) + eps)


# ----------------------------------------------------------------------------
# Helpers for the pins: decoding error and exhaustive subset search (Eq. 7)
# ----------------------------------------------------------------------------
def decode_error(Phi: np.ndarray, W: np.ndarray, removed: Sequence[int]) -> float:
    """||Y - Phi_{:,S} W_{S,:}||_F^2 computed the long way: build Y from every
    micro-expert, build Y_hat from the retained ones, subtract."""
    removed = set(int(i) for i in removed)
    keep = [i for i in range(Phi.shape[1]) if i not in removed]
    Y = Phi @ W
    Y_hat = Phi[:, keep] @ W[keep, :]
    return float(((Y - Y_hat) ** 2).sum())


def best_subset_error(Phi: np.ndarray, W: np.ndarray, m: int) -> Tuple[float, Tuple[int, ...]]:
    """Exact solution of Eq. 7 by trying every retained set of size m."""
    n = Phi.shape[1]
    best = (math.inf, ())
    for S in itertools.combinations(range(n), m):
        err = decode_error(Phi, W, [i for i in range(n) if i not in S])
        if err < best[0]:
            best = (err, S)
    return best


def average_bits(bits: Sequence[int], ratios: Sequence[float], group: int = 0, meta_bits: int = 0) -> float:
    """Average storage cost per weight of a mixed-precision split: the
    ratio-weighted payload plus meta_bits of scale/zero-point per `group`
    weights (appendix "Mixed-precision Settings in CAMERA-Q")."""
    payload = sum(b * r for b, r in zip(bits, ratios))
    return payload + (meta_bits / group if group else 0.0)

"""ctypes binding of libcamera_b200.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/camera.h).  PyTorch is
used for device memory and streams; all arithmetic happens in the CUDA library.  There is no
fallback: if the shared library cannot be built or loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

from . import build as _build

CAMERA_OK = 0
CAMERA_F32, CAMERA_BF16 = 0, 1
CAMERA_DOWN_HF, CAMERA_DOWN_ME_MAJOR = 0, 1
CAMERA_ROUTER_NORM_TOPK, CAMERA_SHARED_GATE_SIGMOID = 1, 2
CAMERA_SCORE_FORCE_SIMT = 1
CAMERA_SCORE_CTA_PAIR = 2
CAMERA_SCORE_ACCUMULATE = 4
CAMERA_SCORE_SINGLE_CTA = 8
CAMERA_FORWARD_TOKEN_ROWS = 16
CAMERA_SCORE_OMEGA_GIVEN = 32
CAMERA_SCORE_SINGLE_PASS = 64
STAGES = ("router", "permute", "rownorm", "score", "combine")


class camera_layer_t(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_routed", C.c_int32), ("top_k", C.c_int32), ("n_shared", C.c_int32),
                ("d_ff", C.POINTER(C.c_int32)), ("dtype", C.c_int32), ("flags", C.c_uint32),
                ("down_layout", C.c_int32), ("w_router", C.c_void_p), ("router_bias", C.c_void_p),
                ("w_shared_gate", C.c_void_p), ("w_gate", C.POINTER(C.c_void_p)),
                ("w_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
                ("w_down_ld", C.POINTER(C.c_int32)), ("prepared", C.c_void_p)]


class camera_score_aux_t(C.Structure):
    _fields_ = [("phi2", C.c_void_p), ("phi_inf_sq", C.c_void_p), ("omega2", C.c_void_p),
                ("topk_idx", C.c_void_p), ("topk_w", C.c_void_p), ("topk_idx_in", C.c_void_p),
                ("topk_w_in", C.c_void_p), ("shared_w", C.c_void_p), ("expert_token_counts", C.c_void_p),
                ("flags", C.c_uint32), ("stage_events", C.c_void_p * 10)]


def _load() -> C.CDLL:
    path = _build.LIB
    if _build.needs_build():
        _build.build()
    if not os.path.exists(path):
        raise ImportError("libcamera_b200.so is missing and could not be built; there is no fallback path")
    lib = C.CDLL(path)
    lib.camera_strerror.restype = C.c_char_p
    lib.camera_strerror.argtypes = [C.c_int]
    lib.camera_version.restype = C.c_int
    lib.camera_score_workspace_bytes.restype = C.c_size_t
    lib.camera_score_workspace_bytes.argtypes = [C.POINTER(camera_layer_t), C.c_int64]
    lib.camera_score_workspace_bytes_single_pass.restype = C.c_size_t
    lib.camera_score_workspace_bytes_single_pass.argtypes = [C.POINTER(camera_layer_t), C.c_int64]
    lib.camera_score_layer.restype = C.c_int
    lib.camera_score_layer.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_int64, C.c_float, C.c_void_p,
                                       C.POINTER(camera_score_aux_t), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.camera_layer_prepared_bytes.restype = C.c_size_t
    lib.camera_layer_prepared_bytes.argtypes = [C.POINTER(camera_layer_t)]
    lib.camera_layer_prepare.restype = C.c_int
    lib.camera_layer_prepare.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
    lib.camera_layer_release.restype = None
    lib.camera_layer_release.argtypes = [C.c_void_p]
    lib.camera_read_status.restype = C.c_int
    lib.camera_read_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.camera_set_wait_limit_ns.restype = C.c_int
    lib.camera_set_wait_limit_ns.argtypes = [C.c_uint64]
    lib.camera_get_wait_limit_ns.restype = C.c_uint64
    lib.camera_get_wait_limit_ns.argtypes = []
    lib.camera_wait_probe.restype = C.c_int
    lib.camera_wait_probe.argtypes = [C.c_void_p, C.c_size_t, C.c_uint64, C.c_void_p]
    lib.camera_select_workspace_bytes.restype = C.c_size_t
    lib.camera_select_workspace_bytes.argtypes = [C.c_int64, C.c_int32, C.c_int32]
    lib.camera_select_prune.restype = C.c_int
    lib.camera_select_prune.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int32, C.c_double, C.c_void_p,
                                        C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
    lib.camera_alloc_bits.restype = C.c_int
    lib.camera_alloc_bits.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int32, C.POINTER(C.c_double),
                                      C.POINTER(C.c_int32), C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.camera_select_prune_static.restype = C.c_int
    lib.camera_select_prune_static.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int32, C.c_double, C.c_void_p,
                                               C.c_void_p, C.c_void_p]
    lib.camera_analyze_workspace_bytes.restype = C.c_size_t
    lib.camera_analyze_workspace_bytes.argtypes = [C.POINTER(camera_layer_t), C.c_int64, C.c_int32]
    lib.camera_analyze_layer_host.restype = C.c_int
    lib.camera_analyze_layer_host.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_int64, C.c_float,
                                              C.POINTER(C.c_double), C.c_int32,
                                              C.POINTER(C.c_double), C.POINTER(C.c_int32), C.c_int32,
                                              C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                              C.c_void_p]
    lib.camera_forward_workspace_bytes.restype = C.c_size_t
    lib.camera_forward_workspace_bytes.argtypes = [C.POINTER(camera_layer_t), C.c_int64]
    lib.camera_layer_forward.restype = C.c_int
    lib.camera_layer_forward.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_int64, C.c_void_p,
                                         C.POINTER(camera_score_aux_t), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.camera_score_forward_layer.restype = C.c_int
    lib.camera_score_forward_layer.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_int64, C.c_float, C.c_void_p,
                                               C.c_void_p, C.POINTER(camera_score_aux_t), C.c_void_p, C.c_size_t,
                                               C.c_void_p]
    lib.camera_select_all.restype = C.c_int
    lib.camera_select_all.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int32, C.POINTER(C.c_double), C.c_int32,
                                      C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int32), C.c_int32, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]
    lib.camera_mask_down_columns.restype = C.c_int
    lib.camera_mask_down_columns.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p]
    lib.camera_pruned_output.restype = C.c_int
    lib.camera_pruned_output.argtypes = [C.POINTER(camera_layer_t), C.POINTER(C.c_void_p), C.c_int64, C.c_void_p,
                                         C.POINTER(camera_score_aux_t), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.camera_output_error_workspace_bytes.restype = C.c_size_t
    lib.camera_output_error_workspace_bytes.argtypes = [C.c_int64]
    lib.camera_output_error.restype = C.c_int
    lib.camera_output_error.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
    lib.camera_residual_norm.restype = C.c_int
    lib.camera_residual_norm.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_int32, C.c_float, C.c_void_p,
                                         C.c_void_p]
    lib.camera_sub_index.restype = C.c_int
    lib.camera_sub_index.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.c_void_p,
                                     C.c_void_p, C.c_void_p]
    lib.camera_compact_workspace_bytes.restype = C.c_size_t
    lib.camera_compact_workspace_bytes.argtypes = [C.c_int32]
    lib.camera_compact_weights.restype = C.c_int
    lib.camera_compact_weights.argtypes = [C.POINTER(camera_layer_t), C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                           C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p),
                                           C.POINTER(C.c_int32), C.c_void_p, C.c_size_t, C.c_void_p]
    return lib


lib = _load()


class CameraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.camera_strerror(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != CAMERA_OK:
        raise CameraError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


class Layer:
    """Holds the tensors of one MoE layer and the camera_layer_t that points at them.

    w_gate / w_up: lists of [d_ff_e, d_model]; w_down: list of [d_model, d_ff_e] (down_layout "hf")
    or [d_ff_e, d_model] ("me_major"); experts ordered routed first, then shared.
    """

    def __init__(self, w_router, w_gate: Sequence[torch.Tensor], w_up, w_down, top_k: int, n_shared: int = 0,
                 router_bias=None, w_shared_gate=None, norm_topk: bool = True, down_layout: str = "hf",
                 down_ld: Optional[Sequence[int]] = None):
        self.tensors = dict(w_router=w_router, router_bias=router_bias, w_shared_gate=w_shared_gate,
                            w_gate=list(w_gate), w_up=list(w_up), w_down=list(w_down))
        ref = w_gate[0]
        for t in list(w_gate) + list(w_up) + list(w_down) + [t for t in (w_router, w_shared_gate) if t is not None]:
            if not (t.is_contiguous() and t.dtype == ref.dtype and t.device == ref.device):
                raise ValueError("layer tensors must be contiguous and share dtype and device")
        if router_bias is not None and router_bias.dtype != torch.float32:
            raise ValueError("router_bias must be float32")
        self.dtype = ref.dtype
        self.device = ref.device
        n = len(w_gate)
        self.n_experts = n
        self.d_model = int(ref.shape[1])
        self.d_ff = [int(w.shape[0]) for w in w_gate]
        self.n_me = sum(self.d_ff)
        self.n_routed = n - n_shared
        self._d_ff = (C.c_int32 * n)(*self.d_ff)
        self._wg = (C.c_void_p * n)(*[w.data_ptr() for w in w_gate])
        self._wu = (C.c_void_p * n)(*[w.data_ptr() for w in w_up])
        self._wd = (C.c_void_p * n)(*[w.data_ptr() for w in w_down])
        flags = (CAMERA_ROUTER_NORM_TOPK if norm_topk else 0) | \
                (CAMERA_SHARED_GATE_SIGMOID if w_shared_gate is not None else 0)
        self.c = camera_layer_t(
            self.d_model, self.n_routed, top_k, n_shared, self._d_ff,
            CAMERA_BF16 if self.dtype == torch.bfloat16 else CAMERA_F32, flags,
            CAMERA_DOWN_HF if down_layout == "hf" else CAMERA_DOWN_ME_MAJOR,
            _ptr(w_router), _ptr(router_bias), _ptr(w_shared_gate), self._wg, self._wu, self._wd,
            None if down_ld is None else (C.c_int32 * n)(*[int(v) for v in down_ld]))
        self._down_ld = self.c.w_down_ld      # keeps the array alive
        self.top_k = top_k
        self.n_shared = n_shared
        self._prepared_mem = None

    def __del__(self):
        try:
            camera_layer_release(self)
        except Exception:
            pass

    @classmethod
    def from_workload(cls, L: Dict[str, object]) -> "Layer":
        """From the dict paper_2508_02322_b200.workloads.make_layer returns."""
        cfg = L["cfg"]
        return cls(L["w_router"], L["w_gate"], L["w_up"], L["w_down"], cfg.top_k, cfg.n_shared, L["router_bias"],
                   L["w_shared_gate"], cfg.norm_topk, L["down_layout"])


def camera_layer_prepare(layer: Layer, stream: Optional[torch.cuda.Stream] = None) -> Layer:
    """Builds the layer's per-call tables and weight tensor maps once (camera_layer_prepare); later calls with this
    Layer enqueue kernels only.  The handle and its device memory live as long as the Layer (or until
    camera_layer_release)."""
    camera_layer_release(layer)
    nbytes = int(lib.camera_layer_prepared_bytes(C.byref(layer.c)))
    if nbytes == 0:
        raise CameraError(-1, "camera_layer_prepared_bytes")
    mem = alloc_workspace(nbytes, layer.device)
    handle = C.c_void_p()
    _check(lib.camera_layer_prepare(C.byref(layer.c), mem.data_ptr(), mem.numel(), _stream_ptr(stream), C.byref(handle)),
           "camera_layer_prepare")
    layer._prepared_mem = mem
    layer.c.prepared = handle.value
    return layer


def camera_layer_release(layer: Layer) -> None:
    if getattr(layer, "_prepared_mem", None) is not None and layer.c.prepared:
        lib.camera_layer_release(layer.c.prepared)
    layer.c.prepared = None
    layer._prepared_mem = None


def camera_score_workspace_bytes(layer: Layer, n_tokens: int) -> int:
    return int(lib.camera_score_workspace_bytes(C.byref(layer.c), n_tokens))


def camera_score_workspace_bytes_single_pass(layer: Layer, n_tokens: int) -> int:
    return int(lib.camera_score_workspace_bytes_single_pass(C.byref(layer.c), n_tokens))


def camera_select_workspace_bytes(n_total: int, n_segments: int, n_levels: int) -> int:
    return int(lib.camera_select_workspace_bytes(n_total, n_segments, n_levels))


def camera_analyze_workspace_bytes(layer: Layer, n_tokens: int, n_levels: int) -> int:
    return int(lib.camera_analyze_workspace_bytes(C.byref(layer.c), n_tokens, n_levels))


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """A 256-byte aligned scratch buffer (torch's caching allocator aligns to 512 bytes)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def camera_score_layer(layer: Layer, x: torch.Tensor, alpha: float, *, energy: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, details: bool = False,
                       routing_in=None, force_simt: bool = False, cta_pair: Optional[bool] = None, stage_events=None,
                       phi2: Optional[torch.Tensor] = None, phi_inf_sq: Optional[torch.Tensor] = None,
                       accumulate: bool = False, omega2: Optional[torch.Tensor] = None, omega_given: bool = False,
                       single_pass: bool = False, stream: Optional[torch.cuda.Stream] = None, check_status: bool = False):
    """Algorithm 1 up to the energies.  Returns energy [N_e] fp32, or with details=True a dict that
    also holds phi2, phi_inf_sq, omega2, topk_idx, topk_w, shared_w and expert_token_counts.
    routing_in = (topk_idx int32 [T,k], topk_w fp32 [T,k]) prescribes the routing.
    stage_events = {stage: (torch.cuda.Event, torch.cuda.Event)} records per-stage timing events.
    phi2 / phi_inf_sq name the tensors that receive those components; with accumulate=True they must
    hold the result of earlier batches of tokens, and this batch is folded into them.  omega2 names the tensor
    for the W_down norms; with omega_given=True it already holds them and the pass over W_down is skipped.
    single_pass=True scores more than 65536 tokens in one pass (larger workspace) instead of in batches of 65536."""
    if not (x.is_contiguous() and x.dtype == layer.dtype and x.dim() == 2 and x.shape[1] == layer.d_model):
        raise ValueError("x must be a contiguous [T, d_model] tensor of the layer's dtype")
    T = int(x.shape[0])
    dev = x.device
    if energy is None:
        energy = torch.empty(layer.n_me, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_score_workspace_bytes_single_pass(layer, T) if single_pass
                                    else camera_score_workspace_bytes(layer, T), dev)
    aux = camera_score_aux_t()
    out = {"energy": energy}
    keep_alive = []
    if details:
        k = layer.top_k if layer.n_routed else 0
        out["phi2"] = torch.empty(layer.n_me, dtype=torch.float32, device=dev)
        out["phi_inf_sq"] = torch.empty(layer.n_me, dtype=torch.float32, device=dev)
        out["omega2"] = torch.empty(layer.n_me, dtype=torch.float32, device=dev)
        out["topk_idx"] = torch.empty((T, k), dtype=torch.int32, device=dev)
        out["topk_w"] = torch.empty((T, k), dtype=torch.float32, device=dev)
        out["shared_w"] = torch.empty((layer.n_shared, T), dtype=torch.float32, device=dev)
        out["expert_token_counts"] = torch.empty(layer.n_experts, dtype=torch.int32, device=dev)
        for name in ("phi2", "phi_inf_sq", "omega2", "topk_idx", "topk_w", "shared_w", "expert_token_counts"):
            setattr(aux, name, out[name].data_ptr())
    if routing_in is not None:
        idx, w = routing_in
        idx = idx.to(device=dev, dtype=torch.int32).contiguous()
        w = w.to(device=dev, dtype=torch.float32).contiguous()
        keep_alive += [idx, w]
        aux.topk_idx_in, aux.topk_w_in = idx.data_ptr(), w.data_ptr()
    for name, t in (("phi2", phi2), ("phi_inf_sq", phi_inf_sq), ("omega2", omega2)):
        if t is not None:
            if not (t.is_contiguous() and t.dtype == torch.float32 and t.numel() == layer.n_me and t.device == dev):
                raise ValueError(f"{name} must be a contiguous fp32 [N_e] tensor on the device of x")
            out[name] = t
            setattr(aux, name, t.data_ptr())
    aux.flags = ((CAMERA_SCORE_FORCE_SIMT if force_simt else 0) | (CAMERA_SCORE_CTA_PAIR if cta_pair else 0) | (CAMERA_SCORE_SINGLE_CTA if cta_pair is False else 0) |
                 (CAMERA_SCORE_ACCUMULATE if accumulate else 0) | (CAMERA_SCORE_OMEGA_GIVEN if omega_given else 0) |
                 (CAMERA_SCORE_SINGLE_PASS if single_pass else 0))
    if stage_events:
        for name, (e0, e1) in stage_events.items():
            i = STAGES.index(name)
            aux.stage_events[2 * i] = e0.cuda_event
            aux.stage_events[2 * i + 1] = e1.cuda_event
    sp = _stream_ptr(stream)
    _check(lib.camera_score_layer(C.byref(layer.c), x.data_ptr(), T, float(alpha), energy.data_ptr(),
                                  C.byref(aux), workspace.data_ptr(), workspace.numel(), sp), "camera_score_layer")
    if check_status:
        _check(camera_read_status(workspace, stream), "camera_score_layer (device status)")
    return out if details else energy


def camera_read_status(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    st = C.c_int32(0)
    _check(lib.camera_read_status(workspace.data_ptr(), _stream_ptr(stream), C.byref(st)), "camera_read_status")
    return int(st.value)


def camera_set_wait_limit_ns(limit_ns: int) -> None:
    """Limit of the waits inside the tensor-core kernels, for every later call of the process."""
    _check(lib.camera_set_wait_limit_ns(int(limit_ns)), "camera_set_wait_limit_ns")


def camera_get_wait_limit_ns() -> int:
    return int(lib.camera_get_wait_limit_ns())


def camera_wait_probe(workspace: torch.Tensor, limit_ns: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launches the self-test kernel whose wait runs out after limit_ns; read the result with camera_read_status."""
    _check(lib.camera_wait_probe(workspace.data_ptr(), workspace.numel(), int(limit_ns), _stream_ptr(stream)),
           "camera_wait_probe")


def _segments(n_total: int, seg_offsets):
    seg = [0, n_total] if seg_offsets is None else [int(v) for v in seg_offsets]
    return (C.c_int64 * len(seg))(*seg), len(seg) - 1


def camera_select_all(energy: torch.Tensor, prune_ratios: Sequence[float], ratios: Optional[Sequence[float]] = None,
                      bits: Optional[Sequence[int]] = None, *, seg_offsets=None, workspace: Optional[torch.Tensor] = None,
                      keep_masks: Optional[torch.Tensor] = None, bits_out: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None):
    """The keep masks at several prune ratios (uint8 [len(prune_ratios), N]) and, with ratios / bits, the bit-widths
    (uint8 [N]) from one set of radix passes.  Returns (keep_masks, bits_out); bits_out is None without ratios."""
    n = energy.numel()
    dev = energy.device
    seg, n_seg = _segments(n, seg_offsets)
    n_prune = len(prune_ratios)
    L = len(ratios) if ratios is not None else 0
    if keep_masks is None:
        keep_masks = torch.empty((n_prune, n), dtype=torch.uint8, device=dev)
    if ratios is not None and bits_out is None:
        bits_out = torch.empty(n, dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_select_workspace_bytes(n, n_seg, max(2, n_prune + max(L, 1))), dev)
    pr = (C.c_double * max(n_prune, 1))(*[float(v) for v in prune_ratios])
    r = (C.c_double * max(L, 1))(*[float(v) for v in (ratios or [])])
    b = (C.c_int32 * max(L, 1))(*[int(v) for v in (bits or [])])
    _check(lib.camera_select_all(energy.data_ptr(), seg, n_seg, pr, n_prune, keep_masks.data_ptr(), r, b, L,
                                 _ptr(bits_out) if ratios is not None else None, workspace.data_ptr(), workspace.numel(),
                                 _stream_ptr(stream)), "camera_select_all")
    return keep_masks, (bits_out if ratios is not None else None)


def camera_select_prune(energy: torch.Tensor, prune_ratio: float, *, seg_offsets=None,
                        expert_offsets: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                        keep_mask: Optional[torch.Tensor] = None, want_threshold: bool = False,
                        stream: Optional[torch.cuda.Stream] = None):
    """CAMERA-P mask.  Returns keep_mask uint8 [N]; with expert_offsets (int64, device) also the
    retained count per expert; with want_threshold the per-segment threshold energies."""
    n = energy.numel()
    dev = energy.device
    seg, n_seg = _segments(n, seg_offsets)
    if keep_mask is None:
        keep_mask = torch.empty(n, dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_select_workspace_bytes(n, n_seg, 2), dev)
    kept = thr = None
    n_exp = 0
    if expert_offsets is not None:
        n_exp = expert_offsets.numel() - 1
        kept = torch.empty(n_exp, dtype=torch.int32, device=dev)
    if want_threshold:
        thr = torch.empty(n_seg, dtype=torch.float32, device=dev)
    _check(lib.camera_select_prune(energy.data_ptr(), seg, n_seg, float(prune_ratio), _ptr(expert_offsets), n_exp,
                                   keep_mask.data_ptr(), _ptr(kept), _ptr(thr), workspace.data_ptr(),
                                   workspace.numel(), _stream_ptr(stream)), "camera_select_prune")
    res = [keep_mask]
    if kept is not None:
        res.append(kept)
    if thr is not None:
        res.append(thr)
    return res[0] if len(res) == 1 else tuple(res)


def camera_select_prune_static(energy: torch.Tensor, prune_ratio: float, keep_mask: torch.Tensor, *,
                               seg_offsets=None, thresholds: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """CAMERA-P mask for callers that cannot allocate device memory: the caller passes the input and
    the output tensors, and the selection's scratch is a fixed array inside the library (at most 32
    segments).  This wrapper creates no tensor either.  Calls share that array: keep them on one
    stream, or order them with events."""
    seg, n_seg = _segments(energy.numel(), seg_offsets)
    _check(lib.camera_select_prune_static(energy.data_ptr(), seg, n_seg, float(prune_ratio), keep_mask.data_ptr(),
                                          _ptr(thresholds), _stream_ptr(stream)), "camera_select_prune_static")
    return keep_mask


def camera_alloc_bits(energy: torch.Tensor, ratios: Sequence[float], bits: Sequence[int], *, seg_offsets=None,
                      expert_offsets: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      bits_out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """CAMERA-Q bit-width per micro-expert.  Returns bits_out uint8 [N]; with expert_offsets also
    class_counts int32 [n_experts, n_levels]."""
    n = energy.numel()
    dev = energy.device
    L = len(ratios)
    seg, n_seg = _segments(n, seg_offsets)
    if bits_out is None:
        bits_out = torch.empty(n, dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_select_workspace_bytes(n, n_seg, L), dev)
    counts = None
    n_exp = 0
    if expert_offsets is not None:
        n_exp = expert_offsets.numel() - 1
        counts = torch.empty((n_exp, L), dtype=torch.int32, device=dev)
    r = (C.c_double * L)(*[float(v) for v in ratios])
    b = (C.c_int32 * L)(*[int(v) for v in bits])
    _check(lib.camera_alloc_bits(energy.data_ptr(), seg, n_seg, r, b, L, _ptr(expert_offsets), n_exp,
                                 bits_out.data_ptr(), _ptr(counts), workspace.data_ptr(), workspace.numel(),
                                 _stream_ptr(stream)), "camera_alloc_bits")
    return bits_out if counts is None else (bits_out, counts)


def camera_analyze_layer_host(layer: Layer, x_host: torch.Tensor, alpha: float, prune_ratios: Sequence[float],
                              ratios: Sequence[float], bits: Sequence[int], *, energy_host: torch.Tensor,
                              keep_host: torch.Tensor, bits_host: torch.Tensor, workspace: torch.Tensor,
                              stream: Optional[torch.cuda.Stream] = None) -> None:
    """One analysis step with host token/result buffers (see camera.h); blocks until done.
    keep_host is [len(prune_ratios), N_e] uint8."""
    if x_host.is_cuda or not x_host.is_contiguous() or x_host.dtype != layer.dtype:
        raise ValueError("x_host must be a contiguous host tensor of the layer's dtype")
    L = len(ratios)
    r = (C.c_double * L)(*[float(v) for v in ratios])
    b = (C.c_int32 * L)(*[int(v) for v in bits])
    n_prune = len(prune_ratios)
    pr = (C.c_double * max(n_prune, 1))(*[float(v) for v in prune_ratios])
    _check(lib.camera_analyze_layer_host(C.byref(layer.c), x_host.data_ptr(), int(x_host.shape[0]), float(alpha),
                                         pr, n_prune, r, b, L, _ptr(energy_host), _ptr(keep_host),
                                         _ptr(bits_host), workspace.data_ptr(), workspace.numel(),
                                         _stream_ptr(stream)), "camera_analyze_layer_host")


def expert_offsets_tensor(layer: Layer) -> torch.Tensor:
    """Global micro-expert offsets of the layer's experts: int64 [n_experts + 1] on its device."""
    off = [0]
    for f in layer.d_ff:
        off.append(off[-1] + f)
    return torch.tensor(off, dtype=torch.int64, device=layer.device)


def camera_sub_index(labels: torch.Tensor, expert_offsets: torch.Tensor, label_order: Sequence[int], *,
                     stream: Optional[torch.cuda.Stream] = None):
    """GetSubIndex.  labels uint8 [N_e] (keep mask or bit-widths), expert_offsets int64 [E+1] on the device.
    Returns (sub_index int32 [N_e], counts int32 [E, len(label_order)])."""
    if labels.dtype != torch.uint8 or not labels.is_contiguous():
        raise ValueError("labels must be a contiguous uint8 tensor")
    n_exp = expert_offsets.numel() - 1
    order = (C.c_int32 * len(label_order))(*[int(v) for v in label_order])
    sub = torch.empty(labels.numel(), dtype=torch.int32, device=labels.device)
    counts = torch.empty((n_exp, len(label_order)), dtype=torch.int32, device=labels.device)
    _check(lib.camera_sub_index(labels.data_ptr(), expert_offsets.data_ptr(), n_exp, order, len(label_order),
                                sub.data_ptr(), counts.data_ptr(), _stream_ptr(stream)), "camera_sub_index")
    return sub, counts


def camera_compact_weights(layer: Layer, sub_index: torch.Tensor, counts: torch.Tensor, n_take: int, *,
                           out: Optional[Dict[str, List[torch.Tensor]]] = None, down_ld: Optional[Sequence[int]] = None,
                           workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Gathers W_gate[S,:], W_up[S,:], W_down[:,S] (Algorithm 2, the slicing step) with S the entries of the first n_take
    labels of every expert's list.  `out` = {"w_gate": [...], "w_up": [...], "w_down": [...]} (per expert, sized
    like the sources unless down_ld says otherwise); allocated when missing.  Returns `out`; the rows / columns
    actually written per expert are counts[:, :n_take].sum(1)."""
    t = layer.tensors
    if out is None:
        out = {k: [torch.empty_like(w) for w in t[k]] for k in ("w_gate", "w_up", "w_down")}
    n = layer.n_experts
    pg = (C.c_void_p * n)(*[w.data_ptr() for w in out["w_gate"]])
    pu = (C.c_void_p * n)(*[w.data_ptr() for w in out["w_up"]])
    pd = (C.c_void_p * n)(*[w.data_ptr() for w in out["w_down"]])
    ld = None if down_ld is None else (C.c_int32 * n)(*[int(v) for v in down_ld])
    if workspace is None:
        workspace = alloc_workspace(int(lib.camera_compact_workspace_bytes(n)), layer.device)
    _check(lib.camera_compact_weights(C.byref(layer.c), sub_index.data_ptr(), counts.data_ptr(), int(counts.shape[1]),
                                      int(n_take), pg, pu, pd, ld, workspace.data_ptr(), workspace.numel(),
                                      _stream_ptr(stream)), "camera_compact_weights")
    return out


def camera_forward_workspace_bytes(layer: Layer, n_tokens: int) -> int:
    return int(lib.camera_forward_workspace_bytes(C.byref(layer.c), n_tokens))


def camera_layer_forward(layer: Layer, x: torch.Tensor, *, y: Optional[torch.Tensor] = None, routing_in=None,
                         workspace: Optional[torch.Tensor] = None, want_routing: bool = False,
                         cta_pair: Optional[bool] = None, token_rows: bool = False,
                         stream: Optional[torch.cuda.Stream] = None):
    """The layer's output y [T, d_model] fp32 (Eq. 1-2).  routing_in = (topk_idx, topk_w) prescribes the routed
    coefficients; want_routing also returns the (topk_idx, topk_w) the call used; cta_pair forces the CTA-pair
    (True) or single-CTA (False) gate/up kernel of the scoring orientation, token_rows the kernel with the tokens on
    the accumulator rows, instead of the library's choice."""
    T = int(x.shape[0])
    dev = x.device
    if y is None:
        y = torch.empty((T, layer.d_model), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_forward_workspace_bytes(layer, T), dev)
    aux = camera_score_aux_t()
    aux.flags = ((CAMERA_SCORE_CTA_PAIR if cta_pair else 0) | (CAMERA_SCORE_SINGLE_CTA if cta_pair is False else 0) |
                 (CAMERA_FORWARD_TOKEN_ROWS if token_rows else 0))
    keep_alive = []
    if routing_in is not None:
        idx = routing_in[0].to(device=dev, dtype=torch.int32).contiguous()
        w = routing_in[1].to(device=dev, dtype=torch.float32).contiguous()
        keep_alive += [idx, w]
        aux.topk_idx_in, aux.topk_w_in = idx.data_ptr(), w.data_ptr()
    routing = None
    if want_routing:
        k = layer.top_k if layer.n_routed else 0
        routing = (torch.empty((T, k), dtype=torch.int32, device=dev), torch.empty((T, k), dtype=torch.float32, device=dev))
        aux.topk_idx, aux.topk_w = routing[0].data_ptr(), routing[1].data_ptr()
    _check(lib.camera_layer_forward(C.byref(layer.c), x.data_ptr(), T, y.data_ptr(), C.byref(aux), workspace.data_ptr(),
                                    workspace.numel(), _stream_ptr(stream)), "camera_layer_forward")
    return (y, routing) if want_routing else y


def camera_score_forward_layer(layer: Layer, x: torch.Tensor, alpha: float, *, energy: Optional[torch.Tensor] = None,
                               y: Optional[torch.Tensor] = None, routing_in=None, workspace: Optional[torch.Tensor] = None,
                               phi2: Optional[torch.Tensor] = None, phi_inf_sq: Optional[torch.Tensor] = None,
                               accumulate: bool = False, omega2: Optional[torch.Tensor] = None,
                               omega_given: bool = False, cta_pair: Optional[bool] = None,
                               stream: Optional[torch.cuda.Stream] = None):
    """Energies (Algorithm 1) and layer output (Eq. 1-2) of one batch from one pass over W_gate and W_up.
    Returns (energy [N_e] fp32, y [T, d_model] fp32); arguments as for camera_score_layer and camera_layer_forward."""
    T = int(x.shape[0])
    dev = x.device
    if energy is None:
        energy = torch.empty(layer.n_me, dtype=torch.float32, device=dev)
    if y is None:
        y = torch.empty((T, layer.d_model), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = alloc_workspace(camera_forward_workspace_bytes(layer, T), dev)
    aux = camera_score_aux_t()
    aux.flags = ((CAMERA_SCORE_CTA_PAIR if cta_pair else 0) | (CAMERA_SCORE_SINGLE_CTA if cta_pair is False else 0) |
                 (CAMERA_SCORE_ACCUMULATE if accumulate else 0) | (CAMERA_SCORE_OMEGA_GIVEN if omega_given else 0))
    keep_alive = []
    if routing_in is not None:
        idx = routing_in[0].to(device=dev, dtype=torch.int32).contiguous()
        w = routing_in[1].to(device=dev, dtype=torch.float32).contiguous()
        keep_alive += [idx, w]
        aux.topk_idx_in, aux.topk_w_in = idx.data_ptr(), w.data_ptr()
    for name, t in (("phi2", phi2), ("phi_inf_sq", phi_inf_sq), ("omega2", omega2)):
        if t is not None:
            if not (t.is_contiguous() and t.dtype == torch.float32 and t.numel() == layer.n_me and t.device == dev):
                raise ValueError(f"{name} must be a contiguous fp32 [N_e] tensor on the device of x")
            setattr(aux, name, t.data_ptr())
    _check(lib.camera_score_forward_layer(C.byref(layer.c), x.data_ptr(), T, float(alpha), energy.data_ptr(), y.data_ptr(),
                                          C.byref(aux), workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)),
           "camera_score_forward_layer")
    return energy, y


def camera_mask_down_columns(layer: Layer, keep: torch.Tensor, *, out=None, stream: Optional[torch.cuda.Stream] = None):
    """W_down of every expert with the columns of the micro-experts outside the selection set to zero.
    keep: uint8 [N_e] on the device; out: list of tensors shaped like the layer's W_down (allocated if None)."""
    if out is None:
        out = [torch.empty_like(w) for w in layer.tensors["w_down"]]
    ptrs = (C.c_void_p * layer.n_experts)(*[t.data_ptr() for t in out])
    _check(lib.camera_mask_down_columns(C.byref(layer.c), keep.data_ptr(), ptrs, _stream_ptr(stream)),
           "camera_mask_down_columns")
    return out


def camera_pruned_output(layer: Layer, w_down_masked, n_tokens: int, workspace: torch.Tensor, *,
                         y: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Y_hat = Phi[:,S] W[S,:] (Eq. 7) from the h that the last camera_score_forward_layer / camera_layer_forward
    call left in `workspace` (same layer, same number of tokens) and W_down with the pruned columns zeroed."""
    if y is None:
        y = torch.empty((n_tokens, layer.d_model), dtype=torch.float32, device=workspace.device)
    ptrs = (C.c_void_p * layer.n_experts)(*[t.data_ptr() for t in w_down_masked])
    _check(lib.camera_pruned_output(C.byref(layer.c), ptrs, int(n_tokens), y.data_ptr(), None, workspace.data_ptr(),
                                    workspace.numel(), _stream_ptr(stream)), "camera_pruned_output")
    return y


def camera_output_error(y: torch.Tensor, y_hat: torch.Tensor, *, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """float64 [3] on the device: ||Y - Y_hat||_F^2, ||Y||_F^2, mean cosine similarity of the token outputs."""
    if y.shape != y_hat.shape or y.dtype != torch.float32 or y_hat.dtype != torch.float32 or y.dim() != 2:
        raise ValueError("y and y_hat must be fp32 [T, d_model] tensors of one shape")
    T, d = int(y.shape[0]), int(y.shape[1])
    out = torch.empty(3, dtype=torch.float64, device=y.device)
    ws = alloc_workspace(int(lib.camera_output_error_workspace_bytes(T)), y.device)
    _check(lib.camera_output_error(y.contiguous().data_ptr(), y_hat.contiguous().data_ptr(), T, d, out.data_ptr(),
                                   ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "camera_output_error")
    return out


def camera_residual_norm(x: torch.Tensor, y: torch.Tensor, *, eps: float = 1e-6, out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Next layer's input of a synthetic stack: (x + y) rescaled to RMS 1 per token, in the dtype of x."""
    if x.shape != y.shape or y.dtype != torch.float32 or x.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("x: bf16 or fp32 [T, d_model], y: fp32 of the same shape")
    if out is None:
        out = torch.empty_like(x)
    _check(lib.camera_residual_norm(x.contiguous().data_ptr(), CAMERA_BF16 if x.dtype == torch.bfloat16 else CAMERA_F32,
                                    y.contiguous().data_ptr(), int(x.shape[0]), int(x.shape[1]), float(eps), out.data_ptr(),
                                    _stream_ptr(stream)), "camera_residual_norm")
    return out

"""Host-only checks of the C ABI: the library loads, exports what include/camera.h declares, and
rejects bad arguments before anything touches a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def P():
    import paper_2508_02322_b200 as pkg
    return pkg


def declared_functions():
    text = open(os.path.join(ROOT, "include", "camera.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(camera_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(P):
    names = declared_functions()
    assert {"camera_score_layer", "camera_select_prune", "camera_alloc_bits"} <= set(names)
    for n in names:
        assert hasattr(P.lib, n), n
    assert P.lib.camera_version() >= 100
    assert P.lib.camera_strerror(0) == b"ok" and b"workspace" in P.lib.camera_strerror(-3)


def _layer_struct(P, d_model=64, n_routed=4, top_k=2, d_ff=(64, 64, 64, 64), n_shared=0, dtype=1, flags=1):
    from paper_2508_02322_b200.binding import camera_layer_t
    n = len(d_ff)
    dff = (C.c_int32 * n)(*d_ff)
    ptrs = (C.c_void_p * n)(*[4096] * n)
    s = camera_layer_t(d_model, n_routed, top_k, n_shared, dff, dtype, flags, 0, 4096, None, None, ptrs, ptrs, ptrs)
    s._keep = (dff, ptrs)
    return s


def test_workspace_query_validates_shapes(P):
    ok = _layer_struct(P)
    assert P.lib.camera_score_workspace_bytes(C.byref(ok), 1000) > 0
    assert P.lib.camera_score_workspace_bytes(C.byref(ok), 0) > 0
    assert P.lib.camera_score_workspace_bytes(C.byref(ok), -1) == 0
    assert P.lib.camera_score_workspace_bytes(C.byref(_layer_struct(P, top_k=5)), 10) == 0      # k > n_routed
    assert P.lib.camera_score_workspace_bytes(C.byref(_layer_struct(P, d_model=60)), 10) == 0   # d_model % 8
    assert P.lib.camera_score_workspace_bytes(C.byref(_layer_struct(P, d_ff=(64, 64, 64, 60))), 10) == 0
    assert P.lib.camera_score_workspace_bytes(C.byref(_layer_struct(P, dtype=7)), 10) == 0
    assert P.lib.camera_score_workspace_bytes(None, 10) == 0
    # more tokens never need less scratch
    a = P.lib.camera_score_workspace_bytes(C.byref(ok), 1000)
    b = P.lib.camera_score_workspace_bytes(C.byref(ok), 100000)
    assert b > a
    assert P.lib.camera_select_workspace_bytes(1000, 1, 2) > 0
    assert P.lib.camera_select_workspace_bytes(1000, 1, 9) == 0
    assert P.lib.camera_analyze_workspace_bytes(C.byref(ok), 1000, 3) > P.lib.camera_score_workspace_bytes(C.byref(ok), 1000)


def test_argument_errors_return_before_any_launch(P):
    ok = _layer_struct(P)
    # alpha outside [0,1], null energy: rejected on the host (pointers here are fake and never dereferenced)
    assert P.lib.camera_score_layer(C.byref(ok), 4096, 10, C.c_float(1.5), 4096, None, 4096, 1 << 30, None) == -1
    assert P.lib.camera_score_layer(C.byref(ok), 4096, 10, C.c_float(0.5), None, None, 4096, 1 << 30, None) == -1
    assert P.lib.camera_score_layer(C.byref(ok), 4096, 10, C.c_float(0.5), 4096, None, None, 0, None) == -3
    from paper_2508_02322_b200.binding import camera_score_aux_t, CAMERA_SCORE_OMEGA_GIVEN
    aux = camera_score_aux_t()
    aux.flags = CAMERA_SCORE_OMEGA_GIVEN                      # says the norms are given, gives none
    assert P.lib.camera_score_layer(C.byref(ok), 4096, 10, C.c_float(0.5), 4096, C.byref(aux), 4096, 1 << 30, None) == -1
    seg = (C.c_int64 * 2)(0, 10)
    bad = (C.c_int64 * 2)(1, 10)
    assert P.lib.camera_select_prune(4096, seg, 1, C.c_double(1.0), None, 0, 4096, None, None, 4096, 1 << 20, None) == -1
    assert P.lib.camera_select_prune(4096, bad, 1, C.c_double(0.5), None, 0, 4096, None, None, 4096, 1 << 20, None) == -1
    assert P.lib.camera_select_prune(4096, seg, 1, C.c_double(0.5), None, 0, 4096, None, None, 4096, 16, None) == -3
    pr = (C.c_double * 3)(0.2, 0.4, 0.6)
    rt = (C.c_double * 3)(0.2, 0.6, 0.2)
    bt = (C.c_int32 * 3)(3, 2, 1)
    assert P.lib.camera_select_all(4096, seg, 1, pr, 3, None, rt, bt, 3, 4096, 4096, 1 << 20, None) == -1     # no masks
    assert P.lib.camera_select_all(4096, seg, 1, pr, 0, None, rt, bt, 3, None, 4096, 1 << 20, None) == -1     # nothing asked for
    assert P.lib.camera_select_all(4096, seg, 1, (C.c_double * 1)(1.0), 1, 4096, rt, bt, 3, 4096, 4096, 1 << 20, None) == -1
    assert P.lib.camera_select_all(4096, seg, 1, pr, 3, 4096, rt, bt, 3, 4096, 4096, 16, None) == -3
    r = (C.c_double * 3)(0.2, 0.5, 0.2)
    b = (C.c_int32 * 3)(3, 2, 1)
    assert P.lib.camera_alloc_bits(4096, seg, 1, r, b, 3, None, 0, 4096, None, 4096, 1 << 20, None) == -1   # ratios sum
    r = (C.c_double * 3)(0.2, 0.6, 0.2)
    b = (C.c_int32 * 3)(3, 2, 300)
    assert P.lib.camera_alloc_bits(4096, seg, 1, r, b, 3, None, 0, 4096, None, 4096, 1 << 20, None) == -1   # bit-width


def test_new_entry_points_reject_bad_arguments_on_the_host(P):
    ok = _layer_struct(P)
    order = (C.c_int32 * 2)(1, 1)
    assert P.lib.camera_sub_index(4096, 4096, 4, order, 2, 4096, 4096, None) == -1               # a label named twice
    assert P.lib.camera_sub_index(None, 4096, 4, order, 1, 4096, 4096, None) == -1
    assert P.lib.camera_compact_workspace_bytes(0) == 0 and P.lib.camera_compact_workspace_bytes(65) >= 65 * 64
    ptrs = (C.c_void_p * 4)(*[4096] * 4)
    assert P.lib.camera_compact_weights(C.byref(ok), 4096, 4096, 1, 2, ptrs, ptrs, ptrs, None, 4096, 1 << 20, None) == -1   # n_take > n_labels
    assert P.lib.camera_compact_weights(C.byref(ok), 4096, 4096, 1, 1, ptrs, ptrs, ptrs, None, None, 0, None) == -3
    assert P.lib.camera_forward_workspace_bytes(C.byref(ok), 1000) > P.lib.camera_score_workspace_bytes(C.byref(ok), 1000)
    # the forward path takes sliced layers: any d_ff >= 0, as long as W_down rows start on 16-byte boundaries
    odd = _layer_struct(P, d_ff=(64, 3, 0, 64))
    assert P.lib.camera_score_workspace_bytes(C.byref(odd), 10) == 0
    assert P.lib.camera_forward_workspace_bytes(C.byref(odd), 10) > 0
    assert P.lib.camera_layer_forward(C.byref(ok), 4096, 10, None, None, 4096, 1 << 30, None) == -1        # no output
    f32 = _layer_struct(P, dtype=0)
    assert P.lib.camera_layer_forward(C.byref(f32), 4096, 10, 4096, None, 4096, 1 << 30, None) == -2       # bf16 only
    assert P.lib.camera_score_forward_layer(C.byref(ok), 4096, 10, C.c_float(0.5), None, 4096, None, 4096, 1 << 30, None) == -1   # no energy
    assert P.lib.camera_score_forward_layer(C.byref(ok), 4096, 10, C.c_float(0.5), 4096, None, None, 4096, 1 << 30, None) == -1   # no output
    assert P.lib.camera_score_forward_layer(C.byref(f32), 4096, 10, C.c_float(0.5), 4096, 4096, None, 4096, 1 << 30, None) == -2
    ptrs4 = (C.c_void_p * 4)(*[4096] * 4)
    assert P.lib.camera_mask_down_columns(C.byref(ok), None, ptrs4, None) == -1                             # no mask
    assert P.lib.camera_mask_down_columns(C.byref(ok), 4100, ptrs4, None) == -1                             # mask not 8-byte aligned
    assert P.lib.camera_mask_down_columns(C.byref(f32), 4096, ptrs4, None) == -2
    assert P.lib.camera_pruned_output(C.byref(ok), None, 10, 4096, None, 4096, 1 << 30, None) == -1
    assert P.lib.camera_pruned_output(C.byref(ok), ptrs4, 10, 4096, None, None, 0, None) == -3
    assert P.lib.camera_output_error(4096, 4096, 10, 0, 4096, 4096, 1 << 20, None) == -1
    assert P.lib.camera_output_error(4096, 4096, 10, 64, 4096, None, 0, None) == -3
    assert P.lib.camera_residual_norm(4096, 1, 4096, 10, 60, C.c_float(1e-6), 4096, None) == -1             # d_model % 8
    assert P.lib.camera_residual_norm(4096, 5, 4096, 10, 64, C.c_float(1e-6), 4096, None) == -1             # dtype
    assert P.lib.camera_residual_norm(None, 1, None, 0, 64, C.c_float(1e-6), None, None) == 0              # nothing to do


def test_prepare_checks_its_arguments_before_touching_a_device(P):
    ok = _layer_struct(P)
    n = P.lib.camera_layer_prepared_bytes(C.byref(ok))
    assert n > 0 and n % 256 == 0
    assert P.lib.camera_layer_prepared_bytes(C.byref(_layer_struct(P, top_k=5))) == 0
    handle = C.c_void_p()
    assert P.lib.camera_layer_prepare(C.byref(ok), None, 0, None, C.byref(handle)) == -3      # no device memory given
    assert handle.value is None
    assert P.lib.camera_layer_prepare(C.byref(ok), 4096, n - 1, None, C.byref(handle)) == -3  # too little of it
    assert P.lib.camera_layer_prepare(C.byref(ok), 4096, n, None, None) == -1
    P.lib.camera_layer_release(None)                                                          # a null handle is ignored


def test_score_scratch_stops_growing_at_one_batch(P):
    ok = _layer_struct(P)
    q = lambda t: P.lib.camera_score_workspace_bytes(C.byref(ok), t)
    one = lambda t: P.lib.camera_score_workspace_bytes_single_pass(C.byref(ok), t)
    assert q(1000) == one(1000) and q(65536) == one(65536)          # up to a batch the two are the same
    assert q(65537) == q(10 ** 6) > q(65536)                         # beyond: one batch's scratch plus the accumulators
    assert one(10 ** 6) > one(65537) and one(10 ** 6) > 4 * q(10 ** 6)    # a single pass keeps growing with the tokens
    assert one(-1) == 0 and P.lib.camera_score_workspace_bytes_single_pass(None, 10) == 0


def test_wait_limit_and_probe_check_their_arguments_on_the_host(P):
    default = P.lib.camera_get_wait_limit_ns()
    assert default == 4_000_000_000
    assert P.lib.camera_set_wait_limit_ns(10) == -1                  # under a microsecond
    assert P.lib.camera_set_wait_limit_ns(10 ** 13) == -1            # over ten minutes
    assert P.lib.camera_get_wait_limit_ns() == default
    assert P.lib.camera_set_wait_limit_ns(2_000_000_000) == 0 and P.lib.camera_get_wait_limit_ns() == 2_000_000_000
    assert P.lib.camera_set_wait_limit_ns(default) == 0
    assert P.lib.camera_wait_probe(4096, 4096, 5_000_000_000, None) == -1      # a probe may wait a second at most
    assert P.lib.camera_wait_probe(None, 4096, 1_000_000, None) == -3          # no workspace
    assert P.lib.camera_wait_probe(4096 + 8, 4096, 1_000_000, None) == -3      # not 256-byte aligned

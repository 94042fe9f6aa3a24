"""The workspace-free selection entry point, camera_select_prune_static.

Some users of the library run where they may not allocate device memory (a plug-in inside a server
whose pool owns the GPU, code that must not trigger cudaMalloc's device-wide synchronisation), so
this entry point keeps its scratch in a fixed array inside the library.  It has to give exactly the
mask of camera_select_prune and of the oracle's selection, also when it is called again and the array
still holds the previous call's histograms and thresholds, and it must leave the amount of free device
memory as it found it.  This file sorts last on purpose: every other test has run by then.
"""
import numpy as np
import pytest
import torch

import oracle as O

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _energies(n, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    E = torch.rand(n, generator=g) ** 3
    E[n // 7: n // 7 + n // 11] = 0.0          # a long run of exact ties at the bottom
    E[n // 2: n // 2 + 5] = E[n // 2]           # a short one in the middle
    return E.to(DEV)


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    import paper_2508_02322_b200 as P
    from paper_2508_02322_b200.binding import camera_select_prune_static

    # call 1: one layer-sized segment; call 2: different data, several segments, other ratio.
    # The second call meets the first call's leftovers in the shared array.
    cases = [(_energies(184320, 1), None, 0.4),
             (_energies(50000, 2), [0, 4096, 4096, 30000, 50000], 0.6),
             (_energies(184320, 3), None, 0.2)]
    for E, seg, ratio in cases:
        n_seg = 1 if seg is None else len(seg) - 1
        keep = torch.full((E.numel(),), 7, dtype=torch.uint8, device=DEV)
        thr = torch.empty(n_seg, dtype=torch.float32, device=DEV)
        camera_select_prune_static(E, ratio, keep, seg_offsets=seg, thresholds=thr)
        ref_keep, ref_thr = P.camera_select_prune(E, ratio, seg_offsets=seg, want_threshold=True)
        torch.cuda.synchronize()
        assert torch.equal(keep, ref_keep)              # masks are integer work: bit-exact
        assert np.array_equal(thr.cpu().numpy(), ref_thr.cpu().numpy())
        # ... and against the oracle's TopSelect, segment by segment (a segment is a layer of its own)
        E_np, got = E.cpu().numpy(), keep.cpu().numpy()
        bounds = [0, E.numel()] if seg is None else seg
        for s0, s1 in zip(bounds[:-1], bounds[1:]):
            assert np.array_equal(got[s0:s1], O.select_prune(E_np[s0:s1], ratio))
    # same input twice, back to back on one stream, no synchronisation in between
    E = cases[0][0]
    a = torch.empty(E.numel(), dtype=torch.uint8, device=DEV)
    b = torch.empty(E.numel(), dtype=torch.uint8, device=DEV)
    camera_select_prune_static(E, 0.4, a)
    camera_select_prune_static(E, 0.4, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(a, P.camera_select_prune(E, 0.4))


def test_static_scratch_leaves_free_device_memory_unchanged():
    """What the entry point is for: no device allocation.  The driver's count of free device memory (which sees every
    cudaMalloc of the process, the library's included, but not torch's reuse of blocks it already holds) is the same
    before and after a series of calls; the first call on the device, which looks the array up, comes before."""
    from paper_2508_02322_b200.binding import camera_select_prune_static

    E = _energies(184320, 5)
    keep = torch.empty(E.numel(), dtype=torch.uint8, device=DEV)
    thr = torch.empty(28, dtype=torch.float32, device=DEV)
    seg = [i * (E.numel() // 28) for i in range(28)] + [E.numel()]
    camera_select_prune_static(E, 0.4, keep)            # first call: set-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for ratio in (0.2, 0.4, 0.6):
        camera_select_prune_static(E, ratio, keep)
        camera_select_prune_static(E, ratio, keep, seg_offsets=seg, thresholds=thr)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    E_np, got = E.cpu().numpy(), keep.cpu().numpy()
    for s0, s1 in zip(seg[:-1], seg[1:]):
        assert np.array_equal(got[s0:s1], O.select_prune(E_np[s0:s1], 0.6))


def test_static_scratch_rejects_too_many_segments():
    import paper_2508_02322_b200 as P
    from paper_2508_02322_b200.binding import camera_select_prune_static

    E = _energies(3300, 4)
    keep = torch.empty(3300, dtype=torch.uint8, device=DEV)
    seg = list(range(0, 3301, 100))                     # 33 segments, one more than the array is sized for
    with pytest.raises(P.CameraError) as err:
        camera_select_prune_static(E, 0.4, keep, seg_offsets=seg)
    assert err.value.status == -2
    seg32 = list(range(0, 3201, 100))                   # 32 segments: the largest count it takes
    Es, ks = E[:3200].contiguous(), keep[:3200]
    camera_select_prune_static(Es, 0.4, ks, seg_offsets=seg32)
    torch.cuda.synchronize()
    assert torch.equal(ks, P.camera_select_prune(Es, 0.4, seg_offsets=seg32))

"""The allocation-free selection entry point must agree, bit for bit, with the one that takes a
caller-provided workspace.  It serves callers that cannot allocate device memory at the point of
the call (a serving loop where cudaMalloc would stall every stream, a process whose device memory
was handed out at start-up), so the test gives it nothing but preallocated buffers, twice in a row:
the second call runs on the scratch contents the first one left behind.

This file sorts after the other test files on purpose: a run that stops at the first failure has
then already gone through everything else."""
import numpy as np
import pytest
import torch

import workloads as wl

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _both(cp, K, C, R, keep, seed, depthwise):
    w = wl.normal_f32(seed, 1, (K, C, R, R), 0.05)
    if K > 8:
        w[5] = w[2]                                  # an exact tie in the ranking
    b = wl.normal_f32(seed, 2, (K,), 0.01)
    wn = wl.normal_f32(seed, 3, (K, 1, 3, 3) if depthwise else (11, K, 3, 3), 0.05)
    dw, db, dwn = _dev(w), _dev(b), _dev(wn)
    ref = cp.cprune_select_filters(dw, keep, db, dwn, next_is_depthwise=depthwise)
    kept = torch.full((keep,), -1, dtype=torch.int32, device="cuda")
    w_out = torch.full((keep, C, R, R), float("nan"), device="cuda")
    b_out = torch.full((keep,), float("nan"), device="cuda")
    wn_out = torch.full(tuple(ref[3].shape), float("nan"), device="cuda")
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    got = cp.cprune_select_filters_static(dw, keep, kept, w_out, db, b_out, dwn, wn_out, next_is_depthwise=depthwise)
    assert torch.cuda.memory_allocated() == before   # nothing was allocated through torch either
    cp.cprune_poll_device_status()
    for g, r in zip(got, ref):
        assert g.cpu().numpy().tobytes() == r.cpu().numpy().tobytes()


def test_static_selection_matches_workspace_selection_twice_in_a_row():
    import paper_2207_01260_b200 as cp
    cp.lib()
    _both(cp, 512, 64, 3, 358, seed=41, depthwise=False)    # fills most of a large prefix of the scratch
    _both(cp, 96, 16, 1, 72, seed=42, depthwise=True)       # a smaller layer on the stale scratch
    _both(cp, 4096, 2, 1, 1000, seed=43, depthwise=False)   # exactly the maximum


def test_static_selection_rejects_more_filters_than_its_buffer_holds():
    import paper_2207_01260_b200 as cp
    K = cp.binding.SELECT_STATIC_MAX_FILTERS + 1
    w = torch.zeros((K, 1, 1, 1), device="cuda")
    kept = torch.empty(4, dtype=torch.int32, device="cuda")
    w_out = torch.empty((4, 1, 1, 1), device="cuda")
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_select_filters_static(w, 4, kept, w_out)
    assert e.value.status == 3

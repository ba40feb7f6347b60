"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

TOL = 2e-2          # max |err| <= TOL * (|b| + sum |x||w| + |res|) per output element


@pytest.fixture(scope="module")
def cp():
    import paper_2207_01260_b200 as m
    m.lib()
    return m


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_task(cp, x, w, b, stride, pad, groups=1, act="relu", res=None, pool=None, kernel="auto"):
    N, H, W, C = x.shape
    K, _, R, S = w.shape
    plan = cp.cprune_task_plan(N, C, H, W, K, R, S, stride, pad, groups, act, res is not None, pool, kernel)
    xb = cp.cprune_cast_input(_dev(x))
    wp, bp = cp.cprune_pack_weights(plan, _dev(w), _dev(b))
    rb = cp.cprune_cast_input(_dev(res)) if res is not None else None
    y = cp.cprune_task_run(plan, xb, wp, bp, rb)
    cp.cprune_poll_device_status()
    return y.float().cpu().numpy(), plan


def check_task(cp, N, C, H, W, K, R, stride, pad, groups=1, act="relu", with_res=False, pool=None, kernel="auto",
               seed=11):
    P, Q = oracle.out_size(H, R, stride, pad), oracle.out_size(W, R, stride, pad)
    x, w, b, res = wl.conv_task_tensors(seed, N, C, H, W, K, R, R, groups, with_res, P, Q)
    y, plan = run_task(cp, x, w, b, stride, pad, groups, act, res, pool, kernel)
    ref, bound = oracle.conv2d(x, w, b, stride, pad, groups, act, res, with_bound=True)
    if pool == "max3x3s2":
        # the error bound of a maximum is at most the largest bound in its window
        ref, bound = oracle.maxpool(ref, 3, 2, 1), oracle.maxpool(bound, 3, 2, 1)
    elif pool:
        ref, bound = oracle.maxpool(ref, 2, 2, 0), oracle.maxpool(bound, 2, 2, 0)
    assert y.shape == (N, plan.out_h, plan.out_w, plan.k_pad)
    assert np.all(y[..., K:] == 0), "pad lanes must be written as zero"
    err = np.abs(y[..., :K] - ref)
    worst = np.max(err / (bound + 1e-30))
    assert worst <= TOL, (worst, np.unravel_index(np.argmax(err / (bound + 1e-30)), err.shape))
    assert np.max(err) > 0 or np.max(np.abs(ref)) == 0   # bf16 data cannot be bit-exact against float64
    return plan


# ------------------------------------------------------------------ selection (bit-exact)

@pytest.mark.parametrize("K,C,R,keep", [(64, 64, 3, 48), (37, 5, 3, 17), (512, 512, 3, 358), (96, 16, 1, 72),
                                        (1280, 7, 1, 999), (9, 3, 7, 1), (300, 20, 3, 300)])
def test_select_filters_bit_exact(cp, K, C, R, keep):
    w = wl.normal_f32(21, 1, (K, C, R, R), 0.05)
    if K >= 30:
        w[11] = w[3]
        w[20] = -w[3]
    b = wl.normal_f32(21, 2, (K,), 0.01)
    wn = wl.normal_f32(21, 3, (13, K, 3, 3), 0.05)
    kept, wo, bo, wno = cp.cprune_select_filters(_dev(w), keep, _dev(b), _dev(wn))
    cp.cprune_poll_device_status()
    rk, rw, rb, rwn = oracle.select_filters(w, b, keep, wn)
    assert np.array_equal(kept.cpu().numpy(), rk)
    assert wo.cpu().numpy().tobytes() == rw.tobytes()
    assert bo.cpu().numpy().tobytes() == rb.tobytes()
    assert wno.cpu().numpy().tobytes() == rwn.tobytes()
    wd = wl.normal_f32(21, 4, (K, 1, 3, 3), 0.05)
    kept2, _, _, wdo = cp.cprune_select_filters(_dev(w), keep, None, _dev(wd), next_is_depthwise=True)
    assert np.array_equal(kept2.cpu().numpy(), rk)
    assert wdo.cpu().numpy().tobytes() == wd[rk].tobytes()
    g = cp.cprune_gather_columns(_dev(wn), kept)
    assert g.cpu().numpy().tobytes() == rwn.tobytes()
    g = cp.cprune_gather_rows(_dev(b), kept)
    assert g.cpu().numpy().tobytes() == rb.tobytes()


def test_select_every_keep_count_nests(cp):
    w = wl.normal_f32(22, 1, (64, 64, 3, 3), 0.06)
    dw = _dev(w)
    for keep in range(16, 65):
        kept, _, _, _ = cp.cprune_select_filters(dw, keep)
        assert np.array_equal(kept.cpu().numpy(), oracle.select_indices(w, keep))


def test_select_flags_bad_weights_and_bad_arguments(cp):
    w = wl.normal_f32(23, 1, (8, 4, 3, 3), 0.05)
    w[2, 1, 1, 1] = np.nan
    cp.cprune_select_filters(_dev(w), 4)
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_poll_device_status()
    assert e.value.status == 7
    cp.cprune_poll_device_status()      # the word was cleared
    good = _dev(wl.normal_f32(23, 2, (8, 4, 3, 3), 0.05))
    for keep in (0, 9, -1):
        with pytest.raises(cp.CpruneError) as e:
            cp.cprune_select_filters(good, keep)
        assert e.value.status == 1
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_select_filters(good, 4, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3


# ------------------------------------------------------------------ single tasks

def test_config1_single_pruned_task(cp):
    m = wl.single_task()
    w, b = wl.model_weights(m)["conv"]
    x = wl.model_input(m, 1)
    kept, wo, bo, _ = cp.cprune_select_filters(_dev(w), 48, _dev(b))
    rk, rw, rb, _ = oracle.select_filters(w, b, 48)
    assert np.array_equal(kept.cpu().numpy(), rk)
    for kernel in ("tensor", "direct"):
        y, plan = run_task(cp, x, wo.cpu().numpy(), bo.cpu().numpy(), 1, 1, kernel=kernel)
        assert cp.KERNEL_NAMES[plan.kernel] == kernel
        ref, bound = oracle.conv2d(x, rw, rb, 1, 1, 1, "relu", with_bound=True)
        assert y.shape == (1, 32, 32, 48)
        assert np.max(np.abs(y - ref) / (bound + 1e-30)) <= TOL


DENSE_CASES = [
    # N, C, H, W, K, R, stride, pad
    (1, 64, 32, 32, 48, 3, 1, 1),
    (2, 44, 13, 17, 101, 3, 1, 1),
    (3, 8, 9, 9, 16, 3, 1, 1),
    (1, 24, 20, 20, 45, 1, 1, 0),
    (2, 72, 14, 14, 24, 1, 1, 0),
    (1, 100, 15, 11, 130, 3, 2, 1),
    (2, 130, 9, 10, 260, 3, 1, 1),
    (1, 64, 28, 28, 128, 1, 2, 0),
    (2, 16, 12, 12, 300, 3, 1, 0),
    (1, 40, 23, 23, 58, 7, 2, 3),
    (5, 187, 8, 8, 171, 3, 1, 1),
    (3, 212, 2, 2, 198, 3, 1, 1),
    (1, 320, 7, 7, 1280, 1, 1, 0),
]


@pytest.mark.parametrize("kernel", ["tensor", "direct"])
@pytest.mark.parametrize("case", DENSE_CASES)
def test_dense_task_parity(cp, case, kernel):
    N, C, H, W, K, R, stride, pad = case
    plan = check_task(cp, N, C, H, W, K, R, stride, pad, kernel=kernel)
    assert cp.KERNEL_NAMES[plan.kernel] == kernel


@pytest.mark.parametrize("kernel", ["tensor", "direct"])
def test_dense_task_epilogues(cp, kernel):
    check_task(cp, 2, 44, 14, 14, 64, 3, 1, 1, act="relu", with_res=True, kernel=kernel)
    check_task(cp, 1, 72, 14, 14, 24, 1, 1, 0, act="none", with_res=True, kernel=kernel)
    check_task(cp, 2, 24, 16, 16, 108, 1, 1, 0, act="relu6", kernel=kernel)
    check_task(cp, 2, 45, 16, 16, 58, 3, 1, 1, act="relu", pool="max2x2", kernel=kernel)
    check_task(cp, 1, 64, 8, 8, 64, 3, 1, 1, act="none", kernel=kernel)


@pytest.mark.parametrize("case", [
    # N, C, HW, K: fused in the filter-major epilogue (Q = 32, 16, 4), in the pixel-major epilogue (Q = 8, 2),
    # in the split-K finalize kernel (few tiles), and as a separate pass (Q not a power of two)
    (3, 45, 32, 58), (2, 101, 16, 96), (5, 20, 4, 40), (4, 171, 8, 163), (40, 64, 2, 243), (2, 250, 4, 212),
    (1, 24, 12, 32), (1, 200, 12, 200)])
def test_fused_maxpool(cp, case):
    N, C, HW, K = case
    check_task(cp, N, C, HW, HW, K, 3, 1, 1, act="relu", pool="max2x2", kernel="tensor")


def test_pointwise_tasks_as_flat_matrix_products(cp):
    # 1x1 stride-1 tasks with enough pixels run on the patch kernel with all pixels viewed as one row: ragged last tile,
    # residual through the staging buffer, several filter tiles, channel counts off the 16 / 64 grid
    plan = check_task(cp, 8, 24, 56, 56, 108, 1, 1, 0, act="relu6", kernel="tensor")
    assert plan.variant == 1
    check_task(cp, 3, 108, 57, 59, 24, 1, 1, 0, act="none", with_res=True, kernel="tensor")
    check_task(cp, 5, 72, 40, 41, 300, 1, 1, 0, act="relu", kernel="tensor")
    check_task(cp, 64, 320, 7, 7, 1280, 1, 1, 0, act="relu6", kernel="tensor")
    # one filter tile and a pixel pitch of an odd number of 16-byte pieces (or 32 bytes): the tile is staged as it lies
    # in memory and leaves by one bulk copy (one and two 64-filter groups, with and without residual, ragged last tile)
    for case in ((12, 16, 50, 53, 72, "relu6", False), (6, 32, 47, 50, 16, "none", False), (4, 150, 45, 46, 40, "relu6", True),
                 (8, 48, 45, 46, 133, "relu", True)):
        N, C, H, W, K, act, res = case
        plan = check_task(cp, N, C, H, W, K, 1, 1, 0, act=act, with_res=res, kernel="tensor")
        assert plan.variant == 2, case


def test_stems_on_the_patch_kernel(cp):
    # enough tiles for the patch kernel: the input is regrouped into 16-channel pixels (stride 1 and 2)
    plan = check_task(cp, 16, 3, 64, 64, 64, 7, 2, 3, kernel="tensor")
    assert plan.variant == 1 and plan.workspace_bytes > 0     # the workspace holds the regrouped input
    check_task(cp, 16, 3, 62, 60, 32, 3, 2, 1, act="relu6", kernel="tensor")
    check_task(cp, 24, 3, 32, 32, 45, 3, 1, 1, kernel="tensor")
    check_task(cp, 20, 4, 36, 28, 24, 5, 1, 2, act="none", kernel="tensor")


@pytest.mark.parametrize("case", [
    # N, C, H, W, K, R, stride, pad: fused in the patch kernel (tiles around whole 3x3 windows, even and odd extents),
    # and as a separate pass (few tiles; a task with wrap-around slots)
    (16, 3, 64, 64, 64, 7, 2, 3), (12, 3, 60, 52, 40, 7, 2, 3), (40, 3, 30, 30, 24, 3, 1, 1),
    (2, 3, 64, 64, 64, 7, 2, 3), (2, 16, 30, 30, 24, 3, 1, 1)])
def test_maxpool_3x3_stride_2(cp, case):
    N, C, H, W, K, R, stride, pad = case
    plan = check_task(cp, N, C, H, W, K, R, stride, pad, act="relu", pool="max3x3s2", kernel="tensor")
    P = oracle.out_size(H, R, stride, pad)
    assert plan.out_h == (P - 1) // 2 + 1


def test_maxpool_3x3_stride_2_pooled_by_the_epilogue_warps(cp, monkeypatch):
    # the fused pool normally runs on separate pooling warps; the measurement switch (read at launch time) selects the
    # instantiation in which the epilogue warps pool the tile themselves, which plans with one staging buffer use
    monkeypatch.setenv("CPRUNE_PATCH_NO_POOL_WARPS", "1")
    check_task(cp, 16, 3, 64, 64, 64, 7, 2, 3, act="relu", pool="max3x3s2", kernel="tensor")
    check_task(cp, 40, 3, 30, 30, 24, 3, 1, 1, act="none", pool="max3x3s2", kernel="tensor")
    monkeypatch.delenv("CPRUNE_PATCH_NO_POOL_WARPS")
    check_task(cp, 40, 3, 30, 30, 24, 3, 1, 1, act="none", pool="max3x3s2", kernel="tensor")


@pytest.mark.parametrize("case", [
    # tasks of the benchmarked models at their full batch-64 sizes, i.e. in the launch configuration bench.py times:
    # N, C, H, W, K, R, stride, pad, groups, act, residual, pool
    (64, 3, 224, 224, 64, 7, 2, 3, 1, "relu", False, "max3x3s2"),      # ResNet stem with its pool (patch kernel, regrouped)
    (64, 64, 56, 56, 44, 3, 1, 1, 1, "relu", False, None),             # stage 1 conv1 (patch kernel, resident filters)
    (64, 179, 14, 14, 256, 3, 1, 1, 1, "relu", True, None),            # stage 3 conv2 + residual (patch kernel, streamed)
    (64, 512, 7, 7, 358, 3, 1, 1, 1, "relu", False, None),             # stage 4 (im2col kernel)
    (64, 64, 56, 56, 89, 3, 2, 1, 1, "relu", False, None),             # stride-2 3x3 (im2col kernel)
    (64, 16, 112, 112, 72, 1, 1, 0, 1, "relu6", False, None),          # MobileNetV2 expand (flat matrix product)
    (64, 108, 56, 56, 24, 1, 1, 0, 1, "none", True, None),             # MobileNetV2 project + residual (flat, one bulk store per tile)
    (64, 72, 112, 112, 72, 3, 2, 1, 72, "relu6", False, None)])        # depthwise, stride 2
def test_full_size_tasks_on_sampled_outputs(cp, case):
    N, C, H, W, K, R, stride, pad, groups, act, with_res, pool = case
    P, Q = oracle.out_size(H, R, stride, pad), oracle.out_size(W, R, stride, pad)
    x, w, b, res = wl.conv_task_tensors(31, N, C, H, W, K, R, R, groups, with_res, P, Q)
    y, plan = run_task(cp, x, w, b, stride, pad, groups, act, res, pool)
    rng = np.random.default_rng(5)
    n_pts = 192
    oh, ow = plan.out_h, plan.out_w
    pts = np.stack([rng.integers(0, N, n_pts), rng.integers(0, oh, n_pts), rng.integers(0, ow, n_pts),
                    rng.integers(0, K, n_pts)], axis=1)
    # corners and edges are where padding, ragged tiles and pooling windows go wrong
    pts[:8, 1:3] = [[0, 0], [0, ow - 1], [oh - 1, 0], [oh - 1, ow - 1], [0, ow // 2], [oh // 2, 0], [oh - 1, ow // 2], [oh // 2, ow - 1]]
    pts[:4, 0] = [0, N - 1, 0, N - 1]
    if pool is None:
        ref, bound = oracle.conv2d_points(x, w, b, stride, pad, groups, act, res, pts)
    else:
        ref = np.full(n_pts, -np.inf)
        bound = np.zeros(n_pts)
        for di in range(3):
            for dj in range(3):
                q = pts.copy()
                q[:, 1] = 2 * pts[:, 1] - 1 + di
                q[:, 2] = 2 * pts[:, 2] - 1 + dj
                inside = (q[:, 1] >= 0) & (q[:, 1] < P) & (q[:, 2] >= 0) & (q[:, 2] < Q)
                v, bd = oracle.conv2d_points(x, w, b, stride, pad, groups, act, res, q[inside])
                ref[inside] = np.maximum(ref[inside], v)
                bound[inside] = np.maximum(bound[inside], bd)
    got = y[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]]
    worst = np.max(np.abs(got - ref) / (bound + 1e-30))
    assert worst <= TOL, (worst, pts[np.argmax(np.abs(got - ref) / (bound + 1e-30))])
    assert np.all(y[..., K:] == 0)


@pytest.mark.parametrize("C", [64, 65, 66, 67, 68, 69, 70, 71, 72, 73, 79, 80, 81])
def test_every_channel_residue(cp, C):
    # C and K sweep the residues modulo 8 and 16 around a 64-channel block boundary
    check_task(cp, 1, C, 10, 10, C + 3, 3, 1, 1, kernel="tensor")


@pytest.mark.parametrize("kernel", ["tensor", "direct"])
def test_three_channel_stems(cp, kernel):
    # 3 input channels: the tensor-core kernel packs 8 taps x 8 padded channels into one K block
    plan = check_task(cp, 1, 3, 32, 32, 45, 3, 1, 1, kernel=kernel)
    assert cp.KERNEL_NAMES[plan.kernel] == kernel
    check_task(cp, 1, 3, 37, 37, 64, 7, 2, 3, kernel=kernel)
    check_task(cp, 2, 3, 30, 30, 32, 3, 2, 1, act="relu6", kernel=kernel)
    check_task(cp, 3, 3, 64, 64, 64, 7, 2, 3, kernel=kernel)
    check_task(cp, 2, 5, 21, 19, 24, 5, 1, 2, kernel=kernel)
    assert cp.KERNEL_NAMES[cp.cprune_task_plan(1, 3, 224, 224, 64, 7, 7, 2, 3).kernel] == "tensor"


@pytest.mark.parametrize("C,H,W,stride", [(32, 16, 16, 1), (72, 15, 17, 2), (108, 14, 14, 1), (144, 7, 9, 2),
                                          (8, 5, 5, 1), (432, 14, 14, 2), (720, 7, 7, 1), (20, 3, 2, 1)])
def test_depthwise_task_parity(cp, C, H, W, stride):
    plan = check_task(cp, 2, C, H, W, C, 3, stride, 1, groups=C, act="relu6")
    assert cp.KERNEL_NAMES[plan.kernel] == "depthwise"


def test_task_runs_are_deterministic(cp):
    x, w, b, _ = wl.conv_task_tensors(5, 2, 89, 14, 14, 128, 3, 3)
    plan = cp.cprune_task_plan(2, 89, 14, 14, 128, 3, 3, 1, 1)
    xb = cp.cprune_cast_input(_dev(x))
    wp, bp = cp.cprune_pack_weights(plan, _dev(w), _dev(b))
    a = cp.cprune_task_run(plan, xb, wp, bp).clone()
    c = cp.cprune_task_run(plan, xb, wp, bp)
    cp.cprune_poll_device_status()
    assert torch.equal(a, c)


def test_channel_subset_property_on_the_gpu(cp):
    # pruning to any K gives the same values as the matching channels of the full-width task
    x, w, b, _ = wl.conv_task_tensors(6, 1, 64, 14, 14, 96, 3, 3)
    full, _ = run_task(cp, x, w, b, 1, 1)
    for keep in (24, 37, 72, 95):
        kept = oracle.select_indices(w, keep)
        y, _ = run_task(cp, x, w[kept], b[kept], 1, 1)
        assert np.array_equal(y[..., :keep], full[..., kept])


def test_task_argument_errors(cp):
    bad = [dict(N=0), dict(C=-1), dict(stride=0), dict(pad=-1), dict(R=40, S=40)]
    base = dict(N=1, C=8, H=8, W=8, K=8, R=3, S=3, stride=1, pad=1)
    for chg in bad:
        a = dict(base, **chg)
        with pytest.raises(cp.CpruneError) as e:
            cp.cprune_task_plan(a["N"], a["C"], a["H"], a["W"], a["K"], a["R"], a["S"], a["stride"], a["pad"])
        assert e.value.status == 1
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_task_plan(1, 8, 8, 8, 16, 3, 3, 1, 1, groups=2)
    assert e.value.status == 2
    plan = cp.cprune_task_plan(1, 8, 8, 8, 8, 3, 3, 1, 1, residual=True)
    xb = torch.zeros((1, 8, 8, 8), dtype=torch.bfloat16, device="cuda")
    wp, bp = cp.cprune_pack_weights(plan, torch.zeros((8, 8, 3, 3), device="cuda"), torch.zeros(8, device="cuda"))
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_task_run(plan, xb, wp, bp, None)          # the plan wants a residual
    assert e.value.status == 1


# ------------------------------------------------------------------ tail operators

def test_cast_pool_gap_fc(cp):
    x = wl.normal_f32(31, 0, (2, 9, 11, 13))
    xb = cp.cprune_cast_input(_dev(x))
    got = xb.float().cpu().numpy()
    assert np.array_equal(got[..., :13], oracle.round_bf16(x)) and np.all(got[..., 13:] == 0)
    xr = oracle.round_bf16(x)
    for k, s, p in ((3, 2, 1), (2, 2, 0)):
        y = cp.cprune_maxpool(xb, 13, k, s, p).float().cpu().numpy()
        assert np.array_equal(y[..., :13], oracle.maxpool(xr, k, s, p))
    g = cp.cprune_global_avgpool(xb, 13).float().cpu().numpy()
    ref = oracle.gap(xr)
    assert np.max(np.abs(g[:, :13] - ref)) <= 2.0 ** -8 * np.max(np.abs(ref)) + 1e-6
    a = wl.normal_f32(31, 1, (5, 243))
    w = wl.normal_f32(31, 2, (37, 243), 0.1)
    b = wl.normal_f32(31, 3, (37,), 0.1)
    ab = cp.cprune_cast_input(_dev(a))
    wp, bp = cp.cprune_fc_pack(_dev(w), _dev(b))
    ref, bound = oracle.fc(a, w, b, "relu", with_bound=True)
    y32 = cp.cprune_fc(ab, 243, wp, bp, 37, "relu", out_f32=True).cpu().numpy()
    assert np.max(np.abs(y32 - ref) / bound) <= TOL
    y16 = cp.cprune_fc(ab, 243, wp, bp, 37, "relu").float().cpu().numpy()
    assert np.max(np.abs(y16[:, :37] - ref) / bound) <= TOL and np.all(y16[:, 37:] == 0)
    assert np.array_equal(cp.cprune_widen_output(ab).cpu().numpy(), ab.float().cpu().numpy())


# ------------------------------------------------------------------ whole models

def model_parity(cp, name, batch, hw=None, kernel="auto"):
    from paper_2207_01260_b200.pipeline import PrunedNetwork
    table = wl.MODELS[name]()
    if hw:
        table["input"] = (hw, hw, table["input"][2])
    weights = wl.model_weights(table)
    x = wl.model_input(table, batch)
    net = PrunedNetwork(table, weights, batch, kernel=kernel)
    cp.cprune_poll_device_status()
    pw, kept = oracle.prune_model(table, weights)
    for lname, idx in kept.items():                     # selection is bit-exact, layer by layer
        assert np.array_equal(net.kept[lname].cpu().numpy(), idx), lname
    for lname, (w, b) in pw.items():
        gw, gb = net.params[lname]
        assert gw.cpu().numpy().tobytes() == w.tobytes() and gb.cpu().numpy().tobytes() == b.tobytes(), lname
    logits = net.run(_dev(x))
    cp.cprune_poll_device_status()
    logits2 = net.run(_dev(x), use_graph=True)
    logits3 = net.run(_dev(x), use_graph=True).clone()
    cp.cprune_poll_device_status()
    got = logits.cpu().numpy()
    assert np.array_equal(got, logits2.cpu().numpy()) and np.array_equal(got, logits3.cpu().numpy())
    # the host-buffer entry point (copies inside the call, two alternating device buffers)
    xh = torch.from_numpy(np.ascontiguousarray(x)).pin_memory()
    lh = torch.empty(got.shape, dtype=torch.float32).pin_memory()
    for _ in range(3):
        net.run_host(xh, lh)
    torch.cuda.synchronize()
    cp.cprune_poll_device_status()
    assert np.array_equal(lh.numpy(), got)
    matched = oracle.model_ref(table, pw, x, matched=True)
    exact = oracle.model_ref(table, pw, x, matched=False)
    rel = np.linalg.norm(got - matched) / np.linalg.norm(matched)
    rel_exact = np.linalg.norm(got - exact) / np.linalg.norm(exact)
    assert rel <= 1e-2, (name, rel, rel_exact)
    # top-1 must agree wherever the oracle's own top-2 gap exceeds the error the two sides can differ by
    err = np.max(np.abs(got - matched), axis=1)
    srt = np.sort(matched, axis=1)
    gap = srt[:, -1] - srt[:, -2]
    decided = gap > 2 * err
    assert np.array_equal(np.argmax(got, 1)[decided], np.argmax(matched, 1)[decided])
    assert decided.mean() >= 0.5, "too many near-ties to say anything"
    return net, rel, rel_exact


def test_vgg16_cifar_parity(cp):
    model_parity(cp, "vgg16_cifar", 4)
    model_parity(cp, "vgg16_cifar", 1, kernel="direct")


def test_resnet18_parity(cp):
    net, _, _ = model_parity(cp, "resnet18", 2)
    kinds = {cp.KERNEL_NAMES[i["kernel"]] for i in net.conv_launch_info().values()}
    assert kinds == {"tensor"}


def test_mobilenet_v2_parity(cp):
    net, _, _ = model_parity(cp, "mobilenet_v2", 2)
    kinds = {cp.KERNEL_NAMES[i["kernel"]] for i in net.conv_launch_info().values()}
    assert kinds == {"tensor", "depthwise"}


def test_intermediate_activations_match(cp):
    from paper_2207_01260_b200.pipeline import PrunedNetwork
    table = wl.resnet18()
    table["input"] = (64, 64, 3)
    weights = wl.model_weights(table)
    x = wl.model_input(table, 2)
    net = PrunedNetwork(table, weights, 2)
    net.run(_dev(x))
    pw, _ = oracle.prune_model(table, weights)
    _, tensors = oracle.model_ref(table, pw, x, matched=True, keep_tensors=True)
    # the stem's 3x3 max-pool is fused into the stem task: its unpooled output "s0" is never stored
    for name in ("p0", "l1b1_h", "l1b1_o", "l2b1_id", "l2b1_o", "l4b2_o", "g"):
        got = net.activation(name)
        ref = tensors[name].reshape(got.shape)
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= 1e-2, (name, rel)
    net = PrunedNetwork(table, weights, 2, fuse_pool=False)
    net.run(_dev(x))
    for name in ("s0", "p0"):
        got = net.activation(name)
        ref = tensors[name].reshape(got.shape)
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= 1e-2, (name, rel)


def test_plan_cache_shares_repeated_shapes(cp):
    from paper_2207_01260_b200.pipeline import PrunedNetwork
    table = wl.resnet18()
    net = PrunedNetwork(table, wl.model_weights(table), 1)
    handles = {p.handle.value for p in net.plans.values()}
    assert len(net.plans) == 20 and len(handles) == 15          # 20 conv tasks, 15 distinct shapes

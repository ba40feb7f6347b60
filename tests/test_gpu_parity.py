"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

TOL = 2e-2          # the contract: max |err| <= TOL * (|b| + sum |x||w| + |res|) per output element, against the exact oracle
# The engineering bound, against the matched oracle (x, w and the residual rounded to bfloat16, float64 arithmetic): what
# is left is the rounding of the stored result to bfloat16 (half a unit in the 8th significant bit: 2^-8 |ref|, taken
# twice here) and the float32 accumulation on the device (a few 1e-6 of the scale; 1e-4 allows for worst-case orders).
# A dropped channel block, tap or tile-edge column changes an output by about 1e-2 of the scale and fails this check.
MATCH_REL, MATCH_ABS = 2.0 ** -7, 1e-4
WORST = {}          # test name -> (worst contract ratio, worst matched ratio), printed at the end of the session


def check_values(name, got, exact, bound, matched, bound_m):
    """got vs the exact oracle under the contract and vs the matched oracle under the engineering bound."""
    r1 = float(np.max(np.abs(got - exact) / (bound + 1e-30)))
    r2 = float(np.max(np.abs(got - matched) / (MATCH_REL * np.abs(matched) + MATCH_ABS * bound_m + 1e-30)))
    prev = WORST.get(name, (0.0, 0.0))
    WORST[name] = (max(prev[0], r1), max(prev[1], r2))
    assert r1 <= TOL, (name, "contract", r1)
    assert r2 <= 1.0, (name, "matched", r2, np.unravel_index(np.argmax(np.abs(got - matched) - MATCH_REL * np.abs(matched) - MATCH_ABS * bound_m), got.shape))
    return r1, r2


@pytest.fixture(scope="module", autouse=True)
def _report_worst_ratios():
    yield
    if WORST:
        print("\nworst error ratios (contract: err / (2e-2-scale bound) must be <= 2e-2; matched: must be <= 1):")
        for k in sorted(WORST):
            print("  %-58s contract %.2e   matched %.3f" % (k, WORST[k][0], WORST[k][1]))


@pytest.fixture(scope="module")
def cp():
    import paper_2207_01260_b200 as m
    m.lib()
    return m


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_task(cp, x, w, b, stride, pad, groups=1, act="relu", res=None, pool=None, kernel="auto", flags=()):
    N, H, W, C = x.shape
    K, _, R, S = w.shape
    plan = cp.cprune_task_plan(N, C, H, W, K, R, S, stride, pad, groups, act, res is not None, pool, kernel, flags)
    xb = cp.cprune_cast_input(_dev(x))
    wp, bp = cp.cprune_pack_weights(plan, _dev(w), _dev(b))
    rb = cp.cprune_cast_input(_dev(res)) if res is not None else None
    y = cp.cprune_task_run(plan, xb, wp, bp, rb)
    cp.cprune_poll_device_status()
    return y.float().cpu().numpy(), plan


def _pooled(ref, bound, pool):
    # the error bound of a maximum is at most the largest bound in its window
    if pool == "max3x3s2":
        return oracle.maxpool(ref, 3, 2, 1), oracle.maxpool(bound, 3, 2, 1)
    if pool:
        return oracle.maxpool(ref, 2, 2, 0), oracle.maxpool(bound, 2, 2, 0)
    return ref, bound


def check_task(cp, N, C, H, W, K, R, stride, pad, groups=1, act="relu", with_res=False, pool=None, kernel="auto",
               seed=11, flags=(), name=None):
    P, Q = oracle.out_size(H, R, stride, pad), oracle.out_size(W, R, stride, pad)
    x, w, b, res = wl.conv_task_tensors(seed, N, C, H, W, K, R, R, groups, with_res, P, Q)
    y, plan = run_task(cp, x, w, b, stride, pad, groups, act, res, pool, kernel, flags)
    ref, bound = _pooled(*oracle.conv2d(x, w, b, stride, pad, groups, act, res, with_bound=True), pool)
    rb = oracle.round_bf16
    ref_m, bound_m = _pooled(*oracle.conv2d(rb(x), rb(w), b, stride, pad, groups, act, None if res is None else rb(res),
                                            with_bound=True), pool)
    assert y.shape == (N, plan.out_h, plan.out_w, plan.k_pad)
    assert np.all(y[..., K:] == 0), "pad lanes must be written as zero"
    label = name or "task N%d C%d %dx%d K%d R%d s%d g%d %s%s%s %s" % (N, C, H, W, K, R, stride, groups, act, "+res" if with_res else "",
                                                                       "+" + pool if pool else "", kernel)
    check_values(label, y[..., :K], ref, bound, ref_m, bound_m)
    assert np.max(np.abs(y[..., :K] - ref)) > 0 or np.max(np.abs(ref)) == 0   # bf16 data cannot be bit-exact against float64
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
        ref_m, bound_m = oracle.conv2d(oracle.round_bf16(x), oracle.round_bf16(rw), rb, 1, 1, 1, "relu", with_bound=True)
        assert y.shape == (1, 32, 32, 48)
        check_values("config 1 (%s)" % kernel, y, ref, bound, ref_m, bound_m)


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
    # one filter tile: the tile is staged pixel by pixel as it lies in memory (variant 2).  A pixel pitch of an odd number of
    # 16-byte pieces (or 32 bytes) leaves by one bulk copy (one and two 64-filter groups, with and without residual, ragged
    # last tile); an even number is staged one piece longer and leaves by one tiled copy whose box is wider than the tensor
    # (without residual; with one such tasks keep the 64-filter-wide stores of variant 1)
    for case in ((12, 16, 50, 53, 72, "relu6", False, 2), (6, 32, 47, 50, 16, "none", False, 2), (4, 150, 45, 46, 40, "relu6", True, 2),
                 (8, 48, 45, 46, 88, "relu", True, 2), (8, 48, 45, 46, 133, "relu", False, 2), (5, 24, 44, 45, 64, "relu", False, 2),
                 (7, 40, 33, 35, 32, "relu6", False, 2), (8, 48, 45, 46, 133, "relu", True, 1), (5, 24, 44, 45, 64, "none", True, 1)):
        N, C, H, W, K, act, res, variant = case
        plan = check_task(cp, N, C, H, W, K, 1, 1, 0, act=act, with_res=res, kernel="tensor")
        assert plan.variant == variant, case


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


def test_maxpool_3x3_stride_2_pooled_by_the_epilogue_warps(cp):
    # the fused pool normally runs on separate pooling warps; a plan flag selects the instantiation in which the epilogue
    # warps pool the tile themselves, which plans with one staging buffer use
    check_task(cp, 16, 3, 64, 64, 64, 7, 2, 3, act="relu", pool="max3x3s2", kernel="tensor", flags=("pool_on_epilogue_warps",))
    check_task(cp, 40, 3, 30, 30, 24, 3, 1, 1, act="none", pool="max3x3s2", kernel="tensor", flags=("pool_on_epilogue_warps",))
    check_task(cp, 40, 3, 30, 30, 24, 3, 1, 1, act="none", pool="max3x3s2", kernel="tensor")


def test_stride_1_tasks_on_the_im2col_kernel(cp):
    # the im2col kernel serves stride-1 tasks too when a plan asks for it (and whenever the patch kernel declines)
    for case in ((16, 64, 32, 32, 48, 3, 1, 1), (8, 130, 14, 14, 260, 3, 1, 1), (8, 24, 56, 56, 108, 1, 1, 0)):
        plan = check_task(cp, *case, kernel="tensor", flags=("im2col_only",))
        assert plan.variant == 0


def big_task_tensors(seed, N, C, H, W, K, R, groups, with_res, P, Q, base=4):
    """Tensors of a full-size task (drawing every image from the generator would take minutes over a whole model)."""
    return wl.conv_task_tensors_tiled(seed, N, C, H, W, K, R, R, groups, with_res, P, Q, base)


def sample_points(rng, N, oh, ow, K, n_pts):
    pts = np.stack([rng.integers(0, N, n_pts), rng.integers(0, oh, n_pts), rng.integers(0, ow, n_pts),
                    rng.integers(0, K, n_pts)], axis=1)
    # corners and edges are where padding, ragged tiles and pooling windows go wrong
    pts[:8, 1:3] = [[0, 0], [0, ow - 1], [oh - 1, 0], [oh - 1, ow - 1], [0, ow // 2], [oh // 2, 0], [oh - 1, ow // 2], [oh // 2, ow - 1]]
    pts[:4, 0] = [0, N - 1, 0, N - 1]
    pts[8:12, 3] = [0, K - 1, K // 2, max(K - 2, 0)]
    return pts


def points_reference(x, w, b, stride, pad, groups, act, res, pool, pts, P, Q):
    """Oracle values and error scales at sampled OUTPUT coordinates (after the optional pool)."""
    if pool is None:
        return oracle.conv2d_points(x, w, b, stride, pad, groups, act, res, pts)
    win, st, off = (3, 2, 1) if pool == "max3x3s2" else (2, 2, 0)
    ref = np.full(len(pts), -np.inf)
    bound = np.zeros(len(pts))
    for di in range(win):
        for dj in range(win):
            q = pts.copy()
            q[:, 1] = st * pts[:, 1] - off + di
            q[:, 2] = st * pts[:, 2] - off + dj
            inside = (q[:, 1] >= 0) & (q[:, 1] < P) & (q[:, 2] >= 0) & (q[:, 2] < Q)
            v, bd = oracle.conv2d_points(x, w, b, stride, pad, groups, act, res, q[inside])
            ref[inside] = np.maximum(ref[inside], v)
            bound[inside] = np.maximum(bound[inside], bd)
    return ref, bound


def check_task_sampled(cp, label, N, C, H, W, K, R, stride, pad, groups, act, with_res, pool, seed, n_pts=160, tensors=None):
    P, Q = oracle.out_size(H, R, stride, pad), oracle.out_size(W, R, stride, pad)
    x, w, b, res = tensors if tensors is not None else big_task_tensors(seed, N, C, H, W, K, R, groups, with_res, P, Q)
    y, plan = run_task(cp, x, w, b, stride, pad, groups, act, res, pool)
    pts = sample_points(np.random.default_rng(seed), N, plan.out_h, plan.out_w, K, n_pts)
    ref, bound = points_reference(x, w, b, stride, pad, groups, act, res, pool, pts, P, Q)
    rb = oracle.round_bf16
    ref_m, bound_m = points_reference(rb(x), rb(w), b, stride, pad, groups, act, None if res is None else rb(res), pool, pts, P, Q)
    got = y[pts[:, 0], pts[:, 1], pts[:, 2], pts[:, 3]]
    check_values(label, got, ref, bound, ref_m, bound_m)
    assert np.all(y[..., K:] == 0)
    return plan


def model_tasks(name, batch):
    """The distinct conv tasks of a pruned model as the pipeline plans them: (key, layer names)."""
    table = wl.MODELS[name]()
    m = wl.pruned_shapes(table)
    sz = wl.spatial_sizes(m)
    layers = m["layers"]
    readers = {}
    for l in layers:
        for key in ("in", "res"):
            if l.get(key) is not None:
                readers.setdefault(l[key], []).append(l["name"])
    out = {}
    for a, nxt in zip(layers, layers[1:] + [None]):
        if a["kind"] != "conv":
            continue
        pool = a.get("pool")
        if (nxt is not None and nxt["kind"] == "maxpool" and nxt["in"] == a["out"] and pool is None and a.get("res") is None
                and (nxt["k"], nxt["stride"], nxt["pad"]) == (3, 2, 1) and readers.get(a["out"]) == [nxt["name"]]):
            pool = "max3x3s2"           # the pipeline folds such a pool into the task
        h, w = sz[a["in"]]
        key = (batch, a["C"], h, w, a["K"], a["R"], a["stride"], a["pad"], a["groups"] if a["groups"] > 1 else 1, a["act"],
               a.get("res") is not None, pool)
        out.setdefault(key, []).append(a["name"])
    return out


BENCH_MODELS = [("resnet18", 64), ("mobilenet_v2", 64), ("vgg16_cifar", 128), ("resnet18", 1), ("mobilenet_v2", 1), ("vgg16_cifar", 1)]


@pytest.mark.parametrize("name,batch", BENCH_MODELS)
def test_every_plan_of_the_benchmarked_models_on_sampled_outputs(cp, name, batch):
    # every distinct task of the pruned model at the batch bench.py times it with, i.e. the very plans (tiles, split
    # reductions, kernel variants) of the benchmark, each checked on sampled outputs
    tasks = model_tasks(name, batch)
    families = {}
    for n_task, (key, names) in enumerate(tasks.items()):
        N, C, H, W, K, R, stride, pad, groups, act, with_res, pool = key
        plan = check_task_sampled(cp, "%s b%d %s" % (name, batch, names[0]), N, C, H, W, K, R, stride, pad, groups, act, with_res,
                                  pool, seed=100 + n_task)
        fam = cp.KERNEL_NAMES[plan.kernel]
        assert fam == ("depthwise" if groups > 1 else "tensor"), (names, fam)      # no dense task falls off the tensor cores
        families[names[0]] = (fam, plan.variant, plan.splits, plan.tile_m, plan.tile_n)
    print("\n%s batch %d: %d distinct tasks" % (name, batch, len(tasks)))
    for k, v in families.items():
        print("  %-14s %s variant %d splits %d tile %dx%d" % ((k,) + v))
    if (name, batch) == ("resnet18", 64):
        assert len(tasks) == 15
        assert families["stem"][1] == 1 and families["l1b1_conv1"][1] == 1 and families["l3b1_conv2"][1] == 1
    if (name, batch) == ("mobilenet_v2", 64):
        assert len(tasks) == 30
        assert families["b2_exp"][1] in (1, 2) and families["b3_proj"][1] in (1, 2)


def sweep_keep_counts(k_full):
    """Kept filter counts checked per swept shape: full width, one less, and every 16 n +- 1 down to a quarter."""
    lo = (k_full + 3) // 4
    ks = {k_full, k_full - 1, lo}
    for n in range(k_full // 16 + 1):
        for k in (16 * n - 1, 16 * n + 1):
            if lo <= k <= k_full:
                ks.add(k)
    return sorted(k for k in ks if k >= 1)


def test_sweep_parity_over_the_kept_filter_count(cp):
    # every distinct conv shape of the models, with the filters that L1 selection keeps at each checked count (for
    # depthwise shapes the input channels go with the filters), at batch 2 on sampled outputs
    n_points = 0
    for si, shp in enumerate(wl.sweep_shapes()):
        dw = shp["groups"] > 1
        R, stride, pad, act = shp["R"], shp["stride"], shp["pad"], shp["act"]
        P, Q = oracle.out_size(shp["H"], R, stride, pad), oracle.out_size(shp["W"], R, stride, pad)
        x, w, b, _ = wl.conv_task_tensors(500 + si, 2, shp["C"], shp["H"], shp["W"], shp["K"], R, R, shp["groups"])
        for K in sweep_keep_counts(shp["K"]):
            kept = oracle.select_indices(w, K)
            xs = np.ascontiguousarray(x[..., kept]) if dw else x
            label = "sweep %s/%s" % (shp["model"], shp["layer"])
            plan = check_task_sampled(cp, label, 2, K if dw else shp["C"], shp["H"], shp["W"], K, R, stride, pad, K if dw else 1, act,
                                      False, None, seed=si * 1000 + K, n_pts=64, tensors=(xs, w[kept], b[kept], None))
            assert cp.KERNEL_NAMES[plan.kernel] == ("depthwise" if dw else "tensor")
            n_points += 1
    assert n_points > 800


@pytest.mark.parametrize("batch", [64, 1])
def test_sweep_parity_at_the_benchmarked_batches(cp, batch):
    # the sweep's own launch configurations: every shape at three kept counts (full, about 60 %, a quarter)
    for si, shp in enumerate(wl.sweep_shapes()):
        dw = shp["groups"] > 1
        R, stride, pad, act = shp["R"], shp["stride"], shp["pad"], shp["act"]
        P, Q = oracle.out_size(shp["H"], R, stride, pad), oracle.out_size(shp["W"], R, stride, pad)
        x, w, b, _ = big_task_tensors(700 + si, batch, shp["C"], shp["H"], shp["W"], shp["K"], R, shp["groups"], False, P, Q, base=2)
        for K in sorted({shp["K"], (3 * shp["K"]) // 5 + 1, (shp["K"] + 3) // 4}):
            kept = oracle.select_indices(w, K)
            xs = np.ascontiguousarray(x[..., kept]) if dw else x
            check_task_sampled(cp, "sweep b%d %s/%s" % (batch, shp["model"], shp["layer"]), batch, K if dw else shp["C"], shp["H"],
                               shp["W"], K, R, stride, pad, K if dw else 1, act, False, None, seed=si * 1000 + K, n_pts=64,
                               tensors=(xs, w[kept], b[kept], None))


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


@pytest.mark.parametrize("C,H,W,stride", [(72, 56, 56, 2), (120, 28, 28, 1), (90, 17, 15, 2), (576, 14, 14, 2), (1152, 7, 7, 1),
                                          (8, 6, 5, 1), (20, 3, 2, 1)])
def test_depthwise_5x5_task_parity(cp, C, H, W, stride):
    # MnasNet's 5x5 depthwise layers (pad 2): ragged tiles, channel counts off the 8 / 64 grid, images smaller than the filter
    plan = check_task(cp, 2, C, H, W, C, 5, stride, 2, groups=C, act="relu")
    assert cp.KERNEL_NAMES[plan.kernel] == "depthwise"
    check_task(cp, 1, C, H, W, C, 5, stride, 2, groups=C, act="none", with_res=(stride == 1))


def test_task_runs_are_deterministic(cp):
    x, w, b, _ = wl.conv_task_tensors(5, 2, 89, 14, 14, 128, 3, 3)
    plan = cp.cprune_task_plan(2, 89, 14, 14, 128, 3, 3, 1, 1)
    xb = cp.cprune_cast_input(_dev(x))
    wp, bp = cp.cprune_pack_weights(plan, _dev(w), _dev(b))
    a = cp.cprune_task_run(plan, xb, wp, bp).clone()
    c = cp.cprune_task_run(plan, xb, wp, bp)
    cp.cprune_poll_device_status()
    assert torch.equal(a, c)


@pytest.mark.parametrize("case", [(1, 64, 14, 14, 96, 3, 1, 1), (4, 96, 14, 14, 576, 1, 1, 0), (2, 128, 28, 28, 256, 3, 2, 1)])
def test_channel_subset_property_on_the_gpu(cp, case):
    # pruning to any K gives the same values as the matching channels of the full-width task: one full-width check
    # therefore vouches for every K of a sweep whose plans accumulate in the same order
    N, C, H, W, K, R, stride, pad = case
    x, w, b, _ = wl.conv_task_tensors(6, N, C, H, W, K, R, R)
    full, _ = run_task(cp, x, w, b, stride, pad)
    for keep in (K // 4, K // 3 + 5, (3 * K) // 4, K - 1):
        kept = oracle.select_indices(w, keep)
        y, _ = run_task(cp, x, w[kept], b[kept], stride, pad)
        assert np.array_equal(y[..., :keep], full[..., kept]), keep


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

def model_parity(cp, name, batch, hw=None, kernel="auto", oracle_images=None):
    """The whole pruned network on `batch` images against the oracle on the first `oracle_images` of them (images are
    independent; the plans are those of the full batch)."""
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
    n_ref = batch if oracle_images is None else min(batch, oracle_images)
    got = got[:n_ref]
    matched = oracle.model_ref(table, pw, x[:n_ref], matched=True)
    exact = oracle.model_ref(table, pw, x[:n_ref], matched=False)
    rel = np.linalg.norm(got - matched) / np.linalg.norm(matched)
    rel_exact = np.linalg.norm(got - exact) / np.linalg.norm(exact)
    assert rel <= 1e-2, (name, rel, rel_exact)
    # Top-1 must agree on every image whose answer is decided a priori: the oracle's top-2 gap exceeds twice the error
    # the tolerance allows a logit (1e-2 of the image's largest logit).  Images inside that margin have several correct
    # answers (random-weight networks have near-tied logits); they are counted, not judged.
    srt = np.sort(matched, axis=1)
    gap = srt[:, -1] - srt[:, -2]
    margin = 2.0 * 1e-2 * np.max(np.abs(matched), axis=1)
    decided = gap > margin
    agree = np.argmax(got, 1) == np.argmax(matched, 1)
    print("\n%s batch %d (%d images checked): rel-L2 %.2e matched / %.2e exact; top-1 agreement %d/%d raw, %d/%d decided a priori"
          % (name, batch, n_ref, rel, rel_exact, agree.sum(), n_ref, (agree & decided).sum(), decided.sum()))
    assert np.all(agree[decided]), np.nonzero(decided & ~agree)
    assert decided.mean() >= 0.25 or n_ref < 4, "too many near-ties to say anything"
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


@pytest.mark.parametrize("name,batch,oracle_images", [("resnet18", 64, 12), ("mobilenet_v2", 64, 12), ("vgg16_cifar", 128, 32),
                                                      ("vgg16_cifar", 1, 1), ("resnet18", 1, 1), ("mobilenet_v2", 1, 1)])
def test_model_parity_at_the_benchmarked_batch(cp, name, batch, oracle_images):
    net, _, _ = model_parity(cp, name, batch, oracle_images=oracle_images)
    kinds = {cp.KERNEL_NAMES[i["kernel"]] for i in net.conv_launch_info().values()}
    assert "direct" not in kinds


def test_mnasnet_parity(cp):
    net, _, _ = model_parity(cp, "mnasnet1_0", 2)
    kinds = {cp.KERNEL_NAMES[i["kernel"]] for i in net.conv_launch_info().values()}
    assert kinds == {"tensor", "depthwise"}
    assert {net.plans[n].R for n in net.plans if n.endswith("_dw")} == {3, 5}
    model_parity(cp, "mnasnet1_0", 16, hw=96, oracle_images=4)


def block_tensors(seed, N, C_in, H, W, hidden, C_out):
    x = wl.normal_f32(seed, 0, (N, H, W, C_in))
    we = wl.normal_f32(seed, 1, (hidden, C_in, 1, 1), np.sqrt(2.0 / C_in))
    wd = wl.normal_f32(seed, 2, (hidden, 1, 3, 3), np.sqrt(2.0 / 9))
    wp = wl.normal_f32(seed, 3, (C_out, hidden, 1, 1), np.sqrt(2.0 / hidden))
    be, bd, bp = (wl.normal_f32(seed, 4 + j, (n,), 0.05) for j, n in enumerate((hidden, hidden, C_out)))
    return x, we, be, wd, bd, wp, bp


def block_reference(t, act, act_out, residual, matched):
    """The block as the chain of its three tasks in the oracle; matched: bf16 where the device rounds to bf16."""
    x, we, be, wd, bd, wp, bp = t
    rnd = oracle.round_bf16 if matched else (lambda a: np.asarray(a, dtype=np.float64))
    xr = rnd(x)
    h1 = rnd(oracle.conv2d(xr, rnd(we), be, 1, 0, 1, act))
    h2 = rnd(oracle.conv2d(h1, rnd(wd), bd, 1, 1, wd.shape[0], act))
    return oracle.conv2d(h2, rnd(wp), bp, 1, 0, 1, act_out, xr if residual else None, with_bound=True)


@pytest.mark.parametrize("case", [
    # N, C_in, H, W, hidden, C_out, act, residual: the stride-1 blocks of pruned MobileNetV2 at 14x14 and 7x7, then ragged
    # extents, channel counts off the 8 / 16 / 64 grid, one and several 64-channel chunks, relu (MnasNet) and no activation
    (3, 64, 14, 14, 288, 64, "relu6", True), (2, 64, 14, 14, 288, 96, "relu6", False), (2, 96, 14, 14, 432, 96, "relu6", True),
    (4, 160, 7, 7, 720, 160, "relu6", True), (2, 24, 9, 11, 100, 40, "relu", False), (1, 75, 13, 14, 75, 75, "none", True),
    (5, 8, 5, 4, 30, 12, "relu6", False), (2, 130, 12, 12, 64, 130, "relu", True), (1, 40, 7, 7, 200, 250, "relu", False)])
def test_fused_inverted_residual_block(cp, case):
    N, C_in, H, W, hidden, C_out, act, residual = case
    t = block_tensors(61, N, C_in, H, W, hidden, C_out)
    x, we, be, wd, bd, wp, bp = t
    blk = cp.cprune_block_plan(N, C_in, H, W, hidden, C_out, act, "none", residual)
    wq, bq = cp.cprune_block_pack(blk, _dev(we.reshape(hidden, C_in)), _dev(be), _dev(wd.reshape(hidden, 9)), _dev(bd),
                                  _dev(wp.reshape(C_out, hidden)), _dev(bp))
    y = cp.cprune_block_run(blk, cp.cprune_cast_input(_dev(x)), wq, bq).float().cpu().numpy()
    cp.cprune_poll_device_status()
    assert y.shape == (N, H, W, blk.k_pad) and np.all(y[..., C_out:] == 0)
    ref, bound = block_reference(t, act, "none", residual, matched=False)
    ref_m, bound_m = block_reference(t, act, "none", residual, matched=True)
    got = y[..., :C_out]
    r1 = float(np.max(np.abs(got - ref) / bound))
    # against the matched chain: the stored result's own rounding, plus what a differently rounded hidden value (float32
    # against float64 sums under the two bf16 roundings inside the block) can move: far below 1e-3 of the scale
    r2 = float(np.max(np.abs(got - ref_m) / (MATCH_REL * np.abs(ref_m) + 1e-3 * bound_m)))
    WORST["fused block %s" % (case,)] = (r1, r2)
    assert r1 <= TOL and r2 <= 1.0, (case, r1, r2)
    # the same three tasks run separately give the same values up to those rounding flips
    p1 = cp.cprune_task_plan(N, C_in, H, W, hidden, 1, 1, 1, 0, 1, act)
    p2 = cp.cprune_task_plan(N, hidden, H, W, hidden, 3, 3, 1, 1, hidden, act)
    p3 = cp.cprune_task_plan(N, hidden, H, W, C_out, 1, 1, 1, 0, 1, "none", residual)
    xb = cp.cprune_cast_input(_dev(x))
    a = cp.cprune_task_run(p1, xb, *cp.cprune_pack_weights(p1, _dev(we), _dev(be)))
    b = cp.cprune_task_run(p2, a, *cp.cprune_pack_weights(p2, _dev(wd), _dev(bd)))
    c = cp.cprune_task_run(p3, b, *cp.cprune_pack_weights(p3, _dev(wp), _dev(bp)), xb if residual else None)
    sep = c.float().cpu().numpy()[..., :C_out]
    assert np.max(np.abs(sep - got) / (MATCH_REL * np.abs(ref_m) + 1e-3 * bound_m)) <= 2.0


def test_fused_block_argument_errors_and_unsupported_shapes(cp):
    for args in ((2, 64, 28, 28, 288, 64), (2, 256, 14, 14, 512, 64), (2, 64, 14, 14, 288, 320)):   # image too large, C_in, C_out
        with pytest.raises(cp.CpruneError) as e:
            cp.cprune_block_plan(*args)
        assert e.value.status == 2
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_block_plan(2, 64, 14, 14, 288, 96, residual=True)        # a residual needs C_in == C_out
    assert e.value.status == 1
    a = cp.cprune_block_plan(2, 64, 14, 14, 288, 64, residual=True)
    b = cp.cprune_block_plan(2, 64, 14, 14, 288, 64, residual=True)
    assert a.handle.value == b.handle.value and a.unfused_bytes > 2 * a.algorithmic_bytes


def test_mobilenet_v2_with_and_without_fused_blocks(cp):
    from paper_2207_01260_b200.pipeline import PrunedNetwork
    table = wl.mobilenet_v2()
    weights = wl.model_weights(table)
    x = wl.model_input(table, 4)
    fused = PrunedNetwork(table, weights, 4, fuse_blocks=True)
    plain = PrunedNetwork(table, weights, 4, fuse_blocks=False)
    # the stride-1 blocks of the 14x14 and 7x7 stages, except the last one (320 filters do not fit one image's accumulator)
    assert sorted(fused.blocks) == sorted(["b8_exp", "b9_exp", "b10_exp", "b11_exp", "b12_exp", "b13_exp", "b15_exp", "b16_exp"])
    assert not PrunedNetwork(table, weights, 64).blocks and PrunedNetwork(table, weights, 2).blocks      # the default follows the batch
    assert fused.model.launches == plain.model.launches - sum(3 - (2 if b.splits > 1 else 1) for b in fused.blocks.values())
    a = fused.run(_dev(x)).cpu().numpy()
    b = plain.run(_dev(x)).cpu().numpy()
    cp.cprune_poll_device_status()
    assert np.linalg.norm(a - b) <= 3e-3 * np.linalg.norm(b)
    pw, _ = oracle.prune_model(table, weights)
    ref = oracle.model_ref(table, pw, x, matched=True)
    assert np.linalg.norm(a - ref) <= 1e-2 * np.linalg.norm(ref)
    print("\nfused blocks: %s; launches %d -> %d" % (sorted(fused.blocks), plain.model.launches, fused.model.launches))


def test_shared_selection_and_shortcut_pruned_resnet(cp):
    # dependency-aware pruning: one ranking for the layers whose outputs meet in a residual add
    ws = [wl.normal_f32(51, 1, (96, 20, 3, 3), 0.1), wl.normal_f32(51, 2, (96, 64, 1, 1), 0.1), wl.normal_f32(51, 3, (96, 7, 3, 3), 0.1)]
    ws[0][5] = ws[0][4]
    ws[1][5] = ws[1][4]
    ws[2][5] = -ws[2][4]                   # filters 4 and 5 tie exactly across the group: the lower index wins
    for keep in (1, 5, 48, 95, 96):
        kept = cp.cprune_select_shared([_dev(w) for w in ws], keep)
        assert np.array_equal(kept.cpu().numpy(), oracle.select_indices_shared(ws, keep)), keep
    cp.cprune_poll_device_status()
    one = cp.cprune_select_shared([_dev(ws[0])], 40)
    assert np.array_equal(one.cpu().numpy(), oracle.select_indices(ws[0], 40))
    net, _, _ = model_parity(cp, "resnet18_shared", 2, hw=64)
    assert net.plans["l2b1_conv2"].K == 96 and net.plans["l2b2_conv1"].C == 96 and net.plans["stem"].K == 48


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

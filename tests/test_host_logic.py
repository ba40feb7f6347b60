"""CPU-only checks of the library boundary: it loads, exports what the header declares, and its
host-side logic (argument validation, plans, plan cache) behaves without a device."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cp():
    from paper_2207_01260_b200 import build
    build.build()
    import paper_2207_01260_b200 as m
    m.lib()
    return m


def test_library_exports_every_declared_symbol(cp):
    header = open(os.path.join(ROOT, "include", "cprune.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cprune_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 25
    assert declared == set(cp.EXPORTS)
    L = cp.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings_and_padding(cp):
    L = cp.lib()
    assert L.cprune_status_string(0) == b"ok"
    assert len({L.cprune_status_string(i) for i in range(8)}) == 8
    assert [cp.cprune_padded_channels(c) for c in (1, 3, 8, 9, 44, 45, 72, 128, 129, 243, 358)] == [8, 8, 8, 16, 48, 48, 72, 128, 144, 256, 368]
    assert cp.cprune_select_workspace_bytes(0) == 0 and cp.cprune_select_workspace_bytes(1280) >= 1280 * 12


def test_plan_shapes_and_families(cp):
    p = cp.cprune_task_plan(64, 64, 56, 56, 44, 3, 3, 1, 1)
    assert (p.P, p.Q, p.c_pad, p.k_pad) == (56, 56, 64, 48)
    # stride-1 3x3 with many tiles: patch kernel, a tile is 4 whole output rows (2 x 128 accumulator rows, 58 per
    # image row with the two wrap-around columns), all 48 padded filters in one MMA
    assert cp.KERNEL_NAMES[p.kernel] == "tensor" and p.tile_m == 256 and p.tile_n == 48
    assert p.tiles_m == 64 * 14 and p.tiles_n == 1 and p.k_alloc == 48 and p.workspace_bytes == 0
    q = cp.cprune_task_plan(64, 256, 14, 14, 358, 3, 3, 1, 1)
    assert q.tile_m in (128, 256) and q.tile_n % 16 == 0 and q.tiles_n * q.tile_n >= 358 and q.k_alloc == q.tiles_n * q.tile_n
    # 1x1 and stride-2 tasks stay on the im2col kernel: K <= 128 puts the filters on the 128-row side, 256 pixels a tile
    r = cp.cprune_task_plan(64, 64, 56, 56, 128, 1, 1, 2, 0)
    assert cp.KERNEL_NAMES[r.kernel] == "tensor" and r.tile_m == 256 and r.tile_n == 128 and r.k_alloc == 128
    # a stem with enough tiles runs on the patch kernel and asks for room for the regrouped input
    s = cp.cprune_task_plan(64, 3, 224, 224, 64, 7, 7, 2, 3)
    assert cp.KERNEL_NAMES[s.kernel] == "tensor" and s.workspace_bytes >= 64 * 112 * 115 * 32
    assert p.flops == 2.0 * 64 * 44 * 64 * 56 * 56 * 9
    assert p.padded_flops >= p.flops
    p = cp.cprune_task_plan(1, 3, 224, 224, 64, 7, 7, 2, 3)
    assert (p.P, p.Q) == (112, 112) and cp.KERNEL_NAMES[p.kernel] == "tensor"
    p = cp.cprune_task_plan(1, 3, 224, 224, 64, 7, 7, 2, 3, kernel="direct")
    assert cp.KERNEL_NAMES[p.kernel] == "direct"
    p = cp.cprune_task_plan(8, 108, 56, 56, 108, 3, 3, 2, 1, groups=108, activation="relu6")
    assert cp.KERNEL_NAMES[p.kernel] == "depthwise" and (p.P, p.Q) == (28, 28) and p.c_pad == 112
    assert p.flops == 2.0 * 8 * 108 * 28 * 28 * 9
    p = cp.cprune_task_plan(128, 45, 32, 32, 58, 3, 3, 1, 1, pool="max2x2")
    # the pool runs inside the conv kernel: the output is the pooled tensor and no unpooled copy is kept
    assert (p.out_h, p.out_w) == (16, 16) and p.workspace_bytes == 0
    # the CUDA-core family does not fuse it: the unpooled output goes to the workspace
    p = cp.cprune_task_plan(128, 45, 32, 32, 58, 3, 3, 1, 1, pool="max2x2", kernel="direct")
    assert (p.out_h, p.out_w) == (16, 16) and p.workspace_bytes == 128 * 32 * 32 * 64 * 2
    # a pointwise stride-1 task with many pixels is planned as a flat matrix product: tiles of 128 or 256 pixels
    f = cp.cprune_task_plan(64, 24, 56, 56, 108, 1, 1, 1, 0, activation="relu6")
    assert f.variant == 1 and f.tile_m in (128, 256) and f.tiles_m == -(-64 * 56 * 56 // f.tile_m) and f.workspace_bytes == 0
    # one filter tile: the tile is staged pixel by pixel as it lies in memory (variant 2; the staged pixels are made an odd
    # number of 16-byte pieces long); a tile too large to stage that way, or several filter tiles, keep the tiled stores
    for K, want in ((72, 2), (24, 2), (16, 2), (40, 2), (32, 2), (64, 2), (108, 1), (300, 1)):
        d = cp.cprune_task_plan(64, 48, 56, 56, K, 1, 1, 1, 0, activation="relu6")
        assert d.variant == want, (K, d.variant)
    # the ResNet stem with its 3x3 stride-2 pool: pooled output extent, pool fused (no unpooled copy in the workspace,
    # only the regrouped input), tiles around whole pooling windows
    sp = cp.cprune_task_plan(64, 3, 224, 224, 64, 7, 7, 2, 3, pool="max3x3s2")
    assert (sp.P, sp.Q, sp.out_h, sp.out_w) == (112, 112, 56, 56) and sp.variant == 1
    assert sp.workspace_bytes == s.workspace_bytes
    # the same pool on a task the patch kernel cannot fuse it into runs as a separate pass over an unpooled copy
    sq = cp.cprune_task_plan(2, 16, 30, 30, 24, 3, 3, 1, 1, pool="max3x3s2")
    assert (sq.out_h, sq.out_w) == (15, 15) and sq.workspace_bytes >= 2 * 30 * 30 * 24 * 2
    # every pruned filter count gets a legal tile: N tile a multiple of 16 within the accumulator
    for K in range(64, 513, 7):
        p = cp.cprune_task_plan(64, 256, 14, 14, K, 3, 3, 1, 1)
        assert p.tile_n % 16 == 0 and 16 <= p.tile_n <= 256 and p.k_alloc >= p.k_pad >= K
        assert 2 <= p.stages <= 8


def test_plan_cache(cp):
    cp.cprune_cache_clear()
    n0, h0 = cp.cprune_cache_stats()
    a = cp.cprune_task_plan(2, 89, 28, 28, 128, 3, 3, 1, 1)
    b = cp.cprune_task_plan(2, 89, 28, 28, 128, 3, 3, 1, 1)
    c = cp.cprune_task_plan(2, 89, 28, 28, 128, 3, 3, 1, 1, activation="none")
    assert a.handle.value == b.handle.value != c.handle.value
    n1, h1 = cp.cprune_cache_stats()
    assert n1 - n0 == 2 and h1 - h0 == 1
    ha = a.handle.value
    del a, b, c
    import gc
    gc.collect()
    cp.cprune_cache_clear()
    assert cp.cprune_cache_stats()[0] == n0
    d = cp.cprune_task_plan(2, 89, 28, 28, 128, 3, 3, 1, 1)
    assert d.info["tile_n"] > 0 and ha is not None


def test_plan_argument_errors(cp):
    for args in [(0, 8, 8, 8, 8, 3, 3, 1, 1), (1, 8, 8, 8, 0, 3, 3, 1, 1), (1, 8, 2, 2, 8, 7, 7, 1, 0),
                 (1, 8, 8, 8, 8, 3, 3, 0, 1)]:
        with pytest.raises(cp.CpruneError) as e:
            cp.cprune_task_plan(*args)
        assert e.value.status == 1
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_task_plan(1, 8, 8, 8, 8, 7, 7, 1, 3, groups=8)      # depthwise is 3x3 or 5x5
    assert e.value.status == 2
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_task_plan(1, 8, 7, 7, 8, 3, 3, 1, 1, pool="max2x2")  # odd extent cannot be pooled 2x2
    assert e.value.status == 1


def test_missing_library_fails_loudly(cp, monkeypatch):
    from paper_2207_01260_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libcprune.so")
    with pytest.raises(RuntimeError):
        binding.lib()


# ------------------------------------------------------------------ pruning decision, task ordering

def test_prune_step_follows_the_lcm_rule_on_the_plans_own_splits(cp):
    import oracle
    cases = [(64, 64, 56, 56, 44, 3, 1, 1, 1), (64, 128, 28, 28, 89, 3, 1, 1, 1), (64, 256, 14, 14, 358, 3, 1, 1, 1),
             (64, 512, 7, 7, 358, 3, 1, 1, 1), (64, 64, 56, 56, 128, 1, 2, 0, 1), (64, 320, 7, 7, 1280, 1, 1, 0, 1),
             (64, 144, 56, 56, 144, 3, 1, 1, 144), (64, 720, 7, 7, 720, 3, 1, 1, 720), (1, 16, 8, 8, 24, 3, 1, 1, 1)]
    for N, C, H, W, K, R, stride, pad, groups in cases:
        p = cp.cprune_task_plan(N, C, H, W, K, R, R, stride, pad, groups)
        want = oracle.prune_step_lcm(p.split_compute, p.split_store, p.unit_compute, p.unit_store)
        got = cp.cprune_prune_step(p)
        assert got == want and 1 <= got <= p.k_alloc, (N, C, K, got, want)
        # the splits describe the plan's own tiling of the filter axis
        prod_c = p.split_compute[0] * p.split_compute[1] * p.unit_compute
        prod_s = p.split_store[0] * p.split_store[1] * p.unit_store
        assert prod_c >= p.k_pad and prod_s >= p.k_pad, (N, C, K, prod_c, prod_s)
    # one filter tile of 48 = 3 groups of 16 and 6 pieces of 8: smallest slices 16 and 8, lcm 16
    p = cp.cprune_task_plan(64, 64, 56, 56, 44, 3, 3, 1, 1)
    assert (p.split_compute, p.unit_compute, p.split_store, p.unit_store) == ([1, 3], 16, [1, 6], 8)
    assert cp.cprune_prune_step(p) == 16


def test_task_estimate_is_a_staircase_in_the_filter_count(cp):
    p = cp.cprune_task_plan(64, 128, 28, 28, 128, 3, 3, 1, 1)
    est = [cp.cprune_task_estimate(p, k) for k in range(128, 31, -1)]
    assert est[0] == pytest.approx(p.est_us) and all(e > 0 for e in est)
    assert all(a >= b - 1e-9 for a, b in zip(est, est[1:])), "fewer filters never cost more in the model"
    levels = sorted(set(round(e, 6) for e in est))
    assert 3 <= len(levels) <= 16, levels           # flat stretches with steps in between, not a ramp
    with pytest.raises(cp.CpruneError) as e:
        cp.cprune_task_estimate(p, 0)
    assert e.value.status == 1
    d = cp.cprune_task_plan(64, 144, 56, 56, 144, 3, 3, 1, 1, groups=144)
    assert cp.cprune_task_estimate(d, 72) < cp.cprune_task_estimate(d, 144)


def test_task_order_matches_the_paper_and_the_oracle(cp):
    import oracle
    assert cp.cprune_task_order([0.954, 0.473, 1.632], [2, 3, 1]) == [0, 2, 1]        # T1, T3, T2 (paper Sec. 3.3)
    assert cp.cprune_task_order([], []) == []
    import workloads as wl
    t = list(wl.normal(77, 1, 40) ** 2)
    c = [1 + (i * 7) % 4 for i in range(40)]
    t[5], c[5], t[9], c[9] = 2.0, 3, 3.0, 2                                           # an exact tie: lower index first
    assert cp.cprune_task_order(t, c) == oracle.task_order(t, c)


def test_no_swept_shape_leaves_the_tensor_cores(cp):
    # every dense shape of the sweep, at every kept filter count from full width to a quarter and at both batch
    # sizes, gets a tensor-core plan; every depthwise shape a depthwise plan
    import workloads as wl
    for N in (1, 64):
        for shp in wl.sweep_shapes():
            dw = shp["groups"] > 1
            for K in range(shp["K"], (shp["K"] + 3) // 4 - 1, -1):
                p = cp.cprune_task_plan(N, K if dw else shp["C"], shp["H"], shp["W"], K, shp["R"], shp["S"], shp["stride"],
                                        shp["pad"], K if dw else 1, shp["act"])
                assert cp.KERNEL_NAMES[p.kernel] == ("depthwise" if dw else "tensor"), (N, shp, K)
        cp.cprune_cache_clear()


def test_plan_flags_are_part_of_the_cache_key(cp):
    a = cp.cprune_task_plan(16, 64, 32, 32, 48, 3, 3, 1, 1)
    b = cp.cprune_task_plan(16, 64, 32, 32, 48, 3, 3, 1, 1, flags=("im2col_only",))
    assert a.handle.value != b.handle.value and a.variant == 1 and b.variant == 0
    with pytest.raises(cp.CpruneError) as e:
        L = cp.lib()
        from paper_2207_01260_b200.binding import TaskOpts
        import ctypes
        h = ctypes.c_void_p()
        st = L.cprune_task_plan(1, 8, 8, 8, 8, 3, 3, 1, 1, 1, ctypes.byref(TaskOpts(1, 0, 0, 0, 64)), ctypes.byref(h))
        raise cp.CpruneError(st, "cprune_task_plan")
    assert e.value.status == 1

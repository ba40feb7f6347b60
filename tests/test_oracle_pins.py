"""Pins for the CPU oracle: it is checked against things other than itself -- hand-computed
values, closed forms, invariants, library routines, and the totals the paper prints."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(seed, shape, std=1.0):
    return wl.normal_f32(seed, 7, shape, std).astype(np.float64)


# ------------------------------------------------------------------ convolution

def test_conv_hand_computed_3x3_pad1():
    # x is one 2x2 image with one channel, w one 3x3 filter; worked out by hand:
    #   x = [[1, 2], [3, 4]],  w = [[1,2,3],[4,5,6],[7,8,9]], pad 1, stride 1.
    # y[0,0] = 5*1 + 6*2 + 8*3 + 9*4 = 77 ; y[0,1] = 4*1 + 5*2 + 7*3 + 8*4 = 67
    # y[1,0] = 2*1 + 3*2 + 5*3 + 6*4 = 47 ; y[1,1] = 1*1 + 2*2 + 4*3 + 5*4 = 37
    x = np.array([[1.0, 2.0], [3.0, 4.0]]).reshape(1, 2, 2, 1)
    w = np.arange(1.0, 10.0).reshape(1, 1, 3, 3)
    y = oracle.conv2d(x, w, None, 1, 1)
    assert y.reshape(2, 2).tolist() == [[77.0, 67.0], [47.0, 37.0]]
    # with bias -50 and ReLU, then ReLU6
    y = oracle.conv2d(x, w, np.array([-50.0]), 1, 1, act="relu")
    assert y.reshape(2, 2).tolist() == [[27.0, 17.0], [0.0, 0.0]]
    y = oracle.conv2d(x, w, np.array([-50.0]), 1, 1, act="relu6")
    assert y.reshape(2, 2).tolist() == [[6.0, 6.0], [0.0, 0.0]]


def test_conv_hand_computed_two_channels_two_filters():
    # 1x1 spatial, C=2, K=2, 1x1 kernel: a 2x2 matrix-vector product.
    x = np.array([3.0, -2.0]).reshape(1, 1, 1, 2)
    w = np.array([[1.0, 10.0], [100.0, 1000.0]]).reshape(2, 2, 1, 1)   # w[k, c]
    y, bound = oracle.conv2d(x, w, np.array([0.5, -0.5]), with_bound=True)
    assert y.ravel().tolist() == [3.0 - 20.0 + 0.5, 300.0 - 2000.0 - 0.5]
    assert bound.ravel().tolist() == [3.0 + 20.0 + 0.5, 300.0 + 2000.0 + 0.5]


def test_conv_residual_is_added_before_activation():
    x = np.array([1.0]).reshape(1, 1, 1, 1)
    w = np.array([2.0]).reshape(1, 1, 1, 1)
    res = np.array([-5.0]).reshape(1, 1, 1, 1)
    assert oracle.conv2d(x, w, np.array([1.0]), act="relu", res=res).item() == 0.0      # relu(2+1-5)
    assert oracle.conv2d(x, w, np.array([1.0]), act="none", res=res).item() == -2.0
    y, bnd = oracle.conv2d(x, w, np.array([1.0]), act="none", res=res, with_bound=True)
    assert bnd.item() == 2.0 + 1.0 + 5.0


def test_conv_identity_1x1_reproduces_input():
    x = _rand(1, (2, 5, 7, 6))
    w = np.eye(6).reshape(6, 6, 1, 1)
    assert np.array_equal(oracle.conv2d(x, w), x)


@pytest.mark.parametrize("r,s", [(0, 0), (0, 2), (1, 1), (2, 0), (2, 2), (1, 0)])
def test_conv_single_tap_is_a_shift(r, s):
    # a 3x3 filter holding a single 1 at tap (r, s): y[p, q] = x[p - 1 + r, q - 1 + s], 0 outside.
    x = _rand(2, (1, 6, 5, 1))
    w = np.zeros((1, 1, 3, 3))
    w[0, 0, r, s] = 1.0
    y = oracle.conv2d(x, w, None, 1, 1)
    exp = np.zeros_like(x)
    for p in range(6):
        for q in range(5):
            h, v = p - 1 + r, q - 1 + s
            if 0 <= h < 6 and 0 <= v < 5:
                exp[0, p, q, 0] = x[0, h, v, 0]
    assert np.array_equal(y, exp)


def test_conv_linearity_in_weights():
    x = _rand(3, (2, 9, 8, 5))
    w1, w2 = _rand(4, (7, 5, 3, 3)), _rand(5, (7, 5, 3, 3))
    a, b = 0.75, -1.5
    lhs = oracle.conv2d(x, a * w1 + b * w2, None, 2, 1)
    rhs = a * oracle.conv2d(x, w1, None, 2, 1) + b * oracle.conv2d(x, w2, None, 2, 1)
    assert np.max(np.abs(lhs - rhs)) <= 1e-12 * np.max(np.abs(lhs))


@pytest.mark.parametrize("R,pad,stride", [(3, 1, 1), (3, 1, 2), (7, 3, 2), (1, 0, 1), (3, 0, 1)])
def test_conv_all_ones_counts_in_bounds_taps(R, pad, stride):
    H, W, C, K = 9, 10, 4, 3
    y = oracle.conv2d(np.ones((1, H, W, C)), np.ones((K, C, R, R)), None, stride, pad)
    P, Q = y.shape[1:3]
    assert P == (H + 2 * pad - R) // stride + 1 and Q == (W + 2 * pad - R) // stride + 1
    for p in range(P):
        nh = sum(1 for r in range(R) if 0 <= p * stride - pad + r < H)
        for q in range(Q):
            nw = sum(1 for s in range(R) if 0 <= q * stride - pad + s < W)
            assert np.all(y[0, p, q] == nh * nw * C)


def test_depthwise_centre_delta_is_identity():
    x = _rand(6, (2, 6, 6, 5))
    w = np.zeros((5, 1, 3, 3))
    w[:, 0, 1, 1] = 1.0
    assert np.array_equal(oracle.conv2d(x, w, None, 1, 1, groups=5), x)


def test_stride2_equals_subsampled_stride1():
    x = _rand(7, (1, 11, 9, 3))
    w = _rand(8, (4, 3, 3, 3))
    y1 = oracle.conv2d(x, w, None, 1, 1)
    y2 = oracle.conv2d(x, w, None, 2, 1)
    assert np.array_equal(y2, y1[:, ::2, ::2])


@pytest.mark.parametrize("N,H,W,C,K,R,stride,pad,groups", [
    (2, 8, 9, 6, 5, 3, 1, 1, 1), (1, 13, 12, 3, 7, 7, 2, 3, 1), (2, 7, 7, 8, 8, 3, 2, 1, 8),
    (1, 6, 5, 4, 6, 1, 2, 0, 1), (1, 10, 10, 6, 4, 3, 1, 0, 2), (3, 4, 4, 5, 9, 3, 1, 1, 1)])
def test_conv_against_library_routine(N, H, W, C, K, R, stride, pad, groups):
    # torch's float64 CPU convolution is an independent implementation of the same definition
    x = _rand(9, (N, H, W, C))
    w = _rand(10, (K, C // groups, R, R))
    b = _rand(11, (K,))
    y = oracle.conv2d(x, w, b, stride, pad, groups)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(w),
                                     torch.from_numpy(b), stride, pad, 1, groups).permute(0, 2, 3, 1).numpy()
    assert y.shape == ref.shape
    assert np.max(np.abs(y - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_bound_is_conv_of_absolute_values():
    x, w, b = _rand(12, (1, 6, 6, 4)), _rand(13, (3, 4, 3, 3)), _rand(14, (3,))
    _, bound = oracle.conv2d(x, w, b, 1, 1, with_bound=True)
    ref = torch.nn.functional.conv2d(torch.from_numpy(np.abs(x)).permute(0, 3, 1, 2), torch.from_numpy(np.abs(w)),
                                     torch.from_numpy(np.abs(b)), 1, 1).permute(0, 2, 3, 1).numpy()
    assert np.allclose(bound, ref, rtol=1e-13, atol=0)


def test_points_equal_full_conv():
    x, w, b = _rand(15, (2, 7, 6, 4)), _rand(16, (5, 4, 3, 3)), _rand(17, (5,))
    res = _rand(18, (2, 4, 3, 5))
    y, bd = oracle.conv2d(x, w, b, 2, 1, 1, "relu", res, with_bound=True)
    pts = np.array([[n, p, q, k] for n in range(2) for p in range(4) for q in range(3) for k in range(5)], dtype=np.int32)
    v, a = oracle.conv2d_points(x, w, b, 2, 1, 1, "relu", res, pts)
    assert np.array_equal(v, y.ravel()) and np.array_equal(a, bd.ravel())


def test_flop_closed_form_and_paper_totals():
    assert oracle.conv_flops(2, 3, 5, 7, 11, 3, 3, 1) == 2 * 2 * 3 * 5 * 7 * 11 * 9
    assert oracle.conv_flops(1, 8, 8, 4, 4, 3, 3, 8) == 2 * 8 * 4 * 4 * 9
    # count the multiply-adds of the plain definition by brute force on a small case (pad 0 so that
    # every tap is in bounds): sum |x||w| with all-ones data counts the taps
    _, bound = oracle.conv2d(np.ones((2, 6, 7, 4)), np.ones((3, 4, 3, 3)), None, 1, 0, with_bound=True)
    assert 2 * int(bound.sum()) == oracle.conv_flops(2, 4, 3, 4, 5, 3, 3)
    totals = {}
    for line in open(os.path.join(GOLDEN, "paper_model_totals.txt")):
        if line.strip() and not line.startswith("#"):
            name, macs, params = line.split()
            totals[name] = (float(macs), float(params))
    for name, fn in (("resnet18", wl.resnet18), ("mobilenet_v2", wl.mobilenet_v2), ("mnasnet1_0", wl.mnasnet1_0)):
        got = oracle.model_counts(fn(None))
        assert abs(got["macs"] - totals[name][0]) <= 0.006 * totals[name][0], (name, got)
        assert abs(got["params"] - totals[name][1]) <= 0.01 * totals[name][1], (name, got)


# ------------------------------------------------------------------ pools, fc, rounding

def test_maxpool_hand_cases_and_padding_never_wins():
    x = np.array([[-1.0, -2.0, -3.0], [-4.0, -5.0, -6.0], [-7.0, -8.0, -9.0]]).reshape(1, 3, 3, 1)
    y = oracle.maxpool(x, 3, 2, 1)          # windows centred on (0,0), (0,2), (2,0), (2,2)
    assert y.reshape(2, 2).tolist() == [[-1.0, -2.0], [-4.0, -5.0]]
    y = oracle.maxpool(x[:, :2, :2], 2, 2, 0)
    assert y.item() == -1.0
    z = _rand(20, (2, 8, 6, 3))
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(z).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(oracle.maxpool(z, 3, 2, 1), ref)


def test_gap_and_fc_against_numpy():
    x = _rand(21, (3, 4, 5, 6))
    assert np.allclose(oracle.gap(x), x.mean(axis=(1, 2)), rtol=1e-14)
    a, w, b = _rand(22, (3, 10)), _rand(23, (4, 10)), _rand(24, (4,))
    y, bound = oracle.fc(a, w, b, "relu", with_bound=True)
    assert np.allclose(y, np.maximum(a @ w.T + b, 0), rtol=1e-13, atol=1e-15)
    assert np.allclose(bound, np.abs(a) @ np.abs(w).T + np.abs(b), rtol=1e-13)
    assert oracle.fc(np.array([[1.0, 2.0]]), np.array([[3.0, 4.0], [5.0, 6.0]]), np.array([0.5, 0.0])).tolist() == [[11.5, 17.0]]


def test_round_bf16_ties_and_library():
    one = 1.0
    ulp = 2.0 ** -7
    cases = {one + ulp / 2: one,                 # tie -> even mantissa (1.0)
             one + 3 * ulp / 2: one + 2 * ulp,   # tie -> even
             one + ulp / 2 + 1e-9: one + ulp, one + ulp / 2 - 1e-9: one,
             -(one + 3 * ulp / 2): -(one + 2 * ulp), 0.0: 0.0, 255.5: 256.0, 3.0e-5: None}
    xs = np.array(list(cases))
    got = oracle.round_bf16(xs)
    for v, e, g in zip(xs, cases.values(), got):
        if e is not None:
            assert g == e, (v, g, e)
    z = wl.normal_f32(3, 3, (20000,)).astype(np.float64) * np.exp(wl.normal(3, 4, 20000) * 4)
    z32 = z.astype(np.float32)
    ref = torch.from_numpy(z32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_bf16(z32.astype(np.float64)), ref)


# ------------------------------------------------------------------ selection

def test_l1_norm_hand_values_and_grid():
    w = np.array([[0.5, -0.25, 1.0], [2.0 ** -40, -(2.0 ** -41), 3 * 2.0 ** -41]], dtype=np.float32).reshape(2, 3, 1, 1)
    n = oracle.l1_norms(w)
    assert n[0] == int(1.75 * 2 ** 40)
    assert n[1] == 1 + 0 + 2            # 2^-41 is a tie -> even (0); 3*2^-41 = 1.5 -> 2
    w = wl.normal_f32(5, 1, (8, 16, 3, 3), 0.05)
    exact = oracle.l1_norms_exact(w)
    grid = oracle.l1_norms(w)
    for g, e in zip(grid, exact):
        assert abs(g / 2.0 ** 40 - e) <= 144 * 2.0 ** -41


def test_select_hand_made_and_ties():
    # norms 4, 1, 4, 3, 1 -> keep 3: the two 4s and the 3; keep 2: filters 0 and 2 ; keep 4: tie of 1s -> lower index
    w = np.array([[4, 0], [1, 0], [-2, -2], [0, 3], [-0.5, 0.5]], dtype=np.float32).reshape(5, 2, 1, 1)
    assert oracle.select_indices(w, 3).tolist() == [0, 2, 3]
    assert oracle.select_indices(w, 2).tolist() == [0, 2]
    assert oracle.select_indices(w, 1).tolist() == [0]             # tie between 0 and 2 -> lower index
    assert oracle.select_indices(w, 4).tolist() == [0, 1, 2, 3]    # tie between 1 and 4 -> lower index
    assert oracle.select_indices(w, 5).tolist() == [0, 1, 2, 3, 4]


def test_select_against_sorted_and_invariances():
    w = wl.normal_f32(6, 1, (37, 5, 3, 3), 0.1)
    w[11] = w[3]                 # duplicate filter
    w[20] = -w[3]                # sign-flipped duplicate
    exact = oracle.l1_norms_exact(w)
    prev = set()
    for keep in range(1, 38):
        got = oracle.select_indices(w, keep)
        order = sorted(range(37), key=lambda k: (-exact[k], k))
        assert got.tolist() == sorted(order[:keep])
        assert prev <= set(got.tolist())          # nesting
        prev = set(got.tolist())
    perm = np.random.RandomState(0).permutation(45)
    wp = w.reshape(37, 45)[:, perm].reshape(w.shape)
    assert np.array_equal(oracle.l1_norms(wp), oracle.l1_norms(w))
    for j in (-3, 2):
        assert np.array_equal(oracle.select_indices(w * np.float32(2.0 ** j), 17), oracle.select_indices(w, 17))
    kept, wo, bo, wn = oracle.select_filters(w, np.arange(37, dtype=np.float32), 37, wl.normal_f32(6, 2, (4, 37, 1, 1)))
    assert kept.tolist() == list(range(37)) and wo.tobytes() == w.tobytes()


def test_slicing_channel_subset_property():
    x = _rand(30, (1, 6, 6, 5))
    w1 = wl.normal_f32(30, 1, (9, 5, 3, 3), 0.2)
    b1 = wl.normal_f32(30, 2, (9,), 0.01)
    w2 = wl.normal_f32(30, 3, (4, 9, 3, 3), 0.2)
    kept, w1p, b1p, w2p = oracle.select_filters(w1, b1, 6, w2)
    full = oracle.conv2d(x, w1, b1, 1, 1, act="relu")
    pruned = oracle.conv2d(x, w1p, b1p, 1, 1, act="relu")
    assert np.array_equal(full[..., kept], pruned)                      # bit for bit
    w2z = w2.copy()
    drop = np.setdiff1d(np.arange(9), kept)
    w2z[:, drop] = 0
    a = oracle.conv2d(pruned, w2p, None, 1, 1)
    b = oracle.conv2d(full, w2z, None, 1, 1)
    assert np.max(np.abs(a - b)) <= 1e-13 * np.max(np.abs(b))
    # depthwise consumer: whole filters follow
    wd = wl.normal_f32(30, 4, (9, 1, 3, 3), 0.2)
    _, _, _, wdp = oracle.select_filters(w1, b1, 6, wd, next_is_depthwise=True)
    assert np.array_equal(wdp, wd[kept])


# ------------------------------------------------------------------ models

def _tiny(model, hw):
    m = dict(model)
    m["input"] = (hw, hw, model["input"][2])
    return m


def test_layer_tables_match_the_pruned_widths():
    m = wl.pruned_shapes(wl.resnet18())
    by = wl.layer_by_name(m)
    assert [by["l%db1_conv1" % s]["K"] for s in (1, 2, 3, 4)] == [44, 89, 179, 358]
    assert by["l3b2_conv2"]["C"] == 179 and by["l3b2_conv2"]["K"] == 256
    m = wl.pruned_shapes(wl.mobilenet_v2())
    by = wl.layer_by_name(m)
    dws = [l["C"] for l in m["layers"] if l["kind"] == "conv" and l["groups"] > 1]
    assert dws == [32, 72, 108, 108, 144, 144, 144, 288, 288, 288, 288, 432, 432, 432, 720, 720, 720]
    assert by["b2_proj"]["C"] == 72 and by["b2_dw"]["groups"] == 72
    m = wl.pruned_shapes(wl.vgg16_cifar())
    by = wl.layer_by_name(m)
    assert [by["c%d" % i]["K"] for i in range(1, 14)] == wl.VGG16_KEEP
    assert by["c5"]["C"] == 96 and by["fc1"]["in_features"] == 243
    assert len(wl.sweep_shapes()) >= 40


@pytest.mark.parametrize("name,hw", [("vgg16_cifar", 32), ("resnet18", 32), ("mobilenet_v2", 32), ("mnasnet1_0", 32),
                                     ("resnet18_shared", 32)])
def test_keep_all_pruning_equals_unpruned_model(name, hw):
    model = _tiny(wl.MODELS[name](), hw)
    weights = wl.model_weights(model)
    keepall = _tiny(wl.MODELS[name](), hw)
    for l in keepall["layers"]:
        if l["kind"] == "conv" and l["keep"] is not None:
            l["keep"] = l["K"]
    pw, kept = oracle.prune_model(keepall, weights)
    for k, (w, b) in weights.items():
        assert pw[k][0].tobytes() == w.tobytes() and pw[k][1].tobytes() == b.tobytes()
    x = wl.model_input(model, 1)
    a = oracle.model_ref(model, weights, x)
    b = oracle.model_ref(keepall, pw, x)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("name,hw", [("vgg16_cifar", 32), ("resnet18", 32), ("mobilenet_v2", 32), ("mnasnet1_0", 32),
                                     ("resnet18_shared", 32)])
def test_pruned_model_equals_unpruned_with_dropped_filters_zeroed(name, hw):
    model = _tiny(wl.MODELS[name](), hw)
    weights = wl.model_weights(model)
    pw, kept = oracle.prune_model(model, weights)
    shapes = wl.layer_by_name(wl.pruned_shapes(model))
    for lname, (w, b) in pw.items():
        l = shapes[lname]
        if l["kind"] == "conv":
            assert w.shape == (l["K"], l["C"] // l["groups"], l["R"], l["S"]) and b.shape == (l["K"],)
        else:
            assert w.shape == (l["out_features"], l["in_features"])
    # zero the dropped filters (weights and bias) in the full model: same logits
    zeroed = {k: (w.copy(), b.copy()) for k, (w, b) in weights.items()}
    full = wl.layer_by_name(model)
    for lname, idx in kept.items():
        w, b = zeroed[lname]
        drop = np.setdiff1d(np.arange(w.shape[0]), idx)
        w[drop] = 0
        b[drop] = 0
        for cname, how in full[lname]["consumers"]:
            if how == "depthwise":      # a removed channel takes its depthwise filter and bias with it
                zeroed[cname][0][drop] = 0
                zeroed[cname][1][drop] = 0
    x = wl.model_input(model, 2)
    a = oracle.model_ref(model, pw, x)
    b = oracle.model_ref(model, zeroed, x)
    assert a.shape == b.shape
    assert np.max(np.abs(a - b)) <= 1e-11 * np.max(np.abs(b))
    # matched (bfloat16-stored) mode stays close to the exact mode
    c = oracle.model_ref(model, pw, x, matched=True)
    assert np.linalg.norm(c - a) <= 5e-2 * np.linalg.norm(a)


def test_generator_is_counter_based_and_normal():
    a = wl.normal(5, 3, 1000)
    b = wl.normal(5, 3, 5000)
    assert np.array_equal(a, b[:1000])
    assert not np.array_equal(wl.normal(5, 4, 1000), a)
    z = wl.normal(9, 0, 400000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01 and abs(np.mean(z ** 4) - 3) < 0.1


# ------------------------------------------------------------------ shared (dependency-aware) selection

def test_shared_selection_hand_made():
    # two member layers, four channels.  Per-channel norms: layer A = 1, 5, 2, 4; layer B = 6, 1, 2, 2.
    # Summed: 7, 6, 4, 6 -> keep 2: channels 0 and 1 (the tie between 1 and 3 keeps the lower index);
    # keep 3: 0, 1, 3.  Ranking either layer alone would choose differently (A alone: 1 and 3).
    a = np.zeros((4, 1, 1, 1), dtype=np.float32)
    b = np.zeros((4, 2, 1, 1), dtype=np.float32)
    a[:, 0, 0, 0] = [1, -5, 2, 4]
    b[:, 0, 0, 0] = [6, 0.5, -2, 1]
    b[:, 1, 0, 0] = [0, -0.5, 0, 1]
    assert oracle.select_indices_shared([a, b], 2).tolist() == [0, 1]
    assert oracle.select_indices_shared([a, b], 3).tolist() == [0, 1, 3]
    assert oracle.select_indices(a, 2).tolist() == [1, 3]
    # one member: the plain selection; member order does not matter
    w = wl.normal_f32(41, 1, (23, 5, 3, 3), 0.1)
    v = wl.normal_f32(41, 2, (23, 7, 1, 1), 0.1)
    for keep in (1, 9, 23):
        assert np.array_equal(oracle.select_indices_shared([w], keep), oracle.select_indices(w, keep))
        assert np.array_equal(oracle.select_indices_shared([w, v], keep), oracle.select_indices_shared([v, w], keep))
    # the group norm is the norm of the members' filters laid side by side
    both = np.concatenate([w.reshape(23, -1), v.reshape(23, -1)], axis=1).reshape(23, -1, 1, 1)
    assert np.array_equal(oracle.select_indices_shared([w, v], 11), oracle.select_indices(both, 11))


def test_shared_groups_of_the_resnet_table_keep_the_same_filters():
    model = _tiny(wl.resnet18_shared(), 32)
    weights = wl.model_weights(model)
    pw, kept = oracle.prune_model(model, weights)
    for stage, members in ((1, ["stem", "l1b1_conv2", "l1b2_conv2"]), (3, ["l3b1_down", "l3b1_conv2", "l3b2_conv2"])):
        ref = oracle.select_indices_shared([weights[m][0] for m in members], (3 * [64, 128, 256, 512][stage - 1]) // 4)
        for m in members:
            assert np.array_equal(kept[m], ref), m
    assert pw["fc"][0].shape == (1000, 384) and pw["l2b1_down"][0].shape == (96, 48, 1, 1)


# ------------------------------------------------------------------ pruning decision, task ordering, task table

def _paper_examples():
    ex = {}
    for line in open(os.path.join(GOLDEN, "paper_worked_examples.txt")):
        if line.strip() and not line.startswith("#"):
            key, val = line.split(":", 1)
            ex[key.strip()] = val.strip()
    return ex


def test_prune_step_matches_the_papers_worked_examples():
    ex = _paper_examples()
    for key in ("lcm_fast_program", "lcm_slow_program"):
        l1, l2, want = ex[key].split("|")
        L1 = [int(v) for v in l1.split("x")]
        L2 = [int(v) for v in l2.split("x")]
        assert oracle.prune_step_lcm(L1, L2) == int(want), key
    # the smallest slice of 4 x 8 x 16 filters is 512 / 16; of 3 x 5 it is 3; lcm(32, 3) = 96
    assert oracle.prune_step_lcm([4, 8, 16], [3, 5]) == 96
    assert oracle.prune_step_lcm([7], [7]) == 1               # one unsplit iterator: any single filter
    assert oracle.prune_step_lcm([2, 6], [2, 6], 16, 8) == 32   # 16 * 12 / 6 = 32 and 8 * 12 / 6 = 16


def test_task_order_matches_the_papers_worked_example():
    ex = _paper_examples()
    times = [float(v) for v in ex["order_times"].split()]
    counts = [int(v) for v in ex["order_subgraphs"].split()]
    impacts = [float(v) for v in ex["order_impacts"].split()]
    assert [round(t * c, 3) for t, c in zip(times, counts)] == impacts
    assert [i + 1 for i in oracle.task_order(times, counts)] == [int(v) for v in ex["order_result"].split()]
    assert oracle.task_order([1.0, 2.0, 1.0, 0.5], [2, 1, 2, 4]) == [0, 1, 2, 3]     # all impacts equal: index order
    assert oracle.task_order([], []) == []


def test_task_table_groups_identical_shapes():
    # pruned ResNet-18: 20 conv layers, 15 distinct tasks; pruned MobileNetV2: 52 conv layers, 30 distinct
    for fn, layers, tasks in ((wl.resnet18, 20, 15), (wl.mobilenet_v2, 52, 30)):
        tab = oracle.task_table(fn())
        assert sum(len(names) for _, names in tab) == layers and len(tab) == tasks
    tab = dict((tuple(n), k) for k, n in oracle.task_table(wl.resnet18()))
    assert ("l1b1_conv1", "l1b2_conv1") in tab and ("l3b1_conv2", "l3b2_conv2") in tab


# ------------------------------------------------------------------ wiring of the layer tables
# The networks written out a second time, straight from their published architecture, with
# torch.nn.functional in float64 and none of the tables' wiring (tensor names, residual sources,
# activation placement): only the weights are looked up, by layer name.

def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).double()


def _fconv(x, wb, stride=1, pad=0, groups=1, act=None):
    import torch.nn.functional as F
    y = F.conv2d(x, _t(wb[0]), _t(wb[1]), stride=stride, padding=pad, groups=groups)
    if act == "relu":
        y = F.relu(y)
    elif act == "relu6":
        y = torch.clamp(y, 0.0, 6.0)
    return y


def _torch_vgg16(W, x):
    import torch.nn.functional as F
    i = 0
    for block in (2, 2, 3, 3, 3):
        for _ in range(block):
            i += 1
            x = _fconv(x, W["c%d" % i], 1, 1, act="relu")
        x = F.max_pool2d(x, 2, 2)
    x = x.flatten(1)
    x = F.relu(F.linear(x, _t(W["fc1"][0]), _t(W["fc1"][1])))
    return F.linear(x, _t(W["fc2"][0]), _t(W["fc2"][1]))


def _torch_resnet18(W, x):
    import torch.nn.functional as F
    x = _fconv(x, W["stem"], 2, 3, act="relu")
    x = F.max_pool2d(x, 3, 2, 1)
    for stage in (1, 2, 3, 4):
        for block in (1, 2):
            pre = "l%db%d" % (stage, block)
            stride = 2 if (stage > 1 and block == 1) else 1
            shortcut = _fconv(x, W[pre + "_down"], stride, 0) if (pre + "_down") in W else x
            h = _fconv(x, W[pre + "_conv1"], stride, 1, act="relu")
            h = _fconv(h, W[pre + "_conv2"], 1, 1)
            x = F.relu(h + shortcut)
    x = x.mean(dim=(2, 3))
    return F.linear(x, _t(W["fc"][0]), _t(W["fc"][1]))


def _torch_inverted_residuals(W, x, settings, act, first_block):
    b = first_block
    for expand, cout, repeats, stride, k in settings:
        for j in range(repeats):
            s = stride if j == 0 else 1
            pre = "b%d" % b
            h = x
            if (pre + "_exp") in W:
                h = _fconv(h, W[pre + "_exp"], act=act)
            ch = h.shape[1]
            h = _fconv(h, W[pre + "_dw"], s, k // 2, groups=ch, act=act)
            h = _fconv(h, W[pre + "_proj"])
            x = x + h if (s == 1 and x.shape[1] == cout) else h
            b += 1
    return x


def _torch_mobilenet_v2(W, x):
    import torch.nn.functional as F
    x = _fconv(x, W["stem"], 2, 1, act="relu6")
    settings = [(1, 16, 1, 1, 3), (6, 24, 2, 2, 3), (6, 32, 3, 2, 3), (6, 64, 4, 2, 3), (6, 96, 3, 1, 3),
                (6, 160, 3, 2, 3), (6, 320, 1, 1, 3)]
    x = _torch_inverted_residuals(W, x, settings, "relu6", 1)
    x = _fconv(x, W["last"], act="relu6").mean(dim=(2, 3))
    return F.linear(x, _t(W["fc"][0]), _t(W["fc"][1]))


def _torch_mnasnet(W, x):
    import torch.nn.functional as F
    x = _fconv(x, W["stem"], 2, 1, act="relu")
    x = _fconv(x, W["sep_dw"], 1, 1, groups=32, act="relu")
    x = _fconv(x, W["sep_pw"])
    settings = [(3, 24, 3, 2, 3), (3, 40, 3, 2, 5), (6, 80, 3, 2, 5), (6, 96, 2, 1, 3), (6, 192, 4, 2, 5), (6, 320, 1, 1, 3)]
    x = _torch_inverted_residuals(W, x, settings, "relu", 1)
    x = _fconv(x, W["last"], act="relu").mean(dim=(2, 3))
    return F.linear(x, _t(W["fc"][0]), _t(W["fc"][1]))


@pytest.mark.parametrize("name,forward,hw", [("vgg16_cifar", _torch_vgg16, 32), ("resnet18", _torch_resnet18, 32),
                                             ("mobilenet_v2", _torch_mobilenet_v2, 32), ("mnasnet1_0", _torch_mnasnet, 32),
                                             ("resnet18", _torch_resnet18, 64)])
def test_table_wiring_against_the_architecture_written_out(name, forward, hw):
    for pruned in (False, True):
        model = _tiny(wl.MODELS[name](), hw)
        weights = wl.model_weights(model)
        if pruned:
            weights, _ = oracle.prune_model(model, weights)
        x = wl.model_input(model, 2)
        ref = forward(weights, _t(x).permute(0, 3, 1, 2)).numpy()
        got = oracle.model_ref(model, weights, x)
        assert got.shape == ref.shape
        assert np.max(np.abs(got - ref)) <= 1e-10 * np.max(np.abs(ref)), (name, pruned)

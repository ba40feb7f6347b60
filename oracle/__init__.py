"""CPU oracle of the pruned-CNN task path.  TEST INFRASTRUCTURE ONLY.

A plain, slow float64 implementation of what the CUDA library computes: the fused
Conv2d + bias + activation task (paper Sec. 3.4 / 3.5), L1-norm filter selection and the
slicing of the next layer's input channels (Sec. 3.5, last paragraph; Sec. 2.1, Fig. 2), and
the pruned networks of Sec. 4.1 run as a chain of such tasks.  Only the tests, the smoke
check and the benchmark's CPU-baseline legs may use it; the library itself never does, and
nothing here is shared with, or imported by, the CUDA path.

The arithmetic lives in ``oracle.c`` (7-loop direct convolution with float64 accumulation,
pools, fully-connected layers, bfloat16 rounding, integer L1 norms, stable selection); this
file marshals numpy arrays into it and walks layer tables.

Parity pins: every function here is pinned by ``tests/test_oracle_pins.py`` (hand-computed
cases, closed forms, invariants, the paper's model totals); none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

ACT = {"none": 0, "relu": 1, "relu6": 2}


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (OpenMP over images and output rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _dp(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    """Threads the OpenMP loops use (all cores unless OMP_NUM_THREADS says otherwise)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def out_size(H, R, stride, pad):
    return (H + 2 * pad - R) // stride + 1


def conv2d(x, w, b=None, stride=1, pad=0, groups=1, act="none", res=None, with_bound=False):
    """x [N,H,W,C], w [K,C/groups,R,S], b [K], res [N,P,Q,K] -> y [N,P,Q,K] (float64).
    y = act(b + sum_{c,r,s} x[n, p*stride-pad+r, q*stride-pad+s, c] * w[k,c,r,s] + res).
    with_bound: also return |b| + sum |x||w| + |res| per element (the error scale)."""
    x, w, b, res = _f64(x), _f64(w), _f64(b), _f64(res)
    N, H, W, C = x.shape
    K, cg, R, S = w.shape
    assert cg * groups == C and K % groups == 0
    P, Q = out_size(H, R, stride, pad), out_size(W, S, stride, pad)
    y = np.empty((N, P, Q, K), dtype=np.float64)
    bound = np.empty_like(y) if with_bound else None
    if res is not None:
        assert res.shape == y.shape
    _load().oracle_conv2d(_dp(x), N, H, W, C, _dp(w), K, R, S, groups, _dp(b), stride, pad, ACT[act],
                          _dp(res), _dp(y), _dp(bound))
    return (y, bound) if with_bound else y


def conv2d_points(x, w, b, stride, pad, groups, act, res, pts):
    """The same task evaluated only at output coordinates pts [n,4] = (n, p, q, k).
    Returns (values, bounds)."""
    x, w, b, res = _f64(x), _f64(w), _f64(b), _f64(res)
    N, H, W, C = x.shape
    K, cg, R, S = w.shape
    pts = np.ascontiguousarray(pts, dtype=np.int32)
    y = np.empty(len(pts), dtype=np.float64)
    bound = np.empty(len(pts), dtype=np.float64)
    _load().oracle_conv2d_points(_dp(x), N, H, W, C, _dp(w), K, R, S, groups, _dp(b), stride, pad, ACT[act],
                                 _dp(res), _dp(pts), len(pts), _dp(y), _dp(bound))
    return y, bound


def maxpool(x, k, stride, pad):
    x = _f64(x)
    N, H, W, C = x.shape
    y = np.empty((N, out_size(H, k, stride, pad), out_size(W, k, stride, pad), C), dtype=np.float64)
    _load().oracle_maxpool(_dp(x), N, H, W, C, k, stride, pad, _dp(y))
    return y


def gap(x):
    x = _f64(x)
    N, H, W, C = x.shape
    y = np.empty((N, C), dtype=np.float64)
    _load().oracle_gap(_dp(x), N, H, W, C, _dp(y))
    return y


def fc(x, w, b=None, act="none", with_bound=False):
    x, w, b = _f64(x), _f64(w), _f64(b)
    N, nin = x.shape
    nout = w.shape[0]
    assert w.shape[1] == nin
    y = np.empty((N, nout), dtype=np.float64)
    bound = np.empty_like(y) if with_bound else None
    _load().oracle_fc(_dp(x), N, nin, _dp(w), nout, _dp(b), ACT[act], _dp(y), _dp(bound))
    return (y, bound) if with_bound else y


def round_bf16(x):
    """Nearest bfloat16 (ties to even) of every element, returned as float64."""
    x = _f64(x)
    y = np.empty_like(x)
    _load().oracle_round_bf16(_dp(x), ctypes.c_size_t(x.size), _dp(y))
    return y


def l1_norms(w) -> np.ndarray:
    """Per-filter sum of |w| on the 2^-40 grid, as int64 (paper Sec. 3.5)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    K = w.shape[0]
    inner = w.size // K
    norms = np.empty(K, dtype=np.int64)
    _load().oracle_l1_norms(_dp(w), K, ctypes.c_size_t(inner), _dp(norms))
    return norms


def l1_norms_exact(w) -> list:
    """Per-filter sum of |w| correctly rounded to float64 (math.fsum), for cross-checking the grid."""
    w = np.asarray(w, dtype=np.float64)
    return [math.fsum(abs(v) for v in w[k].ravel()) for k in range(w.shape[0])]


def select_indices(w, keep_k: int) -> np.ndarray:
    """Indices (ascending) of the keep_k filters with the largest L1 norm; ties keep the lower index."""
    norms = l1_norms(w)
    K = len(norms)
    assert 1 <= keep_k <= K
    kept = np.empty(keep_k, dtype=np.int32)
    _load().oracle_select(_dp(norms), K, keep_k, _dp(kept))
    return kept


def select_indices_shared(ws, keep_k: int) -> np.ndarray:
    """Dependency-aware selection (paper Sec. 3.5, last paragraph): layers whose outputs are added
    on a shortcut lose the SAME output channels.  The importance of channel k is the sum over the
    member layers of that channel's L1 norm (each on the 2^-40 grid); the keep_k largest survive,
    ties keep the lower index.  ws: list of weight tensors that all have K filters."""
    K = ws[0].shape[0]
    total = np.zeros(K, dtype=np.int64)
    for w in ws:
        assert w.shape[0] == K
        total += l1_norms(w)
    assert 1 <= keep_k <= K
    kept = np.empty(keep_k, dtype=np.int32)
    _load().oracle_select(_dp(total), K, keep_k, _dp(kept))
    return kept


def select_filters(w, b, keep_k, w_next=None, next_is_depthwise=False):
    """Prune a layer to keep_k filters and make the next layer consistent (paper Sec. 3.5):
    returns (kept, w[kept], b[kept], w_next sliced).  A dense next layer [K2,K,R2,S2] loses
    input channels; a depthwise next layer [K,1,R2,S2] loses whole filters."""
    kept = select_indices(w, keep_k)
    w_out = np.ascontiguousarray(w[kept])
    b_out = None if b is None else np.ascontiguousarray(b[kept])
    wn = None
    if w_next is not None:
        wn = np.ascontiguousarray(w_next[kept] if next_is_depthwise else w_next[:, kept])
    return kept, w_out, b_out, wn


# ----------------------------------------------------------------------------
# whole models (layer tables come from the caller; see workloads/)
# ----------------------------------------------------------------------------

def prune_model(model: dict, weights: dict):
    """Apply L1 filter pruning to every layer of the table that has a keep count and slice
    its consumers.  Layers that carry the same ``share`` tag write tensors that meet in a
    residual add: they are ranked together (select_indices_shared) when the first of them is
    reached and all lose the same filters (the ranking uses the weights as given, before any
    slicing).  Returns (pruned weights: name -> (w, b), kept:
    name -> indices)."""
    by = {l["name"]: l for l in model["layers"]}
    out = {k: (w.copy(), b.copy()) for k, (w, b) in weights.items()}
    kept_all = {}
    # shared groups are ranked once, on the members' weights as given (full width, before any slicing)
    shared = {}
    for l in model["layers"]:
        tag = l.get("share") if l["kind"] == "conv" else None
        if tag is not None and l["keep"] is not None and tag not in shared:
            members = [m for m in model["layers"] if m["kind"] == "conv" and m.get("share") == tag]
            assert all(m["keep"] == l["keep"] for m in members)
            shared[tag] = select_indices_shared([weights[m["name"]][0] for m in members], l["keep"])

    def follow(layer, kept):
        for cname, how in layer["consumers"]:
            w, b = out[cname]
            if how in ("in_channels", "fc_in"):
                out[cname] = (np.ascontiguousarray(w[:, kept]), b)
            elif how == "depthwise":
                out[cname] = (np.ascontiguousarray(w[kept]), np.ascontiguousarray(b[kept]))
                follow(by[cname], kept)
            else:
                raise ValueError(how)

    for l in model["layers"]:
        if l["kind"] == "conv" and l["keep"] is not None:
            w, b = out[l["name"]]
            tag = l.get("share")
            kept = select_indices(w, l["keep"]) if tag is None else shared[tag]
            out[l["name"]] = (np.ascontiguousarray(w[kept]), np.ascontiguousarray(b[kept]))
            kept_all[l["name"]] = kept
            follow(l, kept)
    return out, kept_all


def model_ref(model: dict, weights: dict, x, matched: bool = False, keep_tensors: bool = False):
    """Run the layer table on x [N,H,W,C] with the given (already pruned) weights.

    matched=False: float32 data as given, float64 arithmetic, no rounding anywhere.
    matched=True: x, every w and every stored activation are rounded to bfloat16 at the points
    where the CUDA library stores bfloat16 (after each task's epilogue, after pools and the
    global average pool); biases and the final logits stay unrounded.
    Returns logits [N, classes] (and the dict of all tensors if keep_tensors)."""
    rnd = round_bf16 if matched else (lambda a: a)
    t = {"x": rnd(np.asarray(x, dtype=np.float64))}
    last = model["output"]
    for l in model["layers"]:
        a = t[l["in"]]
        kind = l["kind"]
        if kind == "conv":
            w, b = weights[l["name"]]
            groups = w.shape[0] if l["groups"] > 1 else 1
            res = t[l["res"]] if l.get("res") else None
            y = conv2d(a, rnd(w), b, l["stride"], l["pad"], groups, l["act"], res)
            if l.get("pool") == "max2x2":
                y = maxpool(y, 2, 2, 0)
            t[l["out"]] = rnd(y)
        elif kind == "maxpool":
            t[l["out"]] = maxpool(a, l["k"], l["stride"], l["pad"])
        elif kind == "gap":
            t[l["out"]] = rnd(gap(a))
        elif kind == "flatten":
            t[l["out"]] = a.reshape(a.shape[0], -1)
        elif kind == "fc":
            w, b = weights[l["name"]]
            y = fc(a, rnd(w), b, l["act"])
            t[l["out"]] = y if l["out"] == last else rnd(y)
        else:
            raise ValueError(kind)
    return (t[last], t) if keep_tensors else t[last]


# ----------------------------------------------------------------------------
# pruning decision and task ordering (host-side steps of the method)
# ----------------------------------------------------------------------------

def prune_step_lcm(L1, L2, unit1: int = 1, unit2: int = 1) -> int:
    """Minimum number of filters to prune while keeping the structure of a task's program
    (paper Sec. 3.5, the LCM equation).  L1 and L2 are the factors into which the program splits
    the two iterators that run over the filters; removing one slice along a factor l of an
    iterator prunes (product of its factors) / l filters, the smallest such number is
    product / max factor, and the step that suits both iterators is the least common multiple
    of the two.  unit1 / unit2: filters behind one count of the factors (1 in the paper's loop
    nests; larger when the innermost group of filters is fixed by an instruction and cannot
    shrink)."""
    def smallest(L, unit):
        L = [int(v) for v in L]
        assert L and all(v >= 1 for v in L)
        prod = 1
        for v in L:
            prod *= v
        return unit * (prod // max(L))
    a, b = smallest(L1, unit1), smallest(L2, unit2)
    return a * b // math.gcd(a, b)


def task_order(times, counts) -> list:
    """Tasks ordered by pruning impact = execution time x number of subgraphs that share the
    task, largest first (paper Sec. 3.3); equal impacts keep the lower index first."""
    impact = [float(t) * int(c) for t, c in zip(times, counts)]
    return sorted(range(len(impact)), key=lambda i: (-impact[i], i))


def task_table(model: dict) -> list:
    """The task / subgraph relationship of a layer table (paper Sec. 3.4): conv layers whose
    shape and fused properties agree form one task.  Returns a list of (key, [layer names]) in
    order of first appearance; key = (C, K, H, W, R, S, stride, pad, groups, act, residual, pool)
    with the widths after pruning."""
    import workloads as wl   # layer tables are data shared with the library's harness
    m = wl.pruned_shapes(model)
    sz = wl.spatial_sizes(m)
    tasks, order = {}, []
    for l in m["layers"]:
        if l["kind"] != "conv":
            continue
        h, w = sz[l["in"]]
        key = (l["C"], l["K"], h, w, l["R"], l["S"], l["stride"], l["pad"], l["groups"], l["act"],
               l.get("res") is not None, l.get("pool"))
        if key not in tasks:
            tasks[key] = []
            order.append(key)
        tasks[key].append(l["name"])
    return [(k, tasks[k]) for k in order]


def conv_flops(N, C, K, P, Q, R, S, groups=1) -> int:
    """Floating-point operations of one conv task: 2 N K C P Q R S / groups."""
    return 2 * N * K * C * P * Q * R * S // groups


def model_counts(model: dict) -> dict:
    """Multiply-accumulates per image and parameter count (weights + biases) of a layer table,
    from the widths in the table as given."""
    H, W, _ = model["input"]
    sz = {"x": (H, W)}
    macs = params = 0
    for l in model["layers"]:
        h, w = sz[l["in"]]
        if l["kind"] == "conv":
            p, q = out_size(h, l["R"], l["stride"], l["pad"]), out_size(w, l["S"], l["stride"], l["pad"])
            macs += conv_flops(1, l["C"], l["K"], p, q, l["R"], l["S"], l["groups"]) // 2
            params += l["K"] * (l["C"] // l["groups"]) * l["R"] * l["S"] + l["K"]
            if l.get("pool") == "max2x2":
                p, q = p // 2, q // 2
            sz[l["out"]] = (p, q)
        elif l["kind"] == "maxpool":
            sz[l["out"]] = (out_size(h, l["k"], l["stride"], l["pad"]), out_size(w, l["k"], l["stride"], l["pad"]))
        elif l["kind"] == "fc":
            macs += l["in_features"] * l["out_features"]
            params += l["in_features"] * l["out_features"] + l["out_features"]
            sz[l["out"]] = (1, 1)
        else:
            sz[l["out"]] = (1, 1)
    return {"macs": macs, "params": params}

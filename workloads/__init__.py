"""Seeded synthetic workloads: tensors and layer tables of the pruned CNNs.

This module is data only.  It draws random tensors from a counter-based
generator and lists, layer by layer, the shapes of the networks the paper
evaluates (VGG-16 for 32x32 inputs, ResNet-18 and MobileNetV2 for 224x224
inputs; paper Sec. 4.1) together with the number of filters each pruned layer
keeps.  It contains none of the method's arithmetic: no convolution, no norm,
no ranking, no slicing.  Both the CPU oracle and the CUDA library are fed from
here, so that they see identical bytes.

Generator.  Element ``i`` of stream ``t`` under seed ``s`` is a function of
``(s, t, i)`` alone: two 64-bit words come from the splitmix64 finaliser applied
to a counter, they become two uniforms in (0, 1), and the Box-Muller transform
turns them into one standard normal in float64, which is then cast to float32.

Layer tables.  A model is a dict ``{"name", "input": (H, W, C), "layers": [...],
"output": tensor name}``.  Every layer reads tensor ``"in"`` and writes tensor
``"out"`` (names are strings).  Layer kinds:

``conv``     C, K, R, S, stride, pad, groups, act in {"none", "relu", "relu6"},
             optional ``res`` (tensor added before the activation), optional
             ``pool`` = "max2x2" (2x2 stride-2 max-pool applied to the result),
             ``keep`` = filters kept by L1 pruning (None: layer is not pruned),
             optional ``share`` = tag of a group of layers whose outputs meet in a residual
             add and therefore keep the SAME filters (one ranking for the whole group),
             ``consumers`` = layers whose input channels follow this layer's
             kept filters: list of (layer name, how) with how in
             {"in_channels", "depthwise", "fc_in"}.
``maxpool``  k, stride, pad (pad positions never win the max).
``gap``      global average pool over H x W.
``fc``       in_features, out_features, act.

Channel counts in a table are the FULL (unpruned) widths; ``pruned_shapes``
gives the widths after pruning.
"""
from __future__ import annotations

import copy
import math

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """The splitmix64 output function (Steele, Lea, Flood 2014) on uint64 arrays."""
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """``n`` standard normals (float64) for ``(seed, stream)``; element i depends on i only."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([np.uint64(seed) * _GOLDEN + np.uint64(stream)], dtype=np.uint64))
        key = _splitmix64(key ^ np.uint64(stream) * _M2)[0]
        out = np.empty(n, dtype=np.float64)
        chunk = 1 << 22
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            ctr = np.arange(lo, hi, dtype=np.uint64) * np.uint64(2)
            a = _splitmix64(key + (ctr + np.uint64(1)) * _GOLDEN)
            b = _splitmix64(key + (ctr + np.uint64(2)) * _GOLDEN)
            u1 = ((a >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
            u2 = ((b >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
            out[lo:hi] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return out


def normal_f32(seed: int, stream: int, shape, std: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    return (normal(seed, stream, n) * std).astype(np.float32).reshape(shape)


# ----------------------------------------------------------------------------
# layer tables
# ----------------------------------------------------------------------------

def _conv(name, tin, tout, C, K, R, stride, pad, act, groups=1, res=None, pool=None,
          keep=None, consumers=(), share=None):
    return {"kind": "conv", "name": name, "in": tin, "out": tout, "C": C, "K": K, "R": R, "S": R,
            "stride": stride, "pad": pad, "groups": groups, "act": act, "res": res, "pool": pool,
            "keep": keep, "consumers": list(consumers), "share": share}


def single_task() -> dict:
    """One 3x3 task, 64 -> 64 filters of which 48 are kept, 32x32 input (the small case)."""
    layers = [_conv("conv", "x", "y", 64, 64, 3, 1, 1, "relu", keep=48)]
    return {"name": "single_task", "input": (32, 32, 64), "layers": layers, "output": "y", "seed": 1001}


VGG16_WIDTHS = [64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]
VGG16_KEEP = [45, 58, 101, 96, 187, 171, 163, 301, 250, 212, 198, 207, 243]
_VGG16_POOL_AFTER = {2, 4, 7, 10, 13}


def vgg16_cifar(keep=VGG16_KEEP) -> dict:
    """Thirteen 3x3 conv+ReLU layers in five blocks with a 2x2 max-pool after each block,
    then FC 512 -> 512 -> 10, for 3x32x32 inputs (the network of the paper's Sec. 3 study)."""
    layers = []
    c, t = 3, "x"
    for i, k in enumerate(VGG16_WIDTHS, start=1):
        nxt = ("c%d" % (i + 1), "in_channels") if i < 13 else ("fc1", "fc_in")
        layers.append(_conv("c%d" % i, t, "a%d" % i, c, k, 3, 1, 1, "relu",
                            pool="max2x2" if i in _VGG16_POOL_AFTER else None,
                            keep=None if keep is None else keep[i - 1], consumers=[nxt]))
        c, t = k, "a%d" % i
    layers.append({"kind": "flatten", "name": "flat", "in": t, "out": "f0"})
    layers.append({"kind": "fc", "name": "fc1", "in": "f0", "out": "f1", "in_features": 512,
                   "out_features": 512, "act": "relu"})
    layers.append({"kind": "fc", "name": "fc2", "in": "f1", "out": "logits", "in_features": 512,
                   "out_features": 10, "act": "none"})
    return {"name": "vgg16_cifar", "input": (32, 32, 3), "layers": layers, "output": "logits", "seed": 1002}


def resnet18(keep_num=7, keep_den=10, out_num=None, out_den=4) -> dict:
    """ResNet-18 for 3x224x224 inputs.  The first conv of every BasicBlock keeps
    floor(keep_num * width / keep_den) filters.  With out_num=None block outputs keep their
    width so that the residual adds keep their shapes; keep_num=None gives the unpruned network.
    With out_num set, the tensors that meet in the residual adds of a stage (the stem or the
    stage's 1x1 shortcut conv, and the second conv of both blocks) are pruned too, to
    floor(out_num * width / out_den) filters, and all of them lose the same filters (one
    ``share`` group per stage: the dependency-aware pruning of the paper's Sec. 3.5)."""
    def okeep(w):
        return None if out_num is None else (out_num * w) // out_den

    # consumers of a stage's shared tensors are filled in as the readers appear
    layers = [_conv("stem", "x", "s0", 3, 64, 7, 2, 3, "relu", keep=okeep(64), share="stage1" if out_num else None),
              {"kind": "maxpool", "name": "pool0", "in": "s0", "out": "p0", "k": 3, "stride": 2, "pad": 1}]
    t, c = "p0", 64
    writer = layers[0]          # the layer that wrote tensor t
    for si, w in enumerate([64, 128, 256, 512], start=1):
        tag = "stage%d" % si if out_num else None
        for bi in (1, 2):
            stride = 2 if (si > 1 and bi == 1) else 1
            pre = "l%db%d" % (si, bi)
            keep = None if keep_num is None else (keep_num * w) // keep_den
            ident = t
            if stride != 1 or c != w:
                layers.append(_conv(pre + "_down", t, pre + "_id", c, w, 1, stride, 0, "none", keep=okeep(w), share=tag))
                ident = pre + "_id"
                if out_num:
                    writer["consumers"].append((pre + "_down", "in_channels"))
            if out_num:
                writer["consumers"].append((pre + "_conv1", "in_channels"))
            layers.append(_conv(pre + "_conv1", t, pre + "_h", c, w, 3, stride, 1, "relu", keep=keep,
                                consumers=[(pre + "_conv2", "in_channels")]))
            layers.append(_conv(pre + "_conv2", pre + "_h", pre + "_o", w, w, 3, 1, 1, "relu", res=ident,
                                keep=okeep(w), share=tag))
            writer = layers[-1]
            t, c = pre + "_o", w
    layers.append({"kind": "gap", "name": "gap", "in": t, "out": "g"})
    layers.append({"kind": "fc", "name": "fc", "in": "g", "out": "logits", "in_features": 512,
                   "out_features": 1000, "act": "none"})
    if out_num:
        writer["consumers"].append(("fc", "fc_in"))
    return {"name": "resnet18", "input": (224, 224, 3), "layers": layers, "output": "logits", "seed": 1003}


def resnet18_shared() -> dict:
    """Pruned ResNet-18 whose block outputs are pruned as well, to 3/4 of their width, with one
    shared filter set per stage (see resnet18)."""
    m = resnet18(out_num=3)
    m["name"] = "resnet18_shared"
    return m


_MBV2_SETTING = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1),
                 (6, 160, 3, 2), (6, 320, 1, 1)]


def mobilenet_v2(keep_num=3, keep_den=4) -> dict:
    """MobileNetV2 (width 1.0) for 3x224x224 inputs: seventeen inverted-residual blocks,
    each 1x1 expand + ReLU6, 3x3 depthwise + ReLU6, 1x1 project, residual add where the
    block keeps its shape.  Every expand layer keeps floor(keep_num * width / keep_den)
    filters; the depthwise layer and the project layer's inputs follow.  The first block
    has expansion 1 and therefore no expand layer and nothing to prune."""
    layers = [_conv("stem", "x", "s0", 3, 32, 3, 2, 1, "relu6")]
    t, c, bi = "s0", 32, 0
    for tfac, cout, n, s in _MBV2_SETTING:
        for j in range(n):
            bi += 1
            stride = s if j == 0 else 1
            pre = "b%d" % bi
            hidden = c * tfac
            h = t
            if tfac != 1:
                keep = None if keep_num is None else (keep_num * hidden) // keep_den
                layers.append(_conv(pre + "_exp", t, pre + "_e", c, hidden, 1, 1, 0, "relu6", keep=keep,
                                    consumers=[(pre + "_dw", "depthwise")]))
                h = pre + "_e"
            layers.append(_conv(pre + "_dw", h, pre + "_d", hidden, hidden, 3, stride, 1, "relu6",
                                groups=hidden, consumers=[(pre + "_proj", "in_channels")]))
            res = t if (stride == 1 and c == cout) else None
            layers.append(_conv(pre + "_proj", pre + "_d", pre + "_o", hidden, cout, 1, 1, 0, "none", res=res))
            t, c = pre + "_o", cout
    layers.append(_conv("last", t, "l0", 320, 1280, 1, 1, 0, "relu6"))
    layers.append({"kind": "gap", "name": "gap", "in": "l0", "out": "g"})
    layers.append({"kind": "fc", "name": "fc", "in": "g", "out": "logits", "in_features": 1280,
                   "out_features": 1000, "act": "none"})
    return {"name": "mobilenet_v2", "input": (224, 224, 3), "layers": layers, "output": "logits", "seed": 1004}


# MnasNet-B1, depth multiplier 1.0 (Tan et al. 2019, the "MnasNet1.0" of the paper's Sec. 4.1):
# (expansion, output channels, repeats, stride of the first block, depthwise kernel size)
_MNASNET_SETTING = [(3, 24, 3, 2, 3), (3, 40, 3, 2, 5), (6, 80, 3, 2, 5), (6, 96, 2, 1, 3),
                    (6, 192, 4, 2, 5), (6, 320, 1, 1, 3)]


def mnasnet1_0(keep_num=3, keep_den=4) -> dict:
    """MnasNet1.0 for 3x224x224 inputs: 3x3 stride-2 stem to 32 channels, a depthwise-separable
    block to 16, six stacks of inverted-residual blocks (1x1 expand + ReLU, 3x3 or 5x5 depthwise
    + ReLU, 1x1 project, residual add where the block keeps its shape), 1x1 conv to 1280, global
    average pool, FC 1280 -> 1000.  Every expand layer keeps floor(keep_num * width / keep_den)
    filters; its depthwise layer and the project layer's inputs follow."""
    layers = [_conv("stem", "x", "s0", 3, 32, 3, 2, 1, "relu"),
              _conv("sep_dw", "s0", "s1", 32, 32, 3, 1, 1, "relu", groups=32),
              _conv("sep_pw", "s1", "s2", 32, 16, 1, 1, 0, "none")]
    t, c, bi = "s2", 16, 0
    for tfac, cout, n, s, k in _MNASNET_SETTING:
        for j in range(n):
            bi += 1
            stride = s if j == 0 else 1
            pre = "b%d" % bi
            hidden = c * tfac
            keep = None if keep_num is None else (keep_num * hidden) // keep_den
            layers.append(_conv(pre + "_exp", t, pre + "_e", c, hidden, 1, 1, 0, "relu", keep=keep,
                                consumers=[(pre + "_dw", "depthwise")]))
            layers.append(_conv(pre + "_dw", pre + "_e", pre + "_d", hidden, hidden, k, stride, k // 2, "relu",
                                groups=hidden, consumers=[(pre + "_proj", "in_channels")]))
            res = t if (stride == 1 and c == cout) else None
            layers.append(_conv(pre + "_proj", pre + "_d", pre + "_o", hidden, cout, 1, 1, 0, "none", res=res))
            t, c = pre + "_o", cout
    layers.append(_conv("last", t, "l0", 320, 1280, 1, 1, 0, "relu"))
    layers.append({"kind": "gap", "name": "gap", "in": "l0", "out": "g"})
    layers.append({"kind": "fc", "name": "fc", "in": "g", "out": "logits", "in_features": 1280,
                   "out_features": 1000, "act": "none"})
    return {"name": "mnasnet1_0", "input": (224, 224, 3), "layers": layers, "output": "logits", "seed": 1005}


MODELS = {"single_task": single_task, "vgg16_cifar": vgg16_cifar, "resnet18": resnet18,
          "mobilenet_v2": mobilenet_v2, "mnasnet1_0": mnasnet1_0, "resnet18_shared": resnet18_shared}


def layer_by_name(model: dict) -> dict:
    return {l["name"]: l for l in model["layers"]}


def pruned_shapes(model: dict) -> dict:
    """A copy of the table in which C, K, groups and in_features are the widths AFTER pruning
    (bookkeeping on integers only; which filters survive is decided elsewhere)."""
    m = copy.deepcopy(model)
    by = layer_by_name(m)

    def follow(src, keep):
        for cname, how in src["consumers"]:
            d = by[cname]
            if how == "in_channels":
                d["C"] = keep
            elif how == "depthwise":
                d["C"] = d["K"] = d["groups"] = keep
                follow(d, keep)
            elif how == "fc_in":
                d["in_features"] = keep
            else:
                raise ValueError(how)

    for l in m["layers"]:
        if l["kind"] == "conv" and l["keep"] is not None:
            l["K"] = l["keep"]
            follow(l, l["keep"])
    return m


def spatial_sizes(model: dict) -> dict:
    """Output (H, W) of every tensor of the table, from the usual floor formula."""
    H, W, _ = model["input"]
    sz = {"x": (H, W)}
    for l in model["layers"]:
        h, w = sz[l["in"]]
        if l["kind"] == "conv":
            p = (h + 2 * l["pad"] - l["R"]) // l["stride"] + 1
            q = (w + 2 * l["pad"] - l["S"]) // l["stride"] + 1
            if l["pool"] == "max2x2":
                p, q = p // 2, q // 2
            sz[l["out"]] = (p, q)
        elif l["kind"] == "maxpool":
            sz[l["out"]] = ((h + 2 * l["pad"] - l["k"]) // l["stride"] + 1,
                            (w + 2 * l["pad"] - l["k"]) // l["stride"] + 1)
        else:
            sz[l["out"]] = (1, 1)
    return sz


def model_weights(model: dict, seed: int | None = None) -> dict:
    """Full-width weights of every conv / fc layer: name -> (w, b), both float32.
    conv w is [K, C/groups, R, S], fc w is [out, in].  w ~ N(0, 2/fan_in) with the fan-in of
    the full layer, b ~ N(0, 0.01^2).  Layer number t (in table order) draws w from stream 2t
    and b from stream 2t+1 of the model's seed."""
    seed = model["seed"] if seed is None else seed
    out = {}
    t = 0
    for l in model["layers"]:
        if l["kind"] == "conv":
            cg = l["C"] // l["groups"]
            shape = (l["K"], cg, l["R"], l["S"])
            fan_in = cg * l["R"] * l["S"]
            nb = l["K"]
        elif l["kind"] == "fc":
            shape = (l["out_features"], l["in_features"])
            fan_in = l["in_features"]
            nb = l["out_features"]
        else:
            continue
        t += 1
        w = normal_f32(seed, 2 * t, shape, math.sqrt(2.0 / fan_in))
        b = normal_f32(seed, 2 * t + 1, (nb,), 0.01)
        out[l["name"]] = (w, b)
    return out


def model_input(model: dict, batch: int, seed: int | None = None) -> np.ndarray:
    """[batch, H, W, C] float32, i.i.d. N(0, 1), stream 0 of the model's seed."""
    seed = model["seed"] if seed is None else seed
    H, W, C = model["input"]
    return normal_f32(seed, 0, (batch, H, W, C))


def conv_task_tensors(seed: int, N, C, H, W, K, R, S, groups=1, with_res=False, P=None, Q=None):
    """Tensors of one stand-alone conv task: x [N,H,W,C], w [K,C/groups,R,S] (Kaiming-normal),
    b [K] and, if asked, a residual [N,P,Q,K]."""
    cg = C // groups
    x = normal_f32(seed, 0, (N, H, W, C))
    w = normal_f32(seed, 1, (K, cg, R, S), math.sqrt(2.0 / (cg * R * S)))
    b = normal_f32(seed, 2, (K,), 0.01)
    res = normal_f32(seed, 3, (N, P, Q, K)) if with_res else None
    return x, w, b, res


def conv_task_tensors_tiled(seed: int, N, C, H, W, K, R, S, groups=1, with_res=False, P=None, Q=None, base=4):
    """The tensors of conv_task_tensors for a LARGE batch without drawing every image: `base` images are drawn
    and image n is image n % base scaled by 1 + n / 256 (exact in float32 for n < 2^15), so that all images differ
    and an output written to the wrong image shows.  Input generation only: no part of the method."""
    nb = min(N, base)
    x, w, b, res = conv_task_tensors(seed, nb, C, H, W, K, R, S, groups, with_res, P, Q)
    scale = (1.0 + np.arange(N, dtype=np.float32) / 256.0).reshape(N, 1, 1, 1)
    idx = np.arange(N) % nb
    x = np.ascontiguousarray(x[idx] * scale)
    if res is not None:
        res = np.ascontiguousarray(res[idx] * scale)
    return x, w, b, res


def sweep_shapes() -> list:
    """The distinct full-width conv task shapes of the models (MnasNet1.0 adds its 5x5 depthwise layers), as dicts
    {C, K, H, W, R, S, stride, pad, groups, act}; depthwise shapes have groups == C == K."""
    seen, out = set(), []
    for fn in (single_task, vgg16_cifar, resnet18, mobilenet_v2, mnasnet1_0):
        m = fn()
        sz = spatial_sizes(m)
        for l in m["layers"]:
            if l["kind"] != "conv":
                continue
            h, w = sz[l["in"]]
            key = (l["C"], l["K"], h, w, l["R"], l["S"], l["stride"], l["pad"], l["groups"] == l["C"] and l["C"] > 1)
            if key in seen:
                continue
            seen.add(key)
            out.append({"C": l["C"], "K": l["K"], "H": h, "W": w, "R": l["R"], "S": l["S"],
                        "stride": l["stride"], "pad": l["pad"], "groups": l["groups"], "act": l["act"],
                        "model": m["name"], "layer": l["name"]})
    return out

"""ctypes binding of libcprune.so.  Same names as the C ABI; torch tensors are used only as device
buffers (``data_ptr``) and for their stream handles.  No arithmetic happens in this file."""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_int, c_int32, c_longlong, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcprune.so")

OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE_TOO_SMALL", 4: "CUDA", 5: "TIMEOUT",
                6: "INTERNAL", 7: "BAD_DATA"}
ACT = {"none": 0, "relu": 1, "relu6": 2}
POOL = {None: 0, "none": 0, "max2x2": 1, "max3x3s2": 2}
KERNEL = {"auto": 0, "direct": 1, "tensor": 2, "depthwise": 3}
KERNEL_NAMES = {v: k for k, v in KERNEL.items()}
FLAGS = {"im2col_only": 1, "pool_on_epilogue_warps": 2}
OP_CONV, OP_MAXPOOL, OP_GAP, OP_FC, OP_BLOCK = 1, 2, 3, 4, 5

# every symbol include/cprune.h declares
EXPORTS = [
    "cprune_status_string", "cprune_last_cuda_error", "cprune_padded_channels", "cprune_select_workspace_bytes",
    "cprune_select_filters", "cprune_select_filters_static", "cprune_gather_rows", "cprune_gather_columns", "cprune_task_plan", "cprune_plan_query",
    "cprune_plan_release", "cprune_cache_clear", "cprune_cache_stats", "cprune_pack_weights", "cprune_task_run",
    "cprune_cast_input", "cprune_widen_output", "cprune_maxpool", "cprune_global_avgpool", "cprune_fc_pack",
    "cprune_fc", "cprune_model_create", "cprune_model_run", "cprune_model_run_host", "cprune_model_tensor", "cprune_model_copy_tensor", "cprune_model_launches",
    "cprune_model_destroy", "cprune_poll_device_status", "cprune_select_shared", "cprune_prune_step",
    "cprune_task_estimate", "cprune_task_order", "cprune_model_task_table", "cprune_model_time_tasks",
    "cprune_selftest_wait_timeout", "cprune_block_plan", "cprune_block_query", "cprune_block_release", "cprune_block_pack",
    "cprune_block_run",
]


class CpruneError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__("%s failed: %s%s" % (where, STATUS_NAMES.get(status, status), (" (" + detail + ")") if detail else ""))


class TaskOpts(ctypes.Structure):
    _fields_ = [("activation", c_int), ("residual", c_int), ("pool", c_int), ("kernel", c_int), ("flags", c_int)]


class PlanInfo(ctypes.Structure):
    _fields_ = [(n, c_int) for n in ("N", "C", "H", "W", "K", "R", "S", "stride", "pad", "groups", "P", "Q", "out_h",
                                      "out_w", "c_pad", "k_pad", "kernel", "tile_m", "tile_n", "tile_k", "stages",
                                      "tiles_m", "tiles_n", "k_alloc")] + \
               [("packed_weight_bytes", c_size_t), ("packed_bias_bytes", c_size_t), ("workspace_bytes", c_size_t),
                ("flops", c_double), ("algorithmic_bytes", c_double), ("padded_flops", c_double), ("variant", c_int),
                ("splits", c_int), ("split_compute", c_int * 2), ("unit_compute", c_int), ("split_store", c_int * 2),
                ("unit_store", c_int), ("est_us", c_double)]

    def as_dict(self):
        d = {n: getattr(self, n) for n, _ in self._fields_}
        d["split_compute"], d["split_store"] = list(d["split_compute"]), list(d["split_store"])
        return d


class TaskEntry(ctypes.Structure):
    _fields_ = [("plan", c_void_p), ("count", c_int), ("first_task", c_int)]


class TaskDesc(ctypes.Structure):
    _fields_ = [("op", c_int), ("in_", c_int), ("out", c_int), ("res", c_int), ("plan", c_void_p), ("w", c_void_p),
                ("b", c_void_p), ("p0", c_int), ("p1", c_int), ("p2", c_int), ("p3", c_int), ("block", c_void_p)]


class BlockInfo(ctypes.Structure):
    _fields_ = [(n, c_int) for n in ("N", "C_in", "H", "W", "hidden", "C_out", "act", "act_out", "residual", "c_in_pad", "k_pad",
                                      "hid_alloc", "k_alloc")] + \
               [("packed_weight_bytes", c_size_t), ("packed_bias_bytes", c_size_t), ("flops", c_double),
                ("algorithmic_bytes", c_double), ("unfused_bytes", c_double), ("splits", c_int), ("workspace_bytes", c_size_t),
                ("est_us", c_double)]


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libcprune.so is missing; build it with `python -m paper_2207_01260_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.cprune_status_string.restype = c_char_p
        L.cprune_last_cuda_error.restype = c_char_p
        L.cprune_select_workspace_bytes.restype = c_size_t
        L.cprune_select_workspace_bytes.argtypes = [c_int]
        L.cprune_select_filters.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_int,
                                            c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                            c_size_t, c_void_p]
        L.cprune_select_filters_static.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_int,
                                                   c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        L.cprune_gather_rows.argtypes = [c_void_p, c_int, c_size_t, c_void_p, c_int, c_void_p, c_void_p]
        L.cprune_gather_columns.argtypes = [c_void_p, c_int, c_int, c_size_t, c_void_p, c_int, c_void_p, c_void_p]
        L.cprune_task_plan.argtypes = [c_int] * 10 + [POINTER(TaskOpts), POINTER(c_void_p)]
        L.cprune_plan_query.argtypes = [c_void_p, POINTER(PlanInfo)]
        L.cprune_plan_release.argtypes = [c_void_p]
        L.cprune_cache_clear.argtypes = [POINTER(c_int)]
        L.cprune_cache_stats.argtypes = [POINTER(c_int), POINTER(c_longlong)]
        L.cprune_pack_weights.argtypes = [c_void_p] * 6
        L.cprune_task_run.argtypes = [c_void_p] * 8
        L.cprune_cast_input.argtypes = [c_void_p, c_size_t, c_int, c_void_p, c_void_p]
        L.cprune_widen_output.argtypes = [c_void_p, c_size_t, c_void_p, c_void_p]
        L.cprune_maxpool.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p]
        L.cprune_global_avgpool.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p]
        L.cprune_fc_pack.argtypes = [c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p]
        L.cprune_fc.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p]
        L.cprune_model_create.argtypes = [c_int, c_int, c_int, c_int, POINTER(TaskDesc), c_int, POINTER(c_void_p)]
        L.cprune_model_run.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p]
        L.cprune_model_run_host.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p]
        L.cprune_model_tensor.argtypes = [c_void_p, c_int, POINTER(c_void_p), POINTER(c_int), POINTER(c_int),
                                          POINTER(c_int), POINTER(c_int)]
        L.cprune_model_copy_tensor.argtypes = [c_void_p, c_int, c_void_p, c_void_p]
        L.cprune_model_launches.argtypes = [c_void_p]
        L.cprune_model_destroy.argtypes = [c_void_p]
        L.cprune_poll_device_status.argtypes = [c_void_p]
        L.cprune_select_shared.argtypes = [POINTER(c_void_p), POINTER(c_size_t), c_int, c_int, c_int, c_void_p, c_void_p,
                                           c_size_t, c_void_p]
        L.cprune_prune_step.argtypes = [c_void_p, POINTER(c_int)]
        L.cprune_task_estimate.argtypes = [c_void_p, c_int, POINTER(c_double)]
        L.cprune_task_order.argtypes = [POINTER(c_double), POINTER(c_int), c_int, POINTER(c_int)]
        L.cprune_model_task_table.argtypes = [c_void_p, POINTER(TaskEntry), c_int, POINTER(c_int)]
        L.cprune_model_time_tasks.argtypes = [c_void_p, c_int, POINTER(c_double), c_void_p]
        L.cprune_selftest_wait_timeout.argtypes = [c_void_p]
        L.cprune_block_plan.argtypes = [c_int] * 9 + [POINTER(c_void_p)]
        L.cprune_block_query.argtypes = [c_void_p, POINTER(BlockInfo)]
        L.cprune_block_release.argtypes = [c_void_p]
        L.cprune_block_pack.argtypes = [c_void_p] * 10
        L.cprune_block_run.argtypes = [c_void_p] * 7
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != OK:
        detail = lib().cprune_last_cuda_error().decode() if status == 4 else ""
        raise CpruneError(status, where, detail)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _dev_f32(t):
    assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    return t


def cprune_padded_channels(C: int) -> int:
    return lib().cprune_padded_channels(C)


def cprune_select_workspace_bytes(K: int) -> int:
    return lib().cprune_select_workspace_bytes(K)


def cprune_select_filters(w, keep_k, b=None, w_next=None, next_is_depthwise=False, workspace=None, stream=None):
    """w [K,C,R,S] float32 on the device.  Returns (kept_idx int32 [keep_k], w_out, b_out, w_next_out)."""
    w = _dev_f32(w)
    K, C, R, S = w.shape
    dev = w.device
    kk = max(int(keep_k), 0)
    kept = torch.empty(kk, dtype=torch.int32, device=dev)
    w_out = torch.empty((kk, C, R, S), dtype=torch.float32, device=dev)
    b_out = torch.empty(kk, dtype=torch.float32, device=dev) if b is not None else None
    K2 = R2 = S2 = 0
    wn_out = None
    if w_next is not None:
        w_next = _dev_f32(w_next)
        if next_is_depthwise:
            _, _, R2, S2 = w_next.shape
            wn_out = torch.empty((kk, 1, R2, S2), dtype=torch.float32, device=dev)
        else:
            K2, _, R2, S2 = w_next.shape
            wn_out = torch.empty((K2, kk, R2, S2), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(max(cprune_select_workspace_bytes(K), 16), dtype=torch.uint8, device=dev)
    st = lib().cprune_select_filters(_ptr(w), _ptr(b), K, C, R, S, int(keep_k), _ptr(w_next), K2, R2, S2,
                                     1 if next_is_depthwise else 0, _ptr(kept), _ptr(w_out), _ptr(b_out), _ptr(wn_out),
                                     _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "cprune_select_filters")
    return kept, w_out, b_out, wn_out


SELECT_STATIC_MAX_FILTERS = 4096


def cprune_select_filters_static(w, keep_k, kept_idx, w_out, b=None, b_out=None, w_next=None, w_next_out=None,
                                 next_is_depthwise=False, stream=None):
    """Selection without any device allocation: the caller passes every output buffer and the library
    uses its built-in scratch (at most SELECT_STATIC_MAX_FILTERS filters).  For callers that cannot
    allocate: serving loops, processes with a fixed memory budget.  Calls that overlap on the GPU race
    on the shared scratch, so keep them ordered on one stream."""
    w = _dev_f32(w)
    K, C, R, S = w.shape
    K2 = R2 = S2 = 0
    if w_next is not None:
        w_next = _dev_f32(w_next)
        if next_is_depthwise:
            _, _, R2, S2 = w_next.shape
        else:
            K2, _, R2, S2 = w_next.shape
    st = lib().cprune_select_filters_static(_ptr(w), _ptr(b), K, C, R, S, int(keep_k), _ptr(w_next), K2, R2, S2,
                                            1 if next_is_depthwise else 0, _ptr(kept_idx), _ptr(w_out), _ptr(b_out),
                                            _ptr(w_next_out), _stream(stream))
    _check(st, "cprune_select_filters_static")
    return kept_idx, w_out, b_out, w_next_out


def cprune_select_shared(ws, keep_k, workspace=None, stream=None):
    """ws: list of float32 device tensors that all have K filters (dim 0).  Returns kept_idx int32 [keep_k]: the
    filters with the largest norm summed over the members."""
    ws = [_dev_f32(w) for w in ws]
    K = ws[0].shape[0]
    ptrs = (c_void_p * len(ws))(*[w.data_ptr() for w in ws])
    inner = (c_size_t * len(ws))(*[w.numel() // K for w in ws])
    kept = torch.empty(max(int(keep_k), 0), dtype=torch.int32, device=ws[0].device)
    if workspace is None:
        workspace = torch.empty(max(cprune_select_workspace_bytes(K), 16), dtype=torch.uint8, device=ws[0].device)
    _check(lib().cprune_select_shared(ptrs, inner, len(ws), K, int(keep_k), _ptr(kept), _ptr(workspace),
                                      workspace.numel(), _stream(stream)), "cprune_select_shared")
    return kept


def cprune_gather_rows(t, idx, stream=None):
    """out[j] = t[idx[j]] along dim 0."""
    t = _dev_f32(t)
    rows = t.shape[0]
    inner = t.numel() // rows
    out = torch.empty((idx.numel(),) + tuple(t.shape[1:]), dtype=torch.float32, device=t.device)
    _check(lib().cprune_gather_rows(_ptr(t), rows, inner, _ptr(idx), idx.numel(), _ptr(out), _stream(stream)),
           "cprune_gather_rows")
    return out


def cprune_gather_columns(t, idx, stream=None):
    """out[:, j] = t[:, idx[j]] along dim 1."""
    t = _dev_f32(t)
    outer, cols = t.shape[0], t.shape[1]
    inner = t.numel() // (outer * cols)
    out = torch.empty((outer, idx.numel()) + tuple(t.shape[2:]), dtype=torch.float32, device=t.device)
    _check(lib().cprune_gather_columns(_ptr(t), outer, cols, inner, _ptr(idx), idx.numel(), _ptr(out), _stream(stream)),
           "cprune_gather_columns")
    return out


class Plan:
    """Handle of a cached task plan (released when collected)."""

    def __init__(self, handle):
        self.handle = handle
        info = PlanInfo()
        _check(lib().cprune_plan_query(handle, byref(info)), "cprune_plan_query")
        self.info = info.as_dict()

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.cprune_plan_release(self.handle)
        except Exception:
            pass

    def __getattr__(self, name):
        info = self.__dict__.get("info", {})
        if name in info:
            return info[name]
        raise AttributeError(name)


def cprune_task_plan(N, C, H, W, K, R, S, stride, pad, groups=1, activation="relu", residual=False, pool=None,
                     kernel="auto", flags=()) -> Plan:
    fl = 0
    for f in flags:
        fl |= FLAGS[f]
    opts = TaskOpts(ACT[activation], 1 if residual else 0, POOL[pool], KERNEL[kernel], fl)
    h = c_void_p()
    _check(lib().cprune_task_plan(N, C, H, W, K, R, S, stride, pad, groups, byref(opts), byref(h)), "cprune_task_plan")
    return Plan(h)


def cprune_prune_step(plan: Plan) -> int:
    step = c_int()
    _check(lib().cprune_prune_step(plan.handle, byref(step)), "cprune_prune_step")
    return step.value


def cprune_task_estimate(plan: Plan, k_new: int) -> float:
    us = c_double()
    _check(lib().cprune_task_estimate(plan.handle, int(k_new), byref(us)), "cprune_task_estimate")
    return us.value


def cprune_task_order(times, counts):
    n = len(times)
    assert len(counts) == n
    t = (c_double * max(n, 1))(*[float(v) for v in times])
    c = (c_int * max(n, 1))(*[int(v) for v in counts])
    o = (c_int * max(n, 1))()
    _check(lib().cprune_task_order(t, c, n, o), "cprune_task_order")
    return [o[j] for j in range(n)]


def cprune_cache_stats():
    n, hits = c_int(), c_longlong()
    _check(lib().cprune_cache_stats(byref(n), byref(hits)), "cprune_cache_stats")
    return n.value, hits.value


def cprune_cache_clear() -> int:
    n = c_int()
    _check(lib().cprune_cache_clear(byref(n)), "cprune_cache_clear")
    return n.value


def cprune_pack_weights(plan: Plan, w, b=None, stream=None):
    w = _dev_f32(w)
    wp = torch.empty(plan.packed_weight_bytes // 2, dtype=torch.bfloat16, device=w.device)
    bp = torch.empty(plan.packed_bias_bytes // 4, dtype=torch.float32, device=w.device)
    _check(lib().cprune_pack_weights(plan.handle, _ptr(w), _ptr(b), _ptr(wp), _ptr(bp), _stream(stream)),
           "cprune_pack_weights")
    return wp, bp


def cprune_task_run(plan: Plan, x, w_packed, b_packed, residual=None, y=None, workspace=None, stream=None):
    """x bf16 [N,H,W,c_pad] -> y bf16 [N,out_h,out_w,k_pad]."""
    if y is None:
        y = torch.empty((plan.N, plan.out_h, plan.out_w, plan.k_pad), dtype=torch.bfloat16, device=x.device)
    if workspace is None and plan.workspace_bytes:
        workspace = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=x.device)
    _check(lib().cprune_task_run(plan.handle, _ptr(x), _ptr(w_packed), _ptr(b_packed), _ptr(residual), _ptr(y),
                                 _ptr(workspace), _stream(stream)), "cprune_task_run")
    return y


class Block:
    """Handle of a cached fused-block plan (released when collected)."""

    def __init__(self, handle):
        self.handle = handle
        info = BlockInfo()
        _check(lib().cprune_block_query(handle, byref(info)), "cprune_block_query")
        self.info = {n: getattr(info, n) for n, _ in info._fields_}

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.cprune_block_release(self.handle)
        except Exception:
            pass

    def __getattr__(self, name):
        info = self.__dict__.get("info", {})
        if name in info:
            return info[name]
        raise AttributeError(name)


def cprune_block_plan(N, C_in, H, W, hidden, C_out, activation="relu6", act_out="none", residual=False) -> Block:
    h = c_void_p()
    _check(lib().cprune_block_plan(N, C_in, H, W, hidden, C_out, ACT[activation], ACT[act_out], 1 if residual else 0, byref(h)),
           "cprune_block_plan")
    return Block(h)


def cprune_block_pack(block: Block, w_expand, b_expand, w_depthwise, b_depthwise, w_project, b_project, stream=None):
    dev = w_expand.device
    wp = torch.empty(block.packed_weight_bytes // 2, dtype=torch.bfloat16, device=dev)
    bp = torch.empty(block.packed_bias_bytes // 4, dtype=torch.float32, device=dev)
    _check(lib().cprune_block_pack(block.handle, _ptr(_dev_f32(w_expand)), _ptr(b_expand), _ptr(_dev_f32(w_depthwise)),
                                   _ptr(b_depthwise), _ptr(_dev_f32(w_project)), _ptr(b_project), _ptr(wp), _ptr(bp),
                                   _stream(stream)), "cprune_block_pack")
    return wp, bp


def cprune_block_run(block: Block, x, w_packed, b_packed, y=None, workspace=None, stream=None):
    """x bf16 [N,H,W,c_in_pad] -> y bf16 [N,H,W,k_pad]."""
    if y is None:
        y = torch.empty((block.N, block.H, block.W, block.k_pad), dtype=torch.bfloat16, device=x.device)
    if workspace is None and block.workspace_bytes:
        workspace = torch.empty(block.workspace_bytes, dtype=torch.uint8, device=x.device)
    _check(lib().cprune_block_run(block.handle, _ptr(x), _ptr(w_packed), _ptr(b_packed), _ptr(y), _ptr(workspace), _stream(stream)),
           "cprune_block_run")
    return y


def cprune_cast_input(x, y=None, stream=None):
    """float32 [N,H,W,C] -> bf16 [N,H,W,c_pad]."""
    x = _dev_f32(x)
    C = x.shape[-1]
    if y is None:
        y = torch.empty(tuple(x.shape[:-1]) + (cprune_padded_channels(C),), dtype=torch.bfloat16, device=x.device)
    _check(lib().cprune_cast_input(_ptr(x), x.numel() // C, C, _ptr(y), _stream(stream)), "cprune_cast_input")
    return y


def cprune_widen_output(x, stream=None):
    y = torch.empty(x.shape, dtype=torch.float32, device=x.device)
    _check(lib().cprune_widen_output(_ptr(x), x.numel(), _ptr(y), _stream(stream)), "cprune_widen_output")
    return y


def cprune_maxpool(x, C, k, stride, pad, stream=None):
    N, H, W, cp = x.shape
    P, Q = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    y = torch.empty((N, P, Q, cp), dtype=torch.bfloat16, device=x.device)
    _check(lib().cprune_maxpool(_ptr(x), N, H, W, C, k, stride, pad, _ptr(y), _stream(stream)), "cprune_maxpool")
    return y


def cprune_global_avgpool(x, C, stream=None):
    N, H, W, cp = x.shape
    y = torch.empty((N, cp), dtype=torch.bfloat16, device=x.device)
    _check(lib().cprune_global_avgpool(_ptr(x), N, H, W, C, _ptr(y), _stream(stream)), "cprune_global_avgpool")
    return y


def cprune_fc_pack(w, b=None, stream=None):
    w = _dev_f32(w)
    out, inn = w.shape
    wp = torch.empty((cprune_padded_channels(out), cprune_padded_channels(inn)), dtype=torch.bfloat16, device=w.device)
    bp = torch.empty(cprune_padded_channels(out), dtype=torch.float32, device=w.device)
    _check(lib().cprune_fc_pack(_ptr(w), _ptr(b), out, inn, _ptr(wp), _ptr(bp), _stream(stream)), "cprune_fc_pack")
    return wp, bp


def cprune_fc(x, in_features, w_packed, b_packed, out_features, activation="none", out_f32=False, stream=None):
    N = x.shape[0]
    if out_f32:
        y = torch.empty((N, out_features), dtype=torch.float32, device=x.device)
    else:
        y = torch.empty((N, cprune_padded_channels(out_features)), dtype=torch.bfloat16, device=x.device)
    _check(lib().cprune_fc(_ptr(x), N, in_features, _ptr(w_packed), _ptr(b_packed), out_features, ACT[activation],
                           1 if out_f32 else 0, _ptr(y), _stream(stream)), "cprune_fc")
    return y


class Model:
    """Handle of a cprune_model; keeps the plans and packed weights it borrows alive."""

    def __init__(self, handle, keep_alive, N, classes):
        self.handle, self._keep, self.N, self.classes = handle, keep_alive, N, classes

    @property
    def launches(self):
        return lib().cprune_model_launches(self.handle)

    def tensor(self, tid):
        """bf16 view [n, h, w, c_pad] of an activation buffer (for tests)."""
        p, n, h, w, c = c_void_p(), c_int(), c_int(), c_int(), c_int()
        _check(lib().cprune_model_tensor(self.handle, tid, byref(p), byref(n), byref(h), byref(w), byref(c)),
               "cprune_model_tensor")
        return p.value, (n.value, h.value, w.value, c.value)

    def copy_tensor(self, tid, stream=None):
        """A bf16 copy [n, h, w, c_pad] of an activation buffer."""
        _, shape = self.tensor(tid)
        dev = torch.device("cuda", torch.cuda.current_device())
        out = torch.empty(shape, dtype=torch.bfloat16, device=dev)
        _check(lib().cprune_model_copy_tensor(self.handle, tid, _ptr(out), _stream(stream)), "cprune_model_copy_tensor")
        return out

    def task_table(self):
        """[(plan handle value, count, first task index)] of the model's distinct conv tasks."""
        n = c_int()
        _check(lib().cprune_model_task_table(self.handle, None, 0, byref(n)), "cprune_model_task_table")
        arr = (TaskEntry * max(n.value, 1))()
        _check(lib().cprune_model_task_table(self.handle, arr, n.value, byref(n)), "cprune_model_task_table")
        return [(arr[j].plan, arr[j].count, arr[j].first_task) for j in range(n.value)]

    def time_tasks(self, reps=5, stream=None):
        """Milliseconds per run of every entry of the task table (blocks)."""
        n = len(self.task_table())
        ms = (c_double * max(n, 1))()
        _check(lib().cprune_model_time_tasks(self.handle, int(reps), ms, _stream(stream)), "cprune_model_time_tasks")
        return [ms[j] for j in range(n)]

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.cprune_model_destroy(self.handle)
                self.handle = None
        except Exception:
            pass


def cprune_model_create(N, H, W, C, tasks, keep_alive=None) -> Model:
    """tasks: list of TaskDesc."""
    arr = (TaskDesc * len(tasks))(*tasks)
    h = c_void_p()
    _check(lib().cprune_model_create(N, H, W, C, arr, len(tasks), byref(h)), "cprune_model_create")
    return Model(h, (keep_alive, arr), N, tasks[-1].p1)


def cprune_model_run(model: Model, x, logits=None, use_graph=False, stream=None):
    """x float32 [N,H,W,C] on the device -> logits float32 [N, classes]."""
    x = _dev_f32(x)
    if logits is None:
        logits = torch.empty((model.N, model.classes), dtype=torch.float32, device=x.device)
    _check(lib().cprune_model_run(model.handle, _ptr(x), _ptr(logits), 1 if use_graph else 0, _stream(stream)),
           "cprune_model_run")
    return logits


def cprune_model_run_host(model: Model, x_host, logits_host, stream=None):
    """x_host float32 [N,H,W,C] and logits_host float32 [N, classes] are HOST tensors (pinned for async
    copies).  Returns immediately; synchronise the stream before reading logits_host."""
    assert not x_host.is_cuda and not logits_host.is_cuda and x_host.dtype == torch.float32
    assert x_host.is_contiguous() and logits_host.is_contiguous() and logits_host.dtype == torch.float32
    _check(lib().cprune_model_run_host(model.handle, _ptr(x_host), _ptr(logits_host), _stream(stream)),
           "cprune_model_run_host")
    return logits_host


def cprune_poll_device_status(stream=None):
    _check(lib().cprune_poll_device_status(_stream(stream)), "cprune_poll_device_status")


def cprune_selftest_wait_timeout(stream=None):
    _check(lib().cprune_selftest_wait_timeout(_stream(stream)), "cprune_selftest_wait_timeout")


__all__ = [n for n in dir() if n.startswith("cprune_")] + ["Plan", "Model", "TaskDesc", "CpruneError", "lib",
                                                           "EXPORTS", "KERNEL_NAMES", "OP_CONV", "OP_MAXPOOL",
                                                           "OP_GAP", "OP_FC", "OP_BLOCK", "Block"]

"""Builds and runs a whole pruned network through the C ABI.

Given a layer table (see ``workloads``) and the full-width float32 parameters, this module
  1. uploads the parameters,
  2. prunes every layer that has a keep count with ``cprune_select_filters`` and slices all of its
     consumers with the gather calls (paper Sec. 3.5: L1-norm ranking, then the next layer's input
     channels follow),
  3. plans and packs every conv task, packs the FC layers,
  4. assembles the task list and creates a ``cprune_model``.
It only sequences library calls and keeps device buffers alive; all arithmetic runs in the kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class PrunedNetwork:
    # Largest batch at which inverted-residual blocks run as the fused kernel by default.  A fused block is a chain of
    # short dependent phases on one thread block per image (and hidden-channel slice): it wins where the three separate
    # tasks are bound by launch and fill latency and loses once they are bound by bandwidth.  Measured on pruned
    # MobileNetV2 (ms per batch, separate / fused): batch 1 0.313 / 0.298, 4 0.348 / 0.317, 16 0.429 / 0.395,
    # 32 0.507 / 0.520, 64 0.702 / 0.779.
    FUSE_BLOCKS_MAX_BATCH = 16

    def __init__(self, table: dict, weights: dict, batch: int, device="cuda:0", kernel="auto", fuse_pool=True, fuse_blocks="auto"):
        self.table, self.batch, self.device = table, batch, torch.device(device)
        self.kernel = kernel
        self.fuse_pool = fuse_pool
        if fuse_blocks == "auto":
            fuse_blocks = batch <= self.FUSE_BLOCKS_MAX_BATCH
        self.fuse_blocks = bool(fuse_blocks) and kernel == "auto"
        self.params = {k: (torch.from_numpy(np.ascontiguousarray(w)).to(self.device),
                           torch.from_numpy(np.ascontiguousarray(b)).to(self.device)) for k, (w, b) in weights.items()}
        self.kept = {}
        self._by = {l["name"]: l for l in table["layers"]}
        self._prune()
        self._assemble()

    # ---------------------------------------------------------------- pruning
    def _follow(self, layer, kept, first_done):
        """Slice the consumers of `layer` by `kept`; the first consumer was already handled by
        cprune_select_filters itself when first_done is set."""
        for i, (cname, how) in enumerate(layer["consumers"]):
            w, b = self.params[cname]
            if how in ("in_channels", "fc_in"):
                if not (first_done and i == 0):
                    self.params[cname] = (B.cprune_gather_columns(w, kept), b)
            elif how == "depthwise":
                if not (first_done and i == 0):
                    w = B.cprune_gather_rows(w, kept)
                    self.params[cname] = (w, b)
                self.params[cname] = (self.params[cname][0], B.cprune_gather_rows(b, kept))
                self._follow(self._by[cname], kept, False)
            else:
                raise ValueError(how)

    def _prune(self):
        # layers whose outputs meet in a residual add carry a common ``share`` tag: one ranking over the whole group,
        # taken on the weights as given (before any slicing), and every member loses the same filters
        shared = {}
        for l in self.table["layers"]:
            tag = l.get("share") if l["kind"] == "conv" else None
            if tag is not None and l["keep"] is not None and tag not in shared:
                members = [m for m in self.table["layers"] if m["kind"] == "conv" and m.get("share") == tag]
                shared[tag] = B.cprune_select_shared([self.params[m["name"]][0] for m in members], l["keep"])
        for l in self.table["layers"]:
            if l["kind"] != "conv" or l["keep"] is None:
                continue
            w, b = self.params[l["name"]]
            if l.get("share") is not None:
                kept = shared[l["share"]]
                self.params[l["name"]] = (B.cprune_gather_rows(w, kept), B.cprune_gather_rows(b, kept))
                self.kept[l["name"]] = kept
                self._follow(l, kept, False)
                continue
            w_next, dw = None, False
            if l["consumers"]:
                cname, how = l["consumers"][0]
                w_next = self.params[cname][0]
                dw = how == "depthwise"
                if how == "fc_in":
                    w_next = w_next.reshape(w_next.shape[0], w_next.shape[1], 1, 1)
            kept, w_out, b_out, wn_out = B.cprune_select_filters(w, l["keep"], b, w_next, dw)
            self.params[l["name"]] = (w_out, b_out)
            self.kept[l["name"]] = kept
            if l["consumers"]:
                cname, how = l["consumers"][0]
                if how == "fc_in":
                    wn_out = wn_out.reshape(wn_out.shape[0], wn_out.shape[1])
                self.params[cname] = (wn_out, self.params[cname][1])
            self._follow(l, kept, True)

    # ---------------------------------------------------------------- assembly
    def _assemble(self):
        H, W, C = self.table["input"]
        ids = {"x": 0}
        shape = {"x": (H, W, C)}
        self.plans, self.packed, tasks = {}, {}, []

        def tid(name):
            if name not in ids:
                ids[name] = len(ids)
            return ids[name]

        # A 3x3 stride-2 pad-1 max-pool that is the only reader of a conv task's output becomes that task's pool
        # option: the unpooled tensor is then never stored.
        layers = self.table["layers"]
        readers = {}
        for l in layers:
            for key in ("in", "res"):
                if l.get(key) is not None:
                    readers.setdefault(l[key], []).append(l["name"])
        fused = {}      # conv name -> the pool layer it absorbs
        if self.fuse_pool:
            for a, b in zip(layers, layers[1:]):
                if (a["kind"] == "conv" and b["kind"] == "maxpool" and b["in"] == a["out"] and a.get("pool") is None
                        and a.get("res") is None and (b["k"], b["stride"], b["pad"]) == (3, 2, 1)
                        and readers.get(a["out"]) == [b["name"]]):
                    fused[a["name"]] = b
        absorbed = {b["name"] for b in fused.values()}
        self.fused_pools, self.absorbed = fused, absorbed

        # An inverted-residual block (1x1 expand, 3x3 stride-1 depthwise, 1x1 project, the block's input as residual)
        # whose intermediate tensors have no other reader runs as one fused kernel where the library supports the shape.
        self.blocks, block_of = {}, {}       # expand layer name -> (Block, dw layer, project layer)
        if self.fuse_blocks:
            for e, d, pr in zip(layers, layers[1:], layers[2:]):
                if not (e["kind"] == d["kind"] == pr["kind"] == "conv"):
                    continue
                if not (e["R"] == 1 and e["stride"] == 1 and e["groups"] == 1 and e.get("res") is None and e.get("pool") is None
                        and d["groups"] > 1 and d["R"] == 3 and d["stride"] == 1 and d["pad"] == 1 and d["in"] == e["out"]
                        and d.get("res") is None and d["act"] == e["act"]
                        and pr["R"] == 1 and pr["stride"] == 1 and pr["groups"] == 1 and pr["in"] == d["out"] and pr.get("pool") is None
                        and pr.get("res") in (None, e["in"])
                        and readers.get(e["out"]) == [d["name"]] and readers.get(d["out"]) == [pr["name"]]):
                    continue
                block_of[e["name"]] = (d, pr)
        skip = set()

        for l in self.table["layers"]:
            kind = l["kind"]
            if l["name"] in absorbed or l["name"] in skip:
                continue
            h, w, c = shape[l["in"]]
            if l["name"] in block_of:
                dl, pl = block_of[l["name"]]
                (we, be), (wd, bd), (wpj, bpj) = self.params[l["name"]], self.params[dl["name"]], self.params[pl["name"]]
                try:
                    blk = B.cprune_block_plan(self.batch, c, h, w, we.shape[0], wpj.shape[0], l["act"], pl["act"], pl.get("res") is not None)
                except B.CpruneError as err:
                    if err.status != 2:          # anything but "unsupported shape" is a real error
                        raise
                    blk = None
                if blk is not None:
                    wq, bq = B.cprune_block_pack(blk, we.reshape(we.shape[0], -1), be, wd.reshape(wd.shape[0], -1), bd,
                                                 wpj.reshape(wpj.shape[0], -1), bpj)
                    self.blocks[l["name"]] = blk
                    self.packed[l["name"]] = (wq, bq)
                    d = B.TaskDesc()
                    d.op, d.in_, d.out, d.res = B.OP_BLOCK, tid(l["in"]), tid(pl["out"]), -1
                    d.block, d.w, d.b = blk.handle, wq.data_ptr(), bq.data_ptr()
                    shape[pl["out"]] = (h, w, wpj.shape[0])
                    skip.update((dl["name"], pl["name"]))
                    tasks.append(d)
                    continue
            if kind == "flatten":
                ids[l["out"]] = ids[l["in"]]
                shape[l["out"]] = shape[l["in"]]
                continue
            d = B.TaskDesc()
            out_name = fused[l["name"]]["out"] if l["name"] in fused else l["out"]
            d.in_, d.out, d.res = tid(l["in"]), tid(out_name), -1
            if kind == "conv":
                wt, bs = self.params[l["name"]]
                K, cg = wt.shape[0], wt.shape[1]
                groups = K if l["groups"] > 1 else 1
                assert cg * groups == c, (l["name"], cg, groups, c)
                plan = B.cprune_task_plan(self.batch, c, h, w, K, l["R"], l["S"], l["stride"], l["pad"], groups,
                                          l["act"], l.get("res") is not None,
                                          "max3x3s2" if l["name"] in fused else l.get("pool"),
                                          self.kernel if groups == 1 else "auto")
                wp, bp = B.cprune_pack_weights(plan, wt, bs)
                self.plans[l["name"]], self.packed[l["name"]] = plan, (wp, bp)
                d.op, d.plan, d.w, d.b = B.OP_CONV, plan.handle, wp.data_ptr(), bp.data_ptr()
                if l.get("res") is not None:
                    d.res = tid(l["res"])
                shape[out_name] = (plan.out_h, plan.out_w, K)
            elif kind == "maxpool":
                d.op, d.p0, d.p1, d.p2 = B.OP_MAXPOOL, l["k"], l["stride"], l["pad"]
                shape[l["out"]] = ((h + 2 * l["pad"] - l["k"]) // l["stride"] + 1,
                                   (w + 2 * l["pad"] - l["k"]) // l["stride"] + 1, c)
            elif kind == "gap":
                d.op = B.OP_GAP
                shape[l["out"]] = (1, 1, c)
            elif kind == "fc":
                wt, bs = self.params[l["name"]]
                wp, bp = B.cprune_fc_pack(wt, bs)
                self.packed[l["name"]] = (wp, bp)
                d.op, d.w, d.b = B.OP_FC, wp.data_ptr(), bp.data_ptr()
                d.p0, d.p1, d.p2 = wt.shape[1], wt.shape[0], B.ACT[l["act"]]
                shape[l["out"]] = (1, 1, wt.shape[0])
            else:
                raise ValueError(kind)
            tasks.append(d)
        self.tensor_ids, self.shapes = ids, shape
        self.model = B.cprune_model_create(self.batch, H, W, C, tasks, keep_alive=(self.plans, self.packed))
        torch.cuda.synchronize(self.device)

    # ---------------------------------------------------------------- running
    def run(self, x, logits=None, use_graph=False):
        """x: float32 [batch, H, W, C] device tensor -> float32 logits [batch, classes]."""
        return B.cprune_model_run(self.model, x, logits, use_graph)

    def run_host(self, x_host, logits_host):
        """Host buffers in and out (see cprune_model_run_host); asynchronous."""
        return B.cprune_model_run_host(self.model, x_host, logits_host)

    def activation(self, name):
        """Copy of a stored activation as float32 numpy [N, h, w, c] without the pad lanes."""
        c = self.shapes[name][2]
        buf = self.model.copy_tensor(self.tensor_ids[name])
        torch.cuda.synchronize(self.device)
        return buf.float().cpu().numpy()[..., :c]

    def task_priorities(self, reps=5):
        """The model's tasks in the order the paper tries them for pruning (Sec. 3.3, 3.4): every distinct plan with
        the layers (subgraphs) that share it, its measured time and its pruning impact = time x subgraphs, sorted by
        impact.  The table comes from cprune_model_task_table, the times from cprune_model_time_tasks, the order from
        cprune_task_order."""
        table = self.model.task_table()
        ms = self.model.time_tasks(reps)
        by_handle = {}
        for name, plan in self.plans.items():
            by_handle.setdefault(plan.handle.value, []).append(name)
        order = B.cprune_task_order(ms, [c for _, c, _ in table])
        return [{"plan": self.plans[by_handle[table[j][0]][0]], "layers": by_handle[table[j][0]], "count": table[j][1],
                 "ms": ms[j], "impact": ms[j] * table[j][1]} for j in order]

    def flops(self):
        return sum(p.flops for p in self.plans.values()) + sum(b.flops for b in self.blocks.values())

    def conv_launch_info(self):
        return {k: p.info for k, p in self.plans.items()}

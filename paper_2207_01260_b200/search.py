"""The latency-gated half of the paper's pruning loop (Algorithm 1, steps 3 to 10), without training.

One iteration: take the tasks in order of pruning impact (Sec. 3.3); for the first one, look up the subgraphs
(layers) that share it and its program (the plan) in the task table (Sec. 3.4); derive the number of filters to
prune from the structure of that program (``cprune_prune_step``, Sec. 3.5); prune those layers by that many
filters to get a candidate model; build it (selection, slicing, planning, packing) and measure its execution
time; accept the candidate if it is faster than the target time, otherwise go on to the next task.  The paper
then trains the candidate briefly and checks its accuracy (steps 11 and 12); there are no datasets here, so
that gate is left to the caller (``accept`` callback).

This module only sequences library calls and edits keep counts in a layer table; all arithmetic (norms,
ranking, slicing, convolution, timing on the device) happens behind the C ABI.
"""
from __future__ import annotations

import copy

import torch

from . import binding as B
from .pipeline import PrunedNetwork


def measure_ms(net: PrunedNetwork, x, steps: int = 10, warmup: int = 3) -> float:
    """Mean milliseconds of one pass of the model (CUDA-graph replay, CUDA events on the launching stream)."""
    logits = torch.empty((net.batch, net.model.classes), dtype=torch.float32, device=x.device)
    for _ in range(warmup):
        net.run(x, logits, True)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        net.run(x, logits, True)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def prunable(layer: dict) -> bool:
    """A layer can lose filters when the table says who consumes its output channels and it is not tied to a
    shortcut group (those are pruned as a whole group, not one task at a time)."""
    return layer["kind"] == "conv" and bool(layer["consumers"]) and layer.get("share") is None


def candidate_table(table: dict, layer_names, step: int, current_widths: dict):
    """A copy of `table` in which the named layers keep `step` fewer filters than they have now; None if any of
    them would be left without filters."""
    cand = copy.deepcopy(table)
    by = {l["name"]: l for l in cand["layers"]}
    for name in layer_names:
        keep = current_widths[name] - step
        if keep < 1:
            return None
        by[name]["keep"] = keep
    return cand


def latency_gated_iteration(table: dict, weights: dict, batch: int, x, target_ms: float | None = None, beta: float = 0.98,
                            build=PrunedNetwork, measure=measure_ms, accept=None, reps: int = 5):
    """One pass over the prioritised task list.  Returns a dict: ``accepted`` (bool), ``table`` (the accepted candidate
    table, or the input table), ``net`` (its built network), ``ms`` (its time), ``base_ms``, ``target_ms`` and
    ``tried``: one record per task tried, with the task's layers, its step and the candidate's time."""
    base = build(table, weights, batch)
    base_ms = measure(base, x)
    if target_ms is None:
        target_ms = beta * base_ms
    tried = []
    for task in base.task_priorities(reps):
        names = [n for n in task["layers"] if prunable(base._by[n])]
        rec = {"layers": task["layers"], "impact": task["impact"], "ms": task["ms"], "step": None, "candidate_ms": None}
        tried.append(rec)
        if not names:
            continue
        step = B.cprune_prune_step(task["plan"])
        rec["step"] = step
        widths = {n: base.plans[n].K for n in names}
        cand = candidate_table(table, names, step, widths)
        if cand is None:
            continue
        net = build(cand, weights, batch)
        ms = measure(net, x)
        rec["candidate_ms"] = ms
        rec["pruned"] = names
        if ms < target_ms and (accept is None or accept(cand, net)):
            return {"accepted": True, "table": cand, "net": net, "ms": ms, "base_ms": base_ms, "target_ms": target_ms,
                    "tried": tried}
    return {"accepted": False, "table": table, "net": base, "ms": base_ms, "base_ms": base_ms, "target_ms": target_ms,
            "tried": tried}

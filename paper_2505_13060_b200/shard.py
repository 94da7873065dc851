"""Layer-sharded scoring over several GPUs (one process per GPU).

Every (layer, operand) of the sensitivity pass is independent up to the
per-layer values (Sec. 2.2), so the path shards by layer with no collective in
the data path: each rank scores its own layers with its own ``Context`` and
only the per-layer table (a few doubles per layer) is exchanged before the
sub-graph sums and the selection (Sec. 2.1), which every rank then runs on the
same table.  The exchange is one ``all_reduce(SUM)`` of a dense ``[L, K]``
float64 table in which a rank fills only its own rows: every row has exactly
one non-zero contributor, and adding zeros is exact, so all ranks end up with
bit-identical tables.  Works with the ``nccl`` backend (device tensors) and
with ``gloo`` (host tensors).
"""
from __future__ import annotations

import numpy as np


def assign_layers(cost_per_layer, world: int) -> np.ndarray:
    """Rank of every layer: largest cost first onto the least-loaded rank
    (ties: lower rank, then lower layer index).  Deterministic, so every rank
    computes the same assignment without talking."""
    cost = np.asarray(cost_per_layer, dtype=np.float64)
    if world < 1:
        raise ValueError("world must be at least 1")
    order = sorted(range(len(cost)), key=lambda i: (-cost[i], i))
    load = [0.0] * world
    owner = np.zeros(len(cost), dtype=np.int32)
    for i in order:
        r = min(range(world), key=lambda k: (load[k], k))
        owner[i] = r
        load[r] += float(cost[i])
    return owner


def layer_row(res: dict, F: int) -> np.ndarray:
    """One row of the exchanged table from ``Context.get_layer``:
    [s_mean, d_model[0..F-1], d_meas[0..F-1]]."""
    return np.concatenate([[res["s_mean"]], np.asarray(res["d_model"], np.float64)[:F],
                           np.asarray(res["d_meas"], np.float64)[:F]])


def gather_layer_table(local_rows: dict, L: int, F: int, group=None, device=None) -> np.ndarray:
    """``local_rows``: {global layer index: row from ``layer_row``} of the layers
    this rank scored.  Returns the full [L, 1 + 2F] table on every rank."""
    import torch
    import torch.distributed as dist

    K = 1 + 2 * F
    table = np.zeros((L, K), dtype=np.float64)
    for i, row in local_rows.items():
        table[i] = row
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        t = torch.from_numpy(table)
        if device is not None:
            t = t.to(device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        table = t.cpu().numpy()
    return table


def select_from_table(binding, table: np.ndarray, F: int, groups, d_mode: int, budget: float):
    """Sub-graph sums and the selection on a gathered table.  ``groups`` is a
    list of (layer indices, Q[Lj, Pj], c[Pj]).  Returns (p, c_total, d_total) or
    None when no assignment meets the budget."""
    col0 = 1 if d_mode == binding.D_MODEL else 1 + F
    d_layer = np.ascontiguousarray(table[:, col0:col0 + F])
    c_tabs, d_tabs = [], []
    for layer_ids, Q, c in groups:
        c_tabs.append(np.asarray(c, dtype=np.float64))
        d_tabs.append(binding.group_costs_table(layer_ids, Q, d_layer))
    return binding.select_tables(c_tabs, d_tabs, budget)


# ---------------------------------------------------------------------------
# Sample-sharded calibration: every rank holds the same layers but only its own
# calibration samples.  Two small exchanges: the per-tensor amax (MAX) between
# the amax pass and the scoring pass, and the per-layer rows (a mean over all
# samples, Sec. 2.2) afterwards.

def reduce_amax(local_amax, group=None, device=None) -> np.ndarray:
    """``local_amax``: [L, 2] float32 from ``Context.get_amax`` on this rank's
    samples.  Returns the element-wise maximum over all ranks (exact)."""
    import torch
    import torch.distributed as dist

    a = np.ascontiguousarray(local_amax, dtype=np.float32)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        t = torch.from_numpy(a.copy())
        if device is not None:
            t = t.to(device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        a = t.cpu().numpy()
    return a


def merge_sample_rows(binding, local_table, R_local: int, group=None, device=None) -> np.ndarray:
    """``local_table``: [L, 1 + 2F] rows (``layer_row``) computed over this rank's
    ``R_local`` samples.  The tables and sample counts of all ranks are gathered
    (a few KB) and ``ampq_merge_sample_tables`` forms the table over all samples
    on every rank, from the same inputs in the same order: bit-identical."""
    import torch
    import torch.distributed as dist

    tab = np.ascontiguousarray(local_table, dtype=np.float64)
    if not (dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1):
        return binding.merge_sample_tables(tab[None], [R_local])
    world = dist.get_world_size(group)
    mine = torch.from_numpy(np.concatenate([tab.reshape(-1), [float(R_local)]]))
    if device is not None:
        mine = mine.to(device)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    parts = [p.cpu().numpy() for p in parts]
    tables = np.stack([p[:-1].reshape(tab.shape) for p in parts])
    return binding.merge_sample_tables(tables, [int(p[-1]) for p in parts])

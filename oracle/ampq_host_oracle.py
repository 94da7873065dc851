"""Plain-Python oracle of the host-side steps around the sensitivity pass.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests import this module; it
shares nothing with the library.  Small inputs only (pure-Python loops).

  * partition(...)        the sequential sub-graphs of a model DAG (Appendix B,
                          Algorithm 2) from their definition: a start vertex is
                          added in front of every source; a vertex is a
                          separator when every start -> end path runs through
                          it (tested by deleting it and searching); the
                          separators are totally ordered along every path, and
                          vertex u belongs to the sub-graph that ends at the
                          first separator u reaches (u itself if it is one).
                          Non-quantisable vertices are dropped and empty groups
                          skipped, as the algorithm's last steps do.
  * gain_table(...)       c_{j,p} = sum_l c_{l, Q_j[l,p]} with the per-layer
                          theoretical time gain N C K delta_T,f (linear) /
                          N C^2 delta_T,f (BGEMM) of Sec. 2.3.2, or the memory
                          gain C K delta_M,f (linear) / 0 (BGEMM) of Sec. 2.3.3.
  * select_in_order(...)  the two baseline strategies of Sec. 3.1: units are
                          switched to low precision one after the other in a
                          given order while the loss-MSE budget holds, stopping
                          at the first that does not fit.  Prefix = the model's
                          own order; Random = a permutation the caller draws.
  * merge_sample_tables(...)  per-layer means over all calibration samples from
                          per-process means over disjoint sample sets (Sec. 2.2:
                          s_l = (1/R) sum_r s_l^r): the R-weighted mean.
"""
from __future__ import annotations

LINEAR, BGEMM = 0, 1
GAIN_MAC, GAIN_MEMORY = 0, 1


def _reach(succ, src, banned=None):
    seen, stack = set(), [src]
    while stack:
        v = stack.pop()
        if v in seen or v == banned:
            continue
        seen.add(v)
        stack.extend(succ[v])
    return seen


def partition(n, edges, quantisable):
    """Returns group_of[n] (-1 for vertices in no group) and the number of groups.
    Vertices 0..n-1, edges (u, v); the graph must be acyclic with one sink."""
    succ = {v: [] for v in range(n)}
    indeg = [0] * n
    for u, v in edges:
        succ[u].append(v)
        indeg[v] += 1
    sinks = [v for v in range(n) if not succ[v]]
    if len(sinks) != 1:
        raise ValueError("the graph needs exactly one sink")
    end, start = sinks[0], n
    succ[start] = [v for v in range(n) if indeg[v] == 0]
    # separators: deleting the vertex cuts start from end
    seps = [v for v in range(n) if v == end or end not in _reach(succ, start, banned=v)]
    # order them along the paths: a reaches b  <=>  a comes first
    sepset = set(seps)
    seps.sort(key=lambda v: -len(_reach(succ, v) & sepset))
    raw = []
    for u in range(n):
        reach = _reach(succ, u)
        raw.append(next(j for j, s in enumerate(seps) if s in reach))
    group_of, renum = [-1] * n, {}
    for j in range(len(seps)):
        members = [u for u in range(n) if raw[u] == j and quantisable[u]]
        if members:
            renum[j] = len(renum)
            for u in members:
                group_of[u] = renum[j]
    return group_of, len(renum)


def layer_gain(kind, layer_kind, N, C, K, delta_f):
    if kind == GAIN_MAC:
        return (N * C * K if layer_kind == LINEAR else N * C * C) * delta_f
    return (C * K if layer_kind == LINEAR else 0) * delta_f


def gain_table(kind, layers, Q, delta):
    """layers: [(layer_kind, N, C, K)] of the group; Q[l][p]; delta[f].  Returns c[p]."""
    P = len(Q[0])
    out = []
    for p in range(P):
        c = 0.0
        for l, (lk, N, C, K) in enumerate(layers):
            c += float(layer_gain(kind, lk, N, C, K, delta[Q[l][p]]))
        out.append(c)
    return out


def select_in_order(order, d_low, c_low, budget):
    chosen = [0] * len(order)
    d = c = 0.0
    for u in order:
        if d + d_low[u] <= budget:
            d += d_low[u]
            c += c_low[u]
            chosen[u] = 1
        else:
            break
    return chosen, c, d


def merge_sample_tables(tables, R_local):
    """tables[i][l][k]: mean over process i's R_local[i] samples.  Returns the
    mean over all samples, [l][k]."""
    total = float(sum(R_local))
    L, K = len(tables[0]), len(tables[0][0])
    out = [[0.0] * K for _ in range(L)]
    for l in range(L):
        for k in range(K):
            acc = 0.0
            for i, R in enumerate(R_local):
                acc += float(R) * tables[i][l][k]
            out[l][k] = acc / total
    return out

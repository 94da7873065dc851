"""Pins for the plain-Python oracle of the host steps (partition into sequential
sub-graphs, gain tables, baseline strategies)."""
import itertools

import numpy as np
import pytest

from oracle import ampq_host_oracle as ho


def _paths(n, edges):
    """Number of start->v and v->end paths (exact integers); start feeds every source."""
    succ = {v: [] for v in range(n)}
    pred = {v: [] for v in range(n)}
    for u, v in edges:
        succ[u].append(v)
        pred[v].append(u)
    order, indeg = [], {v: len(pred[v]) for v in range(n)}
    ready = [v for v in range(n) if indeg[v] == 0]
    while ready:
        v = ready.pop()
        order.append(v)
        for w in succ[v]:
            indeg[w] -= 1
            if indeg[w] == 0:
                ready.append(w)
    down = {}
    for v in order:
        down[v] = 1 if not pred[v] else sum(down[u] for u in pred[v])
    up = {}
    for v in reversed(order):
        up[v] = 1 if not succ[v] else sum(up[w] for w in succ[v])
    return down, up, order


def llama_layer_graph(residual):
    """One Llama-3 decoder layer plus the LM head as in the paper's figure of
    sequential sub-graphs: norm -> {q,k,v} -> qk_matmul -> softmax -> av_matmul ->
    o_proj [-> add] -> norm -> {gate, up} -> act*mul -> down [-> add] -> lm_head."""
    names = ["in", "norm1", "q", "k", "v", "qk", "softmax", "av", "o", "add1", "norm2", "gate", "up", "mul",
             "down", "add2", "lm_head"]
    ix = {s: i for i, s in enumerate(names)}
    e = [("in", "norm1"), ("norm1", "q"), ("norm1", "k"), ("norm1", "v"), ("q", "qk"), ("k", "qk"), ("qk", "softmax"),
         ("softmax", "av"), ("v", "av"), ("av", "o"), ("o", "add1"), ("add1", "norm2"), ("norm2", "gate"),
         ("norm2", "up"), ("gate", "mul"), ("up", "mul"), ("mul", "down"), ("down", "add2"), ("add2", "lm_head")]
    if residual:
        e += [("in", "add1"), ("add1", "add2")]
    quant = [s in ("q", "k", "v", "qk", "av", "o", "gate", "up", "down", "lm_head") for s in names]
    return names, [(ix[a], ix[b]) for a, b in e], quant


def test_partition_of_a_llama_layer_matches_the_papers_figure():
    names, edges, quant = llama_layer_graph(residual=False)
    g, J = ho.partition(len(names), edges, quant)
    groups = [[names[i] for i in range(len(names)) if g[i] == j] for j in range(J)]
    # V1 = the five attention operations, V2 = o_proj, V3 = gate and up, V4 = down, then the LM head
    assert groups == [["q", "k", "v", "qk", "av"], ["o"], ["gate", "up"], ["down"], ["lm_head"]]
    assert all(g[i] == -1 for i in range(len(names)) if not quant[i])
    # with the residual edges drawn, nothing between a block's input and its add is a separator
    g2, J2 = ho.partition(len(names), *llama_layer_graph(residual=True)[1:])
    groups2 = [[names[i] for i in range(len(names)) if g2[i] == j] for j in range(J2)]
    assert groups2 == [["q", "k", "v", "qk", "av", "o"], ["gate", "up", "down"], ["lm_head"]]


def test_partition_special_cases():
    # a chain: every vertex is its own sub-graph (the J = L case of Sec. 2.1)
    g, J = ho.partition(5, [(i, i + 1) for i in range(4)], [1] * 5)
    assert g == [0, 1, 2, 3, 4] and J == 5
    # non-quantisable vertices leave no empty groups behind
    g, J = ho.partition(5, [(i, i + 1) for i in range(4)], [1, 0, 0, 1, 1])
    assert g == [0, -1, -1, 1, 2] and J == 3
    # a diamond is one sub-graph ending at its merge vertex; two sources merge the same way
    g, J = ho.partition(4, [(0, 1), (0, 2), (1, 3), (2, 3)], [1] * 4)
    assert g == [0, 1, 1, 1] and J == 2
    g, J = ho.partition(3, [(0, 2), (1, 2)], [1] * 3)
    assert g == [0, 0, 0] and J == 1
    with pytest.raises(ValueError):
        ho.partition(3, [(0, 1), (0, 2)], [1] * 3)


def test_partition_separators_against_path_counting():
    """Independent characterisation: v is a separator iff (#paths start->v) x
    (#paths v->end) = #paths start->end.  Groups are the stretches between
    consecutive separators in any topological order."""
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(2, 14))
        edges = set()
        for v in range(1, n):   # every vertex but 0.. gets a predecessor; then every vertex a successor
            for u in rng.choice(v, size=min(v, int(rng.integers(1, 3))), replace=False):
                edges.add((int(u), v))
        for u in range(n - 1):
            if not any(a == u for a, _ in edges):
                edges.add((u, int(rng.integers(u + 1, n))))
        perm = rng.permutation(n)   # vertex numbers carry no order
        edges = sorted((int(perm[a]), int(perm[b])) for a, b in edges)
        g, J = ho.partition(n, edges, [1] * n)
        down, up, order = _paths(n, edges)
        total = sum(up[v] for v in range(n) if down[v] == 1 and not any(b == v for _, b in edges))
        seps = [v for v in order if down[v] * up[v] == total]
        assert J == len(seps)
        pos = {v: i for i, v in enumerate(order)}
        for u in range(n):
            first = next(j for j, s in enumerate(seps) if pos[s] >= pos[u])
            assert g[u] == first, (trial, edges, u)


def test_gain_tables_hand_examples():
    layers = [(ho.LINEAR, 10, 4, 8), (ho.BGEMM, 10, 4, 0), (ho.LINEAR, 10, 8, 2)]
    Q = [[0, 1, 0, 1], [0, 0, 1, 1], [0, 1, 1, 0]]
    # MACs: 320, 160, 160; one unit of gain per MAC in format 1
    assert ho.gain_table(ho.GAIN_MAC, layers, Q, [0.0, 1.0]) == [0.0, 480.0, 320.0, 480.0]
    # memory: weights only, 32 and 16 parameters, one byte saved each; a BGEMM saves nothing
    assert ho.gain_table(ho.GAIN_MEMORY, layers, Q, [0.0, 1.0]) == [0.0, 48.0, 16.0, 32.0]
    # additive across layers: a group's table is the sum of its layers' single-layer tables
    for kind in (ho.GAIN_MAC, ho.GAIN_MEMORY):
        whole = ho.gain_table(kind, layers, Q, [0.0, 0.5, 0.75])
        parts = [ho.gain_table(kind, [layers[l]], [Q[l]], [0.0, 0.5, 0.75]) for l in range(3)]
        assert whole == [sum(p[i] for p in parts) for i in range(4)]


def test_baseline_strategies_hand_examples_and_bound():
    d = [0.3, 0.1, 0.5, 0.05]
    c = [1.0, 2.0, 3.0, 4.0]
    assert ho.select_in_order([0, 1, 2, 3], d, c, 0.45) == ([1, 1, 0, 0], 3.0, 0.4)   # Prefix stops at layer 2
    assert ho.select_in_order([3, 2, 1, 0], d, c, 0.45) == ([0, 0, 0, 1], 4.0, 0.05)   # this order stops at layer 2 too
    assert ho.select_in_order([0, 1, 2, 3], d, c, 0.0) == ([0, 0, 0, 0], 0.0, 0.0)
    assert ho.select_in_order([0, 1, 2, 3], d, c, 10.0)[0] == [1, 1, 1, 1]
    # never better than the exhaustive optimum over subsets, always within the budget
    rng = np.random.default_rng(2)
    for _ in range(50):
        L = int(rng.integers(1, 9))
        d, c = rng.uniform(0, 1, L).tolist(), rng.uniform(0, 1, L).tolist()
        budget = float(rng.uniform(0, sum(d)))
        best = max(sum(c[i] for i in s) for k in range(L + 1) for s in itertools.combinations(range(L), k)
                   if sum(d[i] for i in s) <= budget)
        for order in (list(range(L)), rng.permutation(L).tolist()):
            ch, cs, ds = ho.select_in_order(order, d, c, budget)
            assert ds <= budget and cs <= best + 1e-12


def test_merge_of_sample_means_equals_the_mean_over_all_samples():
    """Pin (Sec. 2.2, s_l = (1/R) sum_r s_l^r): per-sample values with few
    significant bits, so that every sum below is exact in double; the merge of
    the per-shard means over unequal shards (3, 1 and 4 samples) must then equal
    the mean over all 8 samples exactly, computed here with rationals."""
    from fractions import Fraction

    import random

    rnd = random.Random(5)
    L, K, shards = 3, 5, [3, 1, 4]
    per_sample = [[[Fraction(rnd.randrange(0, 1 << 12), 1 << 6) * 24 for _ in range(K)] for _ in range(L)]
                  for _ in range(sum(shards))]   # multiples of 24/64: divisible by 3, 4 and 8 without rounding
    tables, r = [], 0
    for n in shards:
        tables.append([[float(sum(per_sample[r + i][l][k] for i in range(n)) / n) for k in range(K)] for l in range(L)])
        r += n
    want = [[float(sum(s[l][k] for s in per_sample) / len(per_sample)) for k in range(K)] for l in range(L)]
    assert ho.merge_sample_tables(tables, shards) == want
    # one shard is the identity; a shard without samples does not count
    assert ho.merge_sample_tables([tables[0]], [3]) == tables[0]
    assert ho.merge_sample_tables([tables[0], tables[1]], [3, 0]) == tables[0]

"""The library's host steps (no GPU) against the plain-Python oracle: partition
into sequential sub-graphs, gain tables, baseline strategies, and the strategies
against the exact selection."""
import numpy as np
import pytest

from oracle import ampq_host_oracle as ho
from test_oracle_host import llama_layer_graph


def _random_dag(rng, n):
    edges = set()
    for v in range(1, n):
        for u in rng.choice(v, size=min(v, int(rng.integers(1, 4))), replace=False):
            if rng.random() < 0.8 or not any(b == v for _, b in edges):
                edges.add((int(u), v))
    for u in range(n - 1):   # one sink: every vertex but the last gets a successor
        if not any(a == u for a, _ in edges):
            edges.add((u, int(rng.integers(u + 1, n))))
    perm = rng.permutation(n)   # vertex numbers carry no order
    return sorted((int(perm[a]), int(perm[b])) for a, b in edges)


def test_partition_matches_definition_on_random_graphs(ampq):
    rng = np.random.default_rng(11)
    for trial in range(300):
        n = int(rng.integers(1, 40))
        edges = _random_dag(rng, n) if n > 1 else []
        quant = (rng.random(n) < 0.7).astype(np.uint8)
        want, J = ho.partition(n, edges, quant.tolist())
        got, Jg = ampq.partition(n, edges, quant)
        assert Jg == J and got.tolist() == want, (trial, n, edges)


def test_partition_llama_layers_and_errors(ampq):
    names, edges, quant = llama_layer_graph(residual=False)
    got, J = ampq.partition(len(names), edges, quant)
    assert J == 5 and got.tolist() == ho.partition(len(names), edges, quant)[0]
    # a stack of 8 such layers: 4 sub-graphs per layer plus the LM head
    n1 = len(names) - 1   # without the head
    big_edges, big_quant = [], []
    for b in range(8):
        big_edges += [(u + b * n1, v + b * n1) for u, v in edges if v < n1]
        big_quant += quant[:n1]
        if b:
            big_edges.append((b * n1 - 1, b * n1))
    big_edges.append((8 * n1 - 1, 8 * n1))
    big_quant.append(True)
    got, J = ampq.partition(8 * n1 + 1, big_edges, big_quant)
    assert J == 33 and got.tolist() == ho.partition(8 * n1 + 1, big_edges, big_quant)[0]
    L = ampq.lib()
    out = np.zeros(3, np.int32)
    import ctypes as C
    J = C.c_int()
    q = np.ones(3, np.uint8)

    def call(src, dst):
        s, d = np.asarray(src, np.int32), np.asarray(dst, np.int32)
        return L.ampq_partition(3, len(src), s.ctypes.data, d.ctypes.data, q.ctypes.data, out.ctypes.data, C.byref(J))

    assert call([0, 1, 2], [1, 2, 0]) == ampq.ERR_INVALID    # a cycle
    assert call([0, 0], [1, 2]) == ampq.ERR_INVALID          # two sinks
    assert call([0, 1], [1, 5]) == ampq.ERR_INVALID          # vertex out of range
    assert call([0, 1], [1, 2]) == 0 and out.tolist() == [0, 1, 2]


def test_gain_tables_match_oracle(ampq):
    rng = np.random.default_rng(12)
    for _ in range(100):
        Lj, F = int(rng.integers(1, 6)), int(rng.integers(2, 4))
        layers = [(int(rng.integers(0, 2)), int(rng.integers(1, 5000)), int(rng.integers(1, 9000)),
                   int(rng.integers(1, 9000))) for _ in range(Lj)]
        P = int(rng.integers(1, 9))
        Q = rng.integers(0, F, (Lj, P)).astype(np.uint8)
        delta = np.concatenate([[0.0], rng.uniform(0, 1e-9, F - 1)])
        for kind in (ampq.GAIN_MAC, ampq.GAIN_MEMORY):
            assert ampq.gain_table(kind, layers, Q, delta).tolist() == ho.gain_table(kind, layers, Q.tolist(), delta.tolist())
    # the attention group of five operations the paper uses as its example: 2^5 columns
    att = [(0, 2048, 4096, 4096), (0, 2048, 4096, 1024), (0, 2048, 4096, 1024), (1, 2048 * 32, 128, 0), (1, 2048 * 32, 128, 0)]
    Q = np.array([[(p >> l) & 1 for p in range(32)] for l in range(5)], np.uint8)
    c = ampq.gain_table(ampq.GAIN_MAC, att, Q, [0.0, 1.0])
    assert c[0] == 0 and c[31] == sum(ho.layer_gain(0, *l, 1.0) for l in att) and len(set(c.tolist())) > 8


def test_baselines_match_oracle_and_never_beat_the_integer_program(ampq):
    rng = np.random.default_rng(13)
    for trial in range(200):
        L = int(rng.integers(1, 30))
        d = rng.uniform(0, 1, L) ** 2
        c = rng.uniform(0.5, 2.0, L)
        budget = float(rng.choice([0.01, 0.05, 0.2, 0.5])) * float(d.sum())
        exact = ampq.select_tables([[0.0, x] for x in c], [[0.0, x] for x in d], budget)
        for order in (np.arange(L), rng.permutation(L)):
            ch, cs, ds = ampq.select_in_order(order, d, c, budget)
            want = ho.select_in_order(order.tolist(), d.tolist(), c.tolist(), budget)
            assert ch.tolist() == want[0] and cs == want[1] and ds == want[2]
            assert ds <= budget and cs <= exact[1] + 1e-12
    import ctypes as C
    o = np.array([0, 0], np.int32)
    z = np.zeros(2)
    ch = np.zeros(2, np.uint8)
    assert ampq.lib().ampq_select_in_order(2, o.ctypes.data, z.ctypes.data, z.ctypes.data, 1.0, ch.ctypes.data,
                                           None, None) == ampq.ERR_INVALID   # not a permutation


def test_merge_sample_tables_matches_oracle(ampq):
    rng = np.random.default_rng(11)
    for nranks, L, K in ((1, 4, 5), (2, 7, 5), (5, 3, 7)):
        tables = rng.uniform(0, 3, (nranks, L, K)) * 10.0 ** rng.integers(-6, 3, (nranks, L, 1))
        R = rng.integers(1, 9, nranks)
        got = ampq.merge_sample_tables(tables, R)
        assert got.tolist() == ho.merge_sample_tables(tables.tolist(), R.tolist())
    with pytest.raises(ampq.AmpqError):
        ampq.merge_sample_tables(np.zeros((2, 1, 1)), [0, 0])     # no samples at all
    with pytest.raises(ampq.AmpqError):
        ampq.merge_sample_tables(np.zeros((2, 1, 1)), [1, -1])


def test_saved_layer_table_round_trips_bit_for_bit(ampq, tmp_path):
    from paper_2505_13060_b200 import shard, table

    rng = np.random.default_rng(14)
    L, F = 23, 3
    tab = np.concatenate([rng.uniform(0, 1, (L, 1)) ** 8, np.zeros((L, 1)), rng.uniform(0, 1e-3, (L, F - 1)),
                          np.zeros((L, 1)), rng.uniform(0, 1e-3, (L, F - 1))], axis=1)
    tab[3] = [5e-324, 0.0, 1.7976931348623157e308, 1e-300, 0.0, 0.1, 1.0 / 3.0]   # awkward doubles survive too
    names = ["blk%d.fc" % i for i in range(L)]
    path = str(tmp_path / "calib.json")
    table.save_table(path, names, [0, 1, 2], tab, meta={"R": 8})
    n2, f2, t2, meta = table.load_table(path)
    assert n2 == names and f2 == [0, 1, 2] and meta == {"R": 8} and t2.tobytes() == tab.tobytes()
    groups = [([i, i + 1], np.array([[0, 1, 2], [0, 1, 2]], np.uint8), np.array([0.0, 1.0 + i, 0.5 + i])) for i in range(0, 10, 2)]
    tab[3] = tab[4]
    table.save_table(path, names, [0, 1, 2], tab)
    t3 = table.load_table(path)[2]
    for mode in (ampq.D_MODEL, ampq.D_MEASURED):
        a = shard.select_from_table(ampq, tab, F, groups, mode, 1e-3)
        b = shard.select_from_table(ampq, t3, F, groups, mode, 1e-3)
        assert a[0].tolist() == b[0].tolist() and a[1:] == b[1:]
    with pytest.raises(ValueError):
        table.save_table(path, names, [0, 1], tab)

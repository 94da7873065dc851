// Host-side steps around the sensitivity pass (include/ampq.h): partition of a
// model graph into sequential sub-graphs (what Appendix B's Algorithm 2
// produces, computed here from dominators), the theoretical-time and memory
// gain tables (Sec. 2.3.2, 2.3.3), the two baseline strategies (Sec. 3.1) and
// the merge of per-rank sample means (Sec. 2.2).  No GPU.
#include <algorithm>
#include <vector>

#include "../../include/ampq.h"

namespace {

// A topological order of the graph with a start vertex (index n) in front of
// every source; empty when the graph has a cycle.
std::vector<int> topological_order(int n, const std::vector<std::vector<int>>& next, std::vector<int> indeg) {
    std::vector<int> order, ready;
    order.reserve(n + 1);
    order.push_back(n);
    for (int v = n - 1; v >= 0; --v)
        if (indeg[v] == 0) ready.push_back(v);
    while (!ready.empty()) {
        const int v = ready.back();
        ready.pop_back();
        order.push_back(v);
        for (int w : next[v])
            if (--indeg[w] == 0) ready.push_back(w);
    }
    if ((int)order.size() != n + 1) order.clear();
    return order;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

// From the definition of a sequential sub-graph (Sec. 2.3.1, Appendix B): a
// sub-graph ends at a vertex that every start -> end path runs through, i.e. at
// a dominator of the end vertex in the graph rooted at the start vertex.  In a
// DAG the immediate dominator of v is the nearest common ancestor, in the
// dominator tree, of v's predecessors, and one sweep in topological order
// finds them all.  The dominators of the end vertex form a chain start = s_0,
// s_1, ..., s_k = end.  Let s_i be the deepest chain vertex that dominates a
// vertex u other than itself.  u cannot reach s_i or anything before it (the
// graph is acyclic and s_i reaches u); some start -> u path avoids s_{i+1}, and
// glued to any u -> end path it must still meet s_{i+1}, so every path from u
// meets s_{i+1}: the first chain vertex u reaches is s_{i+1}, and u belongs to
// the sub-graph that s_{i+1} closes.  A chain vertex belongs to the one it closes.
int ampq_partition(int n, int n_edges, const int* edge_src, const int* edge_dst, const unsigned char* quantisable,
                   int* group_of, int* n_groups) {
    if (n < 1 || n_edges < 0 || !quantisable || !group_of || !n_groups || (n_edges > 0 && (!edge_src || !edge_dst)))
        return AMPQ_ERR_INVALID;
    std::vector<std::vector<int>> next(n), prev(n);
    std::vector<int> indeg(n, 0);
    for (int e = 0; e < n_edges; ++e) {
        const int u = edge_src[e], v = edge_dst[e];
        if (u < 0 || u >= n || v < 0 || v >= n || u == v) return AMPQ_ERR_INVALID;
        next[u].push_back(v);
        prev[v].push_back(u);
        ++indeg[v];
    }
    int end = -1;
    for (int v = 0; v < n; ++v)
        if (next[v].empty()) {
            if (end >= 0) return AMPQ_ERR_INVALID;  // more than one sink
            end = v;
        }
    if (end < 0) return AMPQ_ERR_INVALID;
    const std::vector<int> order = topological_order(n, next, indeg);
    if (order.empty()) return AMPQ_ERR_INVALID;  // a cycle
    const int start = n;
    std::vector<int> rank(n + 1, 0), idom(n + 1, start);
    for (int i = 0; i <= n; ++i) rank[order[i]] = i;
    for (int i = 1; i <= n; ++i) {  // predecessors come earlier in the order, so their dominators are final
        const int v = order[i];
        int dom = -1;
        if (prev[v].empty()) dom = start;
        for (int u : prev[v]) {
            if (dom < 0) { dom = u; continue; }
            int a = dom, b = u;  // nearest common ancestor in the dominator tree
            while (a != b) {
                if (rank[a] > rank[b]) a = idom[a];
                else b = idom[b];
            }
            dom = a;
        }
        idom[v] = dom;
    }
    // the chain of the end vertex's dominators, and for every vertex how many
    // chain vertices (the start vertex not counted) dominate it, itself included
    std::vector<char> on_chain(n + 1, 0);
    for (int v = end; v != start; v = idom[v]) on_chain[v] = 1;
    std::vector<int> chain_above(n + 1, 0);
    for (int i = 1; i <= n; ++i) {
        const int v = order[i];
        chain_above[v] = chain_above[idom[v]] + (on_chain[v] ? 1 : 0);
    }
    int k = chain_above[end];  // sub-graphs before non-quantisable ones are dropped
    std::vector<int> label(k, -1);
    std::vector<char> used(k, 0);
    for (int v = 0; v < n; ++v) {
        const int g = on_chain[v] ? chain_above[v] - 1 : chain_above[v];
        group_of[v] = quantisable[v] ? g : -1;
        if (quantisable[v]) used[g] = 1;
    }
    int groups = 0;
    for (int g = 0; g < k; ++g)
        if (used[g]) label[g] = groups++;
    for (int v = 0; v < n; ++v)
        if (group_of[v] >= 0) group_of[v] = label[group_of[v]];
    *n_groups = groups;
    return AMPQ_OK;
}

int ampq_gain_table(int gain_kind, int Lj, const int* layer_kind, const long long* N, const long long* C,
                    const long long* K, const unsigned char* Q, int Pj, const double* delta, int F, double* c_out) {
    if (!layer_kind || !N || !C || !K || !Q || !delta || !c_out || Lj < 1 || Pj < 1 || F < 1) return AMPQ_ERR_INVALID;
    if (gain_kind != AMPQ_GAIN_MAC && gain_kind != AMPQ_GAIN_MEMORY) return AMPQ_ERR_INVALID;
    for (int l = 0; l < Lj; ++l)
        if ((layer_kind[l] != AMPQ_LINEAR && layer_kind[l] != AMPQ_BGEMM) || N[l] < 0 || C[l] < 0 || K[l] < 0)
            return AMPQ_ERR_INVALID;
    for (long long i = 0; i < (long long)Lj * Pj; ++i)
        if (Q[i] >= F) return AMPQ_ERR_INVALID;
    for (int p = 0; p < Pj; ++p) {
        double c = 0.0;
        for (int l = 0; l < Lj; ++l) {
            const bool lin = layer_kind[l] == AMPQ_LINEAR;
            double units;  // multiply-accumulates, or stored parameters
            if (gain_kind == AMPQ_GAIN_MAC)
                units = lin ? (double)N[l] * (double)C[l] * (double)K[l] : (double)N[l] * (double)C[l] * (double)C[l];
            else
                units = lin ? (double)C[l] * (double)K[l] : 0.0;
            c += units * delta[Q[l + (size_t)Lj * p]];
        }
        c_out[p] = c;
    }
    return AMPQ_OK;
}

int ampq_select_in_order(int L, const int* order, const double* d_low, const double* c_low, double budget,
                         unsigned char* chosen, double* c_total, double* d_total) {
    if (L < 0 || (L > 0 && (!order || !d_low || !c_low || !chosen)) || !(budget >= 0.0)) return AMPQ_ERR_INVALID;
    std::vector<char> seen(L, 0);
    for (int i = 0; i < L; ++i) {
        if (order[i] < 0 || order[i] >= L || seen[order[i]]) return AMPQ_ERR_INVALID;  // not a permutation
        seen[order[i]] = 1;
        chosen[i] = 0;
    }
    double d = 0.0, c = 0.0;
    for (int i = 0; i < L; ++i) {
        const int u = order[i];
        if (!(d + d_low[u] <= budget)) break;
        d += d_low[u];
        c += c_low[u];
        chosen[u] = 1;
    }
    if (c_total) *c_total = c;
    if (d_total) *d_total = d;
    return AMPQ_OK;
}

int ampq_merge_sample_tables(const double* tables, const int* R_local, int nranks, int L, int K, double* out) {
    if (!tables || !R_local || !out || nranks < 1 || L < 0 || K < 1) return AMPQ_ERR_INVALID;
    double total = 0.0;
    for (int i = 0; i < nranks; ++i) {
        if (R_local[i] < 0) return AMPQ_ERR_INVALID;
        total += (double)R_local[i];
    }
    if (!(total > 0.0)) return AMPQ_ERR_INVALID;
    const size_t n = (size_t)L * K;
    for (size_t e = 0; e < n; ++e) {
        double acc = 0.0;  // sum over all samples = sum over ranks of R_i * (mean over rank i's samples)
        for (int i = 0; i < nranks; ++i) acc += (double)R_local[i] * tables[(size_t)i * n + e];
        out[e] = acc / total;
    }
    return AMPQ_OK;
}

#pragma GCC visibility pop
}  // extern "C"

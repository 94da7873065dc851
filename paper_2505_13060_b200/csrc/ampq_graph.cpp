// Host-side steps around the sensitivity pass (include/ampq.h): partition of a
// model graph into sequential sub-graphs (Appendix B, Algorithm 2), the
// theoretical-time and memory gain tables (Sec. 2.3.2, 2.3.3) and the two
// baseline strategies (Sec. 3.1).  No GPU.
#include <algorithm>
#include <set>
#include <vector>

#include "../../include/ampq.h"

namespace {

// Longest path (in edges) from the added start vertex to every vertex, by
// dynamic programming over a topological order; returns false on a cycle.
bool longest_paths(int n, const std::vector<std::vector<int>>& next, const std::vector<int>& indeg0,
                   std::vector<int>& len) {
    std::vector<int> indeg(indeg0), ready;
    len.assign(n, 1);  // start -> source has length 1
    for (int v = 0; v < n; ++v)
        if (indeg[v] == 0) ready.push_back(v);
    int done = 0;
    while (!ready.empty()) {
        const int v = ready.back();
        ready.pop_back();
        ++done;
        for (int w : next[v]) {
            len[w] = std::max(len[w], len[v] + 1);
            if (--indeg[w] == 0) ready.push_back(w);
        }
    }
    return done == n;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

int ampq_partition(int n, int n_edges, const int* edge_src, const int* edge_dst, const unsigned char* quantisable,
                   int* group_of, int* n_groups) {
    if (n < 1 || n_edges < 0 || !quantisable || !group_of || !n_groups || (n_edges > 0 && (!edge_src || !edge_dst)))
        return AMPQ_ERR_INVALID;
    std::vector<std::vector<int>> next(n);
    std::vector<int> indeg(n, 0);
    for (int e = 0; e < n_edges; ++e) {
        const int u = edge_src[e], v = edge_dst[e];
        if (u < 0 || u >= n || v < 0 || v >= n || u == v) return AMPQ_ERR_INVALID;
        next[u].push_back(v);
        ++indeg[v];
    }
    int end = -1;
    for (int v = 0; v < n; ++v)
        if (next[v].empty()) {
            if (end >= 0) return AMPQ_ERR_INVALID;  // more than one sink
            end = v;
        }
    std::vector<int> len;
    if (end < 0 || !longest_paths(n, next, indeg, len)) return AMPQ_ERR_INVALID;  // a cycle

    // Walk from the start vertex.  The frontier holds the vertices whose turn has
    // not come; at level `cur` every frontier vertex whose longest path equals
    // cur moves into the current sub-graph and its successors join the frontier.
    // When one vertex is left, every path runs through it: it closes the sub-graph.
    for (int v = 0; v < n; ++v) group_of[v] = -1;
    int groups = 0;
    std::set<int> frontier;
    for (int v = 0; v < n; ++v)
        if (indeg[v] == 0) frontier.insert(v);
    int cur = 1;  // = len[start] + 1
    bool at_end = false;
    while (!at_end) {
        std::vector<int> members;
        while (frontier.size() > 1) {
            std::vector<int> now;
            for (int v : frontier)
                if (len[v] <= cur) now.push_back(v);
            for (int v : now) {
                frontier.erase(v);
                members.push_back(v);
                for (int w : next[v]) frontier.insert(w);
            }
            ++cur;
        }
        const int exit_vertex = *frontier.begin();
        members.push_back(exit_vertex);
        bool any = false;
        for (int v : members)
            if (quantisable[v]) {
                group_of[v] = groups;
                any = true;
            }
        if (any) ++groups;
        at_end = exit_vertex == end;
        frontier.clear();
        for (int w : next[exit_vertex]) frontier.insert(w);
        cur = len[exit_vertex] + 1;
    }
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

#pragma GCC visibility pop
}  // extern "C"

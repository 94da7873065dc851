// Exact solver of the integer program of Sec. 2.1 (a multiple-choice knapsack):
//   maximise sum_j c_{j,p_j}  subject to  sum_j d_{j,p_j} <= budget,
// one configuration p_j per group.  Host code, no GPU.
//
// Method: dynamic programming over the groups in order j = 0..J-1 on lists of
// partial assignments.  A partial assignment is kept unless another one has
// d <= , c >= AND a lexicographically smaller prefix.  Floating-point addition
// is monotone, so adding the same remaining terms to a dominated prefix can
// never make it strictly better than its dominator; with the lexicographic
// condition it can never win a tie either.  The surviving list therefore still
// contains the prefix of the assignment that an exhaustive enumeration would
// return under the ordering "larger c, then smaller d, then lexicographically
// smaller p", and every sum is the same left fold in double that an
// enumeration forms, so the result is identical to enumeration bit for bit.
//
// To keep the lists short a partial assignment is also dropped when an upper
// bound on what it can still reach -- its c plus the linear relaxation of the
// remaining groups under the remaining budget (per group the upper convex hull
// of its (d, c) points, increments taken greedily by slope) -- lies below an
// incumbent (the relaxation rounded down, evaluated with the exact folds) by
// more than a rounding margin.  The comparison is strict, so assignments that
// tie with the optimum are never cut and the tie-break is unaffected.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <map>
#include <vector>

#include "ampq_select.h"

namespace ampq {

namespace {

struct Cand {
    double d, c;
    uint32_t parent;  // index (= lexicographic rank) of the prefix in the previous level
    uint32_t p;       // configuration chosen for this group
};

struct Back {
    uint32_t parent;
    uint32_t p;
};

// One increment along the upper convex hull of a group's (d, c) points.
struct Step {
    double dd, dc, slope;
    int j, to;
};

// Linear relaxation of the groups >= some level: hull increments by decreasing
// slope with running sums, so that the value for a given room is a binary search.
struct Relaxation {
    std::vector<double> cum_dd, cum_dc, dd, dc;
    void build(const std::vector<Step>& sorted, int from_group) {
        cum_dd.assign(1, 0.0);
        cum_dc.assign(1, 0.0);
        dd.clear();
        dc.clear();
        for (const Step& s : sorted) {
            if (s.j < from_group) continue;
            dd.push_back(s.dd);
            dc.push_back(s.dc);
            cum_dd.push_back(cum_dd.back() + s.dd);
            cum_dc.push_back(cum_dc.back() + s.dc);
        }
    }
    double fill(double room) const {
        if (!(room > 0.0) || dd.empty()) return 0.0;
        // largest k with cum_dd[k] <= room
        size_t k = (size_t)(std::upper_bound(cum_dd.begin(), cum_dd.end(), room) - cum_dd.begin()) - 1;
        double v = cum_dc[k];
        if (k < dd.size()) v += dc[k] * ((room - cum_dd[k]) / dd[k]);
        return v;
    }
};

}  // namespace

int select_mckp(int J, const int* P, const long long* off, const double* c, const double* d,
                double budget, long long state_limit, int* p_out, double* c_total, double* d_total) {
    if (J < 0) return kSelectInvalid;
    for (int j = 0; j < J; ++j) {
        if (P[j] <= 0) return kSelectInvalid;
        for (int p = 0; p < P[j]; ++p) {
            const double dv = d[off[j] + p], cv = c[off[j] + p];
            if (!(dv >= 0.0) || !(cv == cv)) return kSelectInvalid;  // partial sums of d must only grow
        }
    }
    if (!(budget == budget)) return kSelectInvalid;
    // per group: the cheapest option and the hull increments above it
    std::vector<double> base_d_suf((size_t)J + 1, 0.0), base_c_suf((size_t)J + 1, 0.0);
    std::vector<int> base_opt((size_t)J, 0);
    std::vector<Step> steps;
    for (int j = 0; j < J; ++j) {
        const double* cj = c + off[j];
        const double* dj = d + off[j];
        int b = 0;
        for (int p = 1; p < P[j]; ++p)
            if (dj[p] < dj[b] || (dj[p] == dj[b] && cj[p] > cj[b])) b = p;
        base_opt[j] = b;
        int at = b;
        for (;;) {  // walk the hull: steepest remaining rise, farthest on ties
            int nxt = -1;
            double best = 0.0;
            for (int p = 0; p < P[j]; ++p) {
                const double ddv = dj[p] - dj[at], dcv = cj[p] - cj[at];
                if (!(ddv > 0.0) || !(dcv > 0.0)) continue;
                const double sl = dcv / ddv;
                if (nxt < 0 || sl > best || (sl == best && dj[p] > dj[nxt])) { nxt = p; best = sl; }
            }
            if (nxt < 0) break;
            steps.push_back(Step{dj[nxt] - dj[at], cj[nxt] - cj[at], best, j, nxt});
            at = nxt;
        }
    }
    for (int j = J - 1; j >= 0; --j) {
        base_d_suf[j] = base_d_suf[j + 1] + d[off[j] + base_opt[j]];
        base_c_suf[j] = base_c_suf[j + 1] + c[off[j] + base_opt[j]];
    }
    std::stable_sort(steps.begin(), steps.end(), [](const Step& a, const Step& b) { return a.slope > b.slope; });
    // incumbent: the relaxation rounded down, summed exactly as an enumeration would
    bool have_inc = false;
    double inc_c = 0.0;
    {
        std::vector<int> choice(base_opt);
        std::vector<char> stopped((size_t)J, 0);
        double room = budget - base_d_suf[0];
        for (const Step& s : steps) {
            if (stopped[s.j]) continue;
            if (s.dd <= room) { room -= s.dd; choice[s.j] = s.to; }
            else stopped[s.j] = 1;
        }
        for (int pass = 0; pass < 2 && !have_inc; ++pass) {
            double cs = 0.0, ds = 0.0;
            for (int j = 0; j < J; ++j) {
                const int p = pass == 0 ? choice[j] : base_opt[j];
                ds += d[off[j] + p];
                cs += c[off[j] + p];
            }
            if (ds <= budget) { have_inc = true; inc_c = cs; }
        }
    }
    Relaxation relax;
    // level 0: the empty assignment
    std::vector<Cand> cur(1);
    cur[0] = Cand{0.0, 0.0, 0u, 0u};
    std::vector<std::vector<Back>> back((size_t)J);
    std::vector<Cand> cand;
    std::vector<uint32_t> order;
    std::vector<char> keep;
    for (int j = 0; j < J; ++j) {
        const double* cj = c + off[j];
        const double* dj = d + off[j];
        const int Pj = P[j];
        cand.clear();
        relax.build(steps, j + 1);
        const double rest_d = base_d_suf[j + 1], rest_c = base_c_suf[j + 1];
        // candidates in lexicographic order of their prefix: parent rank, then p
        for (uint32_t i = 0; i < (uint32_t)cur.size(); ++i) {
            for (int p = 0; p < Pj; ++p) {
                const double nd = cur[i].d + dj[p];
                if (!(nd <= budget)) continue;  // every later term is >= 0: it can only grow
                const double nc = cur[i].c + cj[p];
                const double md = 1e-9 * (std::fabs(nd + rest_d) + std::fabs(budget)) + 1e-300;
                const double room = budget - nd - rest_d;
                if (room < -md) continue;       // even the cheapest completion overshoots
                if (have_inc) {
                    const double ub = nc + rest_c + relax.fill((room > 0.0 ? room : 0.0) + md);
                    const double mc = 1e-9 * (std::fabs(ub) + std::fabs(inc_c)) + 1e-300;
                    if (ub + mc < inc_c) continue;  // cannot reach the incumbent
                }
                cand.push_back(Cand{nd, nc, i, (uint32_t)p});
                if ((long long)cand.size() > state_limit) return kSelectTooLarge;
            }
        }
        if (cand.empty()) return kSelectInfeasible;
        // sweep in order (d asc, c desc, lexicographic asc); everything already
        // swept has d <= the current d, so domination reduces to: some swept
        // survivor has c >= c_B and a smaller lexicographic index.
        const size_t n = cand.size();
        order.resize(n);
        for (size_t i = 0; i < n; ++i) order[i] = (uint32_t)i;
        std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
            if (cand[a].d != cand[b].d) return cand[a].d < cand[b].d;
            if (cand[a].c != cand[b].c) return cand[a].c > cand[b].c;
            return a < b;
        });
        keep.assign(n, 0);
        // staircase: c -> smallest lexicographic index among survivors with that
        // c or more; kept so that the index strictly increases with c.
        std::map<double, uint32_t> stair;
        for (size_t k = 0; k < n; ++k) {
            const uint32_t b = order[k];
            auto it = stair.lower_bound(cand[b].c);  // smallest c' >= c_B
            if (it != stair.end() && it->second < b) continue;  // dominated
            keep[b] = 1;
            // drop staircase entries made redundant: c' <= c_B with index >= b
            auto ins = stair.insert_or_assign(cand[b].c, b).first;
            while (ins != stair.begin()) {
                auto prev = std::prev(ins);
                if (prev->second >= b) stair.erase(prev);
                else break;
            }
        }
        // survivors, still in lexicographic order
        std::vector<Cand> next;
        next.reserve(n);
        back[j].reserve(n);
        for (size_t i = 0; i < n; ++i) {
            if (!keep[i]) continue;
            next.push_back(cand[i]);
            back[j].push_back(Back{cand[i].parent, cand[i].p});
        }
        cur.swap(next);
    }
    // best final state: larger c, then smaller d, then smaller lexicographic rank
    size_t best = 0;
    bool have = false;
    for (size_t i = 0; i < cur.size(); ++i) {
        if (!(cur[i].d <= budget)) continue;
        if (!have || cur[i].c > cur[best].c || (cur[i].c == cur[best].c && cur[i].d < cur[best].d)) {
            best = i;
            have = true;
        }
    }
    if (!have) return kSelectInfeasible;
    if (c_total) *c_total = cur[best].c;
    if (d_total) *d_total = cur[best].d;
    uint32_t idx = (uint32_t)best;
    for (int j = J - 1; j >= 0; --j) {
        if (p_out) p_out[j] = (int)back[j][idx].p;
        idx = back[j][idx].parent;
    }
    return kSelectOk;
}

}  // namespace ampq

// Exact multiple-choice-knapsack solver for the integer program of Sec. 2.1.
#pragma once

namespace ampq {

enum { kSelectOk = 0, kSelectInvalid = 1, kSelectInfeasible = 2, kSelectTooLarge = 3 };

// Group j owns entries off[j] .. off[j]+P[j]-1 of c[] and d[]; every d must be
// >= 0.  Returns the assignment an exhaustive enumeration would return under
// the ordering: larger c, then smaller d, then lexicographically smaller p,
// with c and d formed as left folds over j in double.  state_limit bounds the
// number of partial assignments held per group (kSelectTooLarge beyond it).
int select_mckp(int J, const int* P, const long long* off, const double* c, const double* d,
                double budget, long long state_limit, int* p_out, double* c_total, double* d_total);

}  // namespace ampq

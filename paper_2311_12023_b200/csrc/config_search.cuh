// Budgeted assignment of one quantization configuration per matrix (Sec. 3.2, Algorithm 3): minimize the summed error
// subject to the summed storage staying within the budget.  The paper hands this integer program to an off-the-shelf
// solver; here it is solved by dynamic programming over the matrices on the Pareto frontier of (storage, error)
// prefixes -- exact while the frontier stays below `kMaxFrontier` points, thinned to evenly spaced storage values
// beyond that.  Host code only.
#pragma once

#include <algorithm>
#include <cstdint>
#include <vector>

namespace lq {
namespace cfgsearch {

constexpr size_t kMaxFrontier = 1 << 15;

struct Node { double storage, error; int parent, choice; };

// E, S: [n][m] row major.  assignment: [n].  Returns 0, or -1 when no assignment fits the budget.
inline int assign(const double* E, const double* S, int n, int m, double budget, int* assignment, double* total_error,
                  double* total_storage) {
    std::vector<std::vector<Node>> levels(n + 1);
    levels[0].push_back(Node{0.0, 0.0, -1, -1});
    // cheapest completion of the remaining matrices, to discard prefixes that cannot fit
    std::vector<double> min_rest(n + 1, 0.0);
    for (int i = n - 1; i >= 0; --i) {
        double mn = S[static_cast<size_t>(i) * m];
        for (int c = 1; c < m; ++c) mn = std::min(mn, S[static_cast<size_t>(i) * m + c]);
        min_rest[i] = min_rest[i + 1] + mn;
    }
    for (int i = 0; i < n; ++i) {
        std::vector<Node> cand;
        cand.reserve(levels[i].size() * m);
        for (size_t pidx = 0; pidx < levels[i].size(); ++pidx) {
            const Node& pn = levels[i][pidx];
            for (int c = 0; c < m; ++c) {
                const double st = pn.storage + S[static_cast<size_t>(i) * m + c];
                if (st + min_rest[i + 1] > budget) continue;
                cand.push_back(Node{st, pn.error + E[static_cast<size_t>(i) * m + c], static_cast<int>(pidx), c});
            }
        }
        if (cand.empty()) return -1;
        // Pareto frontier: ascending storage, strictly descending error (ties: first configuration index wins)
        std::stable_sort(cand.begin(), cand.end(), [](const Node& a, const Node& b) {
            if (a.storage != b.storage) return a.storage < b.storage;
            return a.error < b.error;
        });
        std::vector<Node>& fr = levels[i + 1];
        double best = 1e300;
        for (const Node& nd : cand)
            if (nd.error < best) { fr.push_back(nd); best = nd.error; }
        if (fr.size() > kMaxFrontier) {
            std::vector<Node> thin;
            const double lo = fr.front().storage, hi = fr.back().storage;
            const double step = (hi - lo) / static_cast<double>(kMaxFrontier);
            double next = lo;
            for (size_t k = 0; k < fr.size(); ++k) {
                // keep the last point (least error) below each storage mark, and always the final point
                const bool last_in_bin = (k + 1 == fr.size()) || (fr[k + 1].storage > next + step);
                if (last_in_bin) { thin.push_back(fr[k]); next = fr[k].storage; }
            }
            fr.swap(thin);
        }
    }
    // the frontier of the last level is sorted by storage with falling error: its last point has the least error
    const std::vector<Node>& fin = levels[n];
    int idx = static_cast<int>(fin.size()) - 1;
    if (total_error) *total_error = fin[idx].error;
    if (total_storage) *total_storage = fin[idx].storage;
    for (int i = n; i >= 1; --i) {
        const Node& nd = levels[i][idx];
        assignment[i - 1] = nd.choice;
        idx = nd.parent;
    }
    return 0;
}

}  // namespace cfgsearch
}  // namespace lq

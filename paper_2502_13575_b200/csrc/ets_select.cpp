// Selection step (see ets_select.hpp).
//
// The paper solves Eq. 5 / Eq. 6 with a general ILP solver.  The problem has a tree structure that makes
// a dedicated exact method short: without the coverage term the best subset follows from one bottom-up
// pass (a node is worth keeping iff what can be gained below it exceeds its own cost), and the coverage
// term couples trajectories only through clusters.  So: branch and bound over trajectories; the bound
// is the bottom-up pass in which every undecided trajectory of a cluster that no fixed trajectory
// covers yet is credited the whole cluster bonus (an over-count when the pass keeps several of them);
// when the pass keeps at most one per such cluster the bound is attained and the branch is closed.
#include "ets_select.hpp"

#include "../../include/ets.h"

#include <algorithm>
#include <cmath>
#include <numeric>

namespace ets {

void rebase_weights(int32_t n, const double* reward, const int32_t* member, int32_t width, double temperature,
                    int32_t* out) {
    std::vector<int32_t> order;
    for (int32_t i = 0; i < n; ++i) {
        out[i] = 0;
        if (!member || member[i]) order.push_back(i);
    }
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return reward[a] > reward[b]; });
    if (order.empty()) return;
    const double top = reward[order[0]];
    std::vector<double> e(order.size());
    for (size_t k = 0; k < order.size(); ++k) e[k] = std::exp((reward[order[k]] - top) / temperature);
    int64_t left = width;
    for (size_t k = 0; k < order.size() && left > 0; ++k) {
        double denom = 0.0;
        for (size_t j = k; j < order.size(); ++j) denom += e[j];
        const int64_t w = (int64_t)std::ceil((double)left * (e[k] / denom));   // the last share is exactly 1
        out[order[k]] = (int32_t)w;
        left -= w;
    }
}

namespace {

struct Solver {
    int32_t n = 0, L = 0, K = 0;
    const int32_t* parent = nullptr;
    const int32_t* leaf_node = nullptr;
    std::vector<double> w;           // W_i / sum W
    std::vector<int32_t> cl;         // dense cluster id or -1
    double beta = 0.0, delta = 0.0;  // cost of a node, bonus of a cluster
    std::vector<int32_t> leaf_off, leaf_at;   // trajectories sitting at each node
    // search state
    std::vector<int8_t> fix;         // -1 undecided, 0 pruned, 1 kept
    std::vector<int32_t> best_keep;
    double best = -INFINITY;
    int64_t nodes = 0, limit = 0;
    bool hit_limit = false;
    // scratch
    std::vector<double> val;
    std::vector<int8_t> forced, take;
    std::vector<int32_t> covered, picked;

    double exact(const std::vector<int32_t>& keep) const {
        std::vector<int8_t> nk((size_t)n, 0), ck((size_t)std::max(K, 1), 0);
        double g = 0.0;
        int32_t nn = 0, nc = 0;
        for (int32_t i = 0; i < L; ++i) {
            if (!keep[i]) continue;
            g += w[i];
            for (int32_t v = leaf_node[i]; v >= 0 && !nk[v]; v = parent[v]) { nk[v] = 1; ++nn; }
            if (cl[i] >= 0 && !ck[cl[i]]) { ck[cl[i]] = 1; ++nc; }
        }
        return g - beta * nn + delta * nc;
    }

    // Upper bound for the current fixings and the selection that attains it in the relaxed problem.
    // Returns false when the fixings keep nothing and the relaxed optimum is the empty set.
    bool relax(double& ub, std::vector<int32_t>& sel, bool with_bonus = true) {
        std::fill(covered.begin(), covered.end(), 0);
        int32_t n_cov = 0;
        for (int32_t i = 0; i < L; ++i)
            if (fix[i] == 1 && cl[i] >= 0 && !covered[cl[i]]) { covered[cl[i]] = 1; ++n_cov; }
        std::fill(val.begin(), val.end(), 0.0);
        std::fill(forced.begin(), forced.end(), 0);
        auto gain = [&](int32_t i) { return w[i] + ((with_bonus && cl[i] >= 0 && !covered[cl[i]]) ? delta : 0.0); };
        // children come after their parent: one pass from the last node up
        for (int32_t v = n - 1; v >= 0; --v) {
            double x = val[v] - beta;
            for (int32_t k = leaf_off[v]; k < leaf_off[v + 1]; ++k) {
                const int32_t i = leaf_at[k];
                if (fix[i] == 1) { x += w[i]; forced[v] = 1; }
                else if (fix[i] == -1 && gain(i) > 0.0) x += gain(i);
            }
            val[v] = x;
            if (parent[v] >= 0) {
                if (forced[v]) { val[parent[v]] += x; forced[parent[v]] = 1; }
                else if (x > 0.0) val[parent[v]] += x;
            }
        }
        ub = delta * n_cov;
        bool any = false;
        for (int32_t v = 0; v < n; ++v)
            if (parent[v] < 0 && (forced[v] || val[v] > 0.0)) { ub += val[v]; any = true; }
        // the selection: walk down through the nodes that are worth keeping
        sel.assign((size_t)L, 0);
        for (int32_t v = 0; v < n; ++v) {
            const bool up = parent[v] < 0 || take[parent[v]];
            take[v] = up && (forced[v] || val[v] > 0.0);
            if (!take[v]) continue;
            for (int32_t k = leaf_off[v]; k < leaf_off[v + 1]; ++k) {
                const int32_t i = leaf_at[k];
                if (fix[i] == 1 || (fix[i] == -1 && gain(i) > 0.0)) sel[i] = 1;
            }
        }
        return any;
    }

    void search() {
        if (hit_limit) return;
        if (++nodes > limit) { hit_limit = true; return; }
        double ub;
        std::vector<int32_t> sel;
        // What is worth keeping without any cluster bonus is part of some optimum: the value without the
        // coverage term is supermodular in the kept set (a trajectory costs less the more of its path is
        // already kept) and coverage only grows, so adding this set to an optimum never lowers it.  Fixing
        // it covers most clusters at once and leaves only trajectories that need the bonus undecided.
        relax(ub, sel, false);
        std::vector<int32_t> fixed_here;
        for (int32_t i = 0; i < L; ++i)
            if (sel[i] && fix[i] == -1) { fix[i] = 1; fixed_here.push_back(i); }
        struct Undo {
            std::vector<int8_t>& fix; std::vector<int32_t>& ids;
            ~Undo() { for (int32_t i : ids) fix[i] = -1; }
        } undo{fix, fixed_here};
        const bool any = relax(ub, sel);
        if (!any) {
            // nothing is worth keeping here, but one trajectory must be: open a branch per undecided one
            std::vector<int32_t> cand;
            for (int32_t i = 0; i < L; ++i)
                if (fix[i] == -1) cand.push_back(i);
            for (int32_t i : cand) {
                fix[i] = 1;
                search();
                fix[i] = -1;
            }
            return;
        }
        if (ub <= best + 1e-13) return;
        const double lb = exact(sel);
        if (lb > best) { best = lb; best_keep = sel; }
        if (ub - lb <= 1e-13) return;
        // the gap comes from a cluster credited more than once: branch on its heaviest undecided pick
        std::fill(picked.begin(), picked.end(), 0);
        int32_t branch = -1;
        for (int32_t i = 0; i < L; ++i)
            if (sel[i] && fix[i] == -1 && cl[i] >= 0 && !covered[cl[i]]) ++picked[cl[i]];
        for (int32_t i = 0; i < L; ++i)
            if (sel[i] && fix[i] == -1 && cl[i] >= 0 && !covered[cl[i]] && picked[cl[i]] > 1 && (branch < 0 || w[i] > w[branch]))
                branch = i;
        if (branch < 0) return;   // no over-count left: the difference is rounding
        fix[branch] = 1;
        search();
        fix[branch] = 0;
        search();
        fix[branch] = -1;
    }
};

}  // namespace

int32_t select_trajectories(int32_t n_nodes, const int32_t* parent, int32_t n_leaves, const int32_t* leaf_node,
                            const double* reward, const int32_t* cluster, const SelectParams& p, SelectResult& out,
                            std::string& err) {
    if (n_nodes <= 0 || n_leaves <= 0 || !parent || !leaf_node || !reward) { err = "empty tree or null array"; return -1; }
    if (!(p.temperature > 0.0) || p.width <= 0 || p.lambda_b < 0.0 || p.lambda_d < 0.0) {
        err = "temperature and width must be positive, the lambdas non-negative"; return -1;
    }
    for (int32_t v = 0; v < n_nodes; ++v)
        if (parent[v] < -1 || parent[v] >= v) { err = "parent[" + std::to_string(v) + "] must lie in [-1, i)"; return -2; }
    for (int32_t i = 0; i < n_leaves; ++i) {
        if (leaf_node[i] < 0 || leaf_node[i] >= n_nodes) { err = "leaf_node out of range"; return -2; }
        if (!std::isfinite(reward[i])) { err = "reward must be finite"; return -1; }
    }
    out = SelectResult();
    out.weight.assign((size_t)n_leaves, 0);
    rebase_weights(n_leaves, reward, nullptr, p.width, p.temperature, out.weight.data());

    Solver s;
    s.n = n_nodes; s.L = n_leaves; s.parent = parent; s.leaf_node = leaf_node;
    const double total = (double)std::accumulate(out.weight.begin(), out.weight.end(), (int64_t)0);
    s.w.resize((size_t)n_leaves);
    for (int32_t i = 0; i < n_leaves; ++i) s.w[i] = total > 0 ? out.weight[i] / total : 0.0;
    // dense cluster ids (negative = the trajectory belongs to no cluster)
    s.cl.assign((size_t)n_leaves, -1);
    if (cluster) {
        std::vector<int32_t> ids;
        for (int32_t i = 0; i < n_leaves; ++i)
            if (cluster[i] >= 0) ids.push_back(cluster[i]);
        std::sort(ids.begin(), ids.end());
        ids.erase(std::unique(ids.begin(), ids.end()), ids.end());
        s.K = (int32_t)ids.size();
        for (int32_t i = 0; i < n_leaves; ++i)
            if (cluster[i] >= 0) s.cl[i] = (int32_t)(std::lower_bound(ids.begin(), ids.end(), cluster[i]) - ids.begin());
    }
    s.beta = p.lambda_b / n_nodes;
    s.delta = s.K > 0 ? p.lambda_d / s.K : 0.0;
    s.leaf_off.assign((size_t)n_nodes + 1, 0);
    for (int32_t i = 0; i < n_leaves; ++i) ++s.leaf_off[leaf_node[i] + 1];
    for (int32_t v = 0; v < n_nodes; ++v) s.leaf_off[v + 1] += s.leaf_off[v];
    s.leaf_at.resize((size_t)n_leaves);
    {
        std::vector<int32_t> cur(s.leaf_off.begin(), s.leaf_off.end() - 1);
        for (int32_t i = 0; i < n_leaves; ++i) s.leaf_at[cur[leaf_node[i]]++] = i;
    }
    s.fix.assign((size_t)n_leaves, -1);
    s.val.assign((size_t)n_nodes, 0.0);
    s.forced.assign((size_t)n_nodes, 0);
    s.take.assign((size_t)n_nodes, 0);
    s.covered.assign((size_t)std::max(s.K, 1), 0);
    s.picked.assign((size_t)std::max(s.K, 1), 0);
    s.limit = p.node_limit > 0 ? p.node_limit : ((int64_t)1 << 20);
    s.search();
    if (s.best_keep.empty()) {   // cannot happen for a valid tree, but never return an empty selection
        s.best_keep.assign((size_t)n_leaves, 0);
        s.best_keep[0] = 1;
        s.best = s.exact(s.best_keep);
    }
    out.keep = s.best_keep;
    out.objective = s.best;
    out.proven_optimal = !s.hit_limit;
    out.nodes_explored = s.nodes;
    out.continuations.assign((size_t)n_leaves, 0);
    rebase_weights(n_leaves, reward, out.keep.data(), p.width, p.temperature, out.continuations.data());
    out.node_kept.assign((size_t)n_nodes, 0);
    for (int32_t i = 0; i < n_leaves; ++i)
        if (out.keep[i])
            for (int32_t v = leaf_node[i]; v >= 0 && !out.node_kept[v]; v = parent[v]) out.node_kept[v] = 1;
    return 0;
}

}  // namespace ets

extern "C" int32_t ets_select(int32_t n_nodes, const int32_t* parent, int32_t n_leaves, const int32_t* leaf_node,
                              const double* reward, const int32_t* cluster, const ets_select_params* params,
                              int32_t* weight, int32_t* keep, int32_t* continuations, int32_t* node_kept,
                              ets_select_result* result) {
    if (!params || !result) return ETS_ERR_INVALID_ARG;
    ets::SelectParams p;
    p.temperature = params->temperature;
    p.lambda_b = params->lambda_b;
    p.lambda_d = params->lambda_d;
    p.width = params->width;
    p.node_limit = params->node_limit;
    ets::SelectResult r;
    std::string err;
    const int32_t rc = ets::select_trajectories(n_nodes, parent, n_leaves, leaf_node, reward, cluster, p, r, err);
    if (rc == -1) return ETS_ERR_INVALID_ARG;
    if (rc == -2) return ETS_ERR_BAD_TREE;
    auto copy = [](int32_t* dst, const std::vector<int32_t>& v) { if (dst) std::copy(v.begin(), v.end(), dst); };
    copy(weight, r.weight);
    copy(keep, r.keep);
    copy(continuations, r.continuations);
    copy(node_kept, r.node_kept);
    result->objective = r.objective;
    result->nodes_explored = r.nodes_explored;
    result->proven_optimal = r.proven_optimal ? 1 : 0;
    result->n_kept = (int32_t)std::count(r.keep.begin(), r.keep.end(), 1);
    result->n_nodes_kept = (int32_t)std::count(r.node_kept.begin(), r.node_kept.end(), 1);
    result->reserved = 0;
    result->kv_tokens_kept = result->kv_tokens_all = 0;
    if (params->node_tokens) {
        std::vector<char> reached((size_t)n_nodes, 0);   // nodes with any trajectory at or below them
        for (int32_t i = 0; i < n_leaves; ++i)
            for (int32_t v = leaf_node[i]; v >= 0 && !reached[v]; v = parent[v]) reached[v] = 1;
        for (int32_t v = 0; v < n_nodes; ++v) {
            if (reached[v]) result->kv_tokens_all += params->node_tokens[v];
            if (r.node_kept[v]) result->kv_tokens_kept += params->node_tokens[v];
        }
    }
    return ETS_OK;
}

// Selection step of the search (Section 4 and Appendix B of the paper): which trajectories to keep so
// that promising and semantically different ones survive while the retained tree, whose KV the decode
// kernels stream, stays small.  Pure host C++.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace ets {

struct SelectParams {
    double temperature = 0.2;   // T_R of Eq. 1
    double lambda_b = 0.0;      // weight of the retained-tree size (Eq. 2)
    double lambda_d = 0.0;      // weight of the cluster coverage (Eq. 4)
    int32_t width = 0;          // continuations to hand out
    int64_t node_limit = 0;     // bound on branch-and-bound nodes (0 = 1 << 20)
};

struct SelectResult {
    std::vector<int32_t> weight;         // W_i of Eq. 1, all trajectories
    std::vector<int32_t> keep;           // 0/1 per trajectory
    std::vector<int32_t> continuations;  // W'_i of Eq. 3 (0 for pruned trajectories)
    std::vector<int32_t> node_kept;      // 0/1 per node of the tree
    double objective = 0.0;              // value of Eq. 4 for `keep`
    bool proven_optimal = false;         // false: the node limit was reached, `keep` is the best found
    int64_t nodes_explored = 0;
};

// Eq. 1 / Eq. 3: continuations per trajectory, highest reward first; `member` (nullable) restricts the
// walk to the retained trajectories.  Reading of what the paper leaves to the REBASE code: the budget
// starts at `width`, drops by each W_i, and the walk stops when nothing is left.
void rebase_weights(int32_t n, const double* reward, const int32_t* member, int32_t width, double temperature,
                    int32_t* out);

// Returns 0, or -1 (invalid argument) / -2 (bad tree) with a message.
int32_t select_trajectories(int32_t n_nodes, const int32_t* parent, int32_t n_leaves, const int32_t* leaf_node,
                            const double* reward, const int32_t* cluster, const SelectParams& p, SelectResult& out,
                            std::string& err);

}  // namespace ets

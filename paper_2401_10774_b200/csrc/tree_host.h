// Host representation of the static tree buffers.
#pragma once
#include <cstdint>
#include <vector>

#define MEDUSA_MAX_T 256
#define MEDUSA_MAX_DEPTH 8

namespace medusa {

struct TreeHost {
    int T = 0, P = 0, depth = 0, topk = 0;
    std::vector<uint64_t> mask;  // [T][mask_words]: bit j of row i (word j / 64, bit j % 64) -- node j is i or an ancestor
    int mask_words = 1;          // ceil(T / 64)
    std::vector<int32_t> pos, tree_idx, parent, retrieve;  // retrieve: [P][depth+1]
};

int32_t default_tree_paths(const int32_t *topk, int32_t depth, int32_t n_nodes, int32_t *out);
int32_t tree_paths_from_accuracies(const double *acc, int32_t depth, int32_t topk, int32_t n_nodes, int32_t *out,
                                   double *expected_len);
int32_t build_tree(const int32_t *paths, int32_t n_paths, int32_t max_depth, TreeHost &tr);

}  // namespace medusa

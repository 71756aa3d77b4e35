// Host side of the static candidate tree (paper Sec. 2.1.2, Fig. 2; sparse tree of Sec. 2.3.3).
// The tree never changes during decoding, so everything here runs once at set-up time on the CPU and the
// resulting buffers are uploaded to the device.
#include <algorithm>
#include <cstdint>
#include <queue>
#include <vector>

#include "../../include/medusa.h"
#include "tree_host.h"

namespace medusa {

namespace {

using Tuple = std::vector<int32_t>;

// lexicographic on elements; std::vector's operator< already puts a proper prefix before its extensions
bool by_depth_then_tuple(const Tuple &a, const Tuple &b)
{
    if (a.size() != b.size())
        return a.size() < b.size();
    return a < b;
}

}  // namespace

int32_t default_tree_paths(const int32_t *topk, int32_t depth, int32_t n_nodes, int32_t *out)
{
    if (!topk || !out || depth < 1 || depth > MEDUSA_MAX_DEPTH || n_nodes < 1)
        return MEDUSA_ERR_INVALID_ARG;
    // every node of the Cartesian tree with its accuracy denominator prod (rank+1)
    struct Cand { int64_t den; Tuple t; };
    std::vector<Cand> all;
    std::vector<Tuple> frontier{Tuple{}};
    for (int k = 0; k < depth; ++k) {
        if (topk[k] < 1)
            return MEDUSA_ERR_INVALID_ARG;
        std::vector<Tuple> next;
        for (const Tuple &p : frontier)
            for (int32_t r = 0; r < topk[k]; ++r) {
                Tuple c = p;
                c.push_back(r);
                int64_t den = 1;
                for (int32_t x : c) den *= (x + 1);
                all.push_back({den, c});
                next.push_back(std::move(c));
            }
        frontier.swap(next);
        if (all.size() > (1u << 20))
            return MEDUSA_ERR_SHAPE;
    }
    if ((size_t)(n_nodes - 1) > all.size())
        return MEDUSA_ERR_SHAPE;
    // Estimated accuracies never increase along a path, so the n best nodes by (accuracy desc, tuple asc)
    // form a connected tree and equal what adding the best connected node one at a time produces.
    std::stable_sort(all.begin(), all.end(), [](const Cand &a, const Cand &b) {
        if (a.den != b.den) return a.den < b.den;
        return a.t < b.t;
    });
    for (int i = 0; i < n_nodes - 1; ++i)
        for (int j = 0; j < depth; ++j)
            out[(size_t)i * depth + j] = j < (int)all[i].t.size() ? all[i].t[j] : -1;
    return n_nodes - 1;
}

// Sparse tree from an accuracy table (paper Sec. 2.3.3): best-first growth.  The frontier holds every child of a
// node already taken; the child with the largest path accuracy (product formed root to leaf in double) is taken
// next, ties going to the smaller tuple (a prefix before its extensions), and its own children join the frontier.
int32_t tree_paths_from_accuracies(const double *acc, int32_t depth, int32_t topk, int32_t n_nodes, int32_t *out,
                                   double *expected_len)
{
    if (!acc || !out || depth < 1 || depth > MEDUSA_MAX_DEPTH || topk < 1 || n_nodes < 1)
        return MEDUSA_ERR_INVALID_ARG;
    if (n_nodes > MEDUSA_MAX_T)
        return MEDUSA_ERR_SHAPE;
    for (int i = 0; i < depth * topk; ++i)
        if (!(acc[i] >= 0.0 && acc[i] <= 1.0))
            return MEDUSA_ERR_INVALID_ARG;
    double total = 0.0, level = 1.0;
    for (int k = 0; k < depth; ++k) {
        level *= (double)topk;
        total += level;
    }
    if ((double)(n_nodes - 1) > total)
        return MEDUSA_ERR_SHAPE;
    struct Cand { double a; Tuple t; };
    auto worse = [](const Cand &x, const Cand &y) {  // priority_queue keeps the "largest": y before x
        if (x.a != y.a) return x.a < y.a;
        return y.t < x.t;
    };
    std::priority_queue<Cand, std::vector<Cand>, decltype(worse)> frontier(worse);
    auto push_children = [&](const Tuple &parent, double pa) {
        const int k = (int)parent.size();
        if (k == depth) return;
        for (int32_t i = 0; i < topk; ++i) {
            Tuple c = parent;
            c.push_back(i);
            frontier.push({pa * acc[(size_t)k * topk + i], std::move(c)});
        }
    };
    push_children(Tuple{}, 1.0);
    double expect = 0.0;
    for (int n = 0; n < n_nodes - 1; ++n) {
        Cand best = frontier.top();
        frontier.pop();
        for (int j = 0; j < depth; ++j)
            out[(size_t)n * depth + j] = j < (int)best.t.size() ? best.t[j] : -1;
        expect += best.a;
        push_children(best.t, best.a);
    }
    if (expected_len)
        *expected_len = expect;
    return n_nodes - 1;
}

int32_t build_tree(const int32_t *paths, int32_t n_paths, int32_t max_depth, TreeHost &tr)
{
    if (n_paths < 0 || max_depth < 1 || (n_paths > 0 && !paths))
        return MEDUSA_ERR_INVALID_ARG;
    if (n_paths + 1 > MEDUSA_MAX_T || max_depth > MEDUSA_MAX_DEPTH)
        return MEDUSA_ERR_SHAPE;
    std::vector<Tuple> nodes;
    nodes.emplace_back();  // root
    for (int p = 0; p < n_paths; ++p) {
        Tuple t;
        bool ended = false;
        for (int j = 0; j < max_depth; ++j) {
            int32_t v = paths[(size_t)p * max_depth + j];
            if (v < 0) ended = true;
            else if (ended) return MEDUSA_ERR_INVALID_ARG;  // value after padding
            else t.push_back(v);
        }
        if (t.empty())
            return MEDUSA_ERR_INVALID_ARG;
        nodes.push_back(std::move(t));
    }
    std::sort(nodes.begin() + 1, nodes.end(), by_depth_then_tuple);
    const int T = (int)nodes.size();
    for (int i = 2; i < T; ++i)
        if (nodes[i] == nodes[i - 1])
            return MEDUSA_ERR_INVALID_ARG;  // duplicate
    tr = TreeHost{};
    tr.T = T;
    const int MW = (T + 63) / 64;
    tr.mask_words = MW;
    tr.mask.assign((size_t)T * MW, 0);
    tr.pos.assign(T, 0);
    tr.tree_idx.assign(T, 0);
    tr.parent.assign(T, -1);
    for (int i = 1; i < T; ++i) {
        tr.depth = std::max<int>(tr.depth, (int)nodes[i].size());
        for (int32_t r : nodes[i]) tr.topk = std::max<int>(tr.topk, r + 1);
    }
    tr.mask[0] = 1;
    for (int i = 1; i < T; ++i) {
        const Tuple &t = nodes[i];
        Tuple par(t.begin(), t.end() - 1);
        // parents are at the previous depth, which sorts earlier: binary search in [0, i)
        auto it = std::lower_bound(nodes.begin(), nodes.begin() + i, par, by_depth_then_tuple);
        if (it == nodes.begin() + i || *it != par)
            return MEDUSA_ERR_INVALID_ARG;  // not prefix-closed
        int pi = (int)(it - nodes.begin());
        tr.parent[i] = pi;
        for (int w = 0; w < MW; ++w)
            tr.mask[(size_t)i * MW + w] = tr.mask[(size_t)pi * MW + w];
        tr.mask[(size_t)i * MW + (i >> 6)] |= 1ull << (i & 63);
        tr.pos[i] = (int32_t)t.size();
        tr.tree_idx[i] = 1 + ((int32_t)t.size() - 1) * tr.topk + t.back();
    }
    std::vector<char> has_child(T, 0);
    for (int i = 1; i < T; ++i) has_child[tr.parent[i]] = 1;
    std::vector<int> leaves;
    for (int i = 0; i < T; ++i)
        if (!has_child[i]) leaves.push_back(i);
    std::sort(leaves.begin(), leaves.end(), [&](int a, int b) { return nodes[a] < nodes[b]; });
    tr.P = (int)leaves.size();
    const int W = tr.depth + 1;
    tr.retrieve.assign((size_t)tr.P * W, -1);
    for (int r = 0; r < tr.P; ++r) {
        int v = leaves[r];
        for (int j = (int)nodes[v].size(); v >= 0; v = tr.parent[v], --j)
            tr.retrieve[(size_t)r * W + j] = v;
    }
    return MEDUSA_OK;
}

}  // namespace medusa

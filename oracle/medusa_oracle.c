/*
 * medusa_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of one Medusa tree-verification
 * decode step (Medusa, arXiv 2401.10774), written from the paper's definitions.
 * It exists so that the CUDA library can be checked against something that
 * shares no code with it.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the product never does.
 *
 * Numerics: inputs are float32 arrays (or bf16 bit patterns widened exactly);
 * every activation is a double; every dot product / sum accumulates in double
 * in ascending index order.  Every token row is processed by the same loop
 * nest whether it is alone (plain decoding) or one of T tree rows, so
 * "Medusa-1 greedy == plain greedy" holds bit-for-bit inside this file.
 *
 * Function -> passage of the paper it restates
 *   ora_default_tree_paths     Sec. 2.3.3 (greedy node adding), App. C (64-node tree)
 *   ora_tree_paths_from_accuracies   Sec. 2.3.3 (greedy node adding from an accuracy table)
 *   ora_build_tree_buffers     Sec. 2.1.2, Fig. 2 (tree mask, positions, candidates)
 *   ora_medusa_heads           Sec. 2.1.1 (head definition)
 *   ora_topk / ora_expand_candidates   Sec. 2.1.2 (top-s_k per head, Cartesian tree)
 *   ora_tree_attention         Sec. 2.1.2, Fig. 2; App. G Table 5 ("parallel decoding" QK^T, PV)
 *   ora_tree_pass              App. G Table 5 (linears on q tokens) on a Llama-style block
 *   ora_evaluate_posterior     Sec. 2.3.1 (typical acceptance), Fig. 1 (longest accepted prefix)
 *   ora_evaluate_rejection     Sec. 1 / Sec. 2.3.1 first paragraph (rejection sampling of speculative decoding, reused)
 *   ora_accept_and_update_kv   (paper silent; KV cache implied by Sec. 3.3 / App. G)
 *   ora_generate / ora_generate_plain   Sec. 2 (the three sub-steps per decoding step)
 *
 * Parity pins: every function above is pinned by tests/test_oracle_*.py against
 * values fixed outside this file (paper figures, closed forms, library routines,
 * brute force).  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORA_MAX_T 256

/* Ancestor masks: node i owns W = ceil(T / 64) consecutive 64-bit words, bit j of the row (word j / 64, bit j % 64)
 * says whether node j is visible to node i.  Trees of up to 64 nodes have one word per node. */
static inline int mask_words(int T) { return (T + 63) / 64; }
static inline int mask_bit(const uint64_t *mask, int W, int i, int j)
{
    return (int)((mask[(size_t)i * W + (j >> 6)] >> (j & 63)) & 1ull);
}
static inline void mask_set(uint64_t *mask, int W, int i, int j) { mask[(size_t)i * W + (j >> 6)] |= 1ull << (j & 63); }
#define ORA_MAX_DEPTH 8

/* ------------------------------------------------------------------ helpers */

/* weight element i of array w; dt 0 = float32, 1 = bf16 bit pattern (uint16) */
static inline double wget(const void *w, size_t i, int dt)
{
    if (dt == 0)
        return (double)((const float *)w)[i];
    uint32_t u = ((uint32_t)((const uint16_t *)w)[i]) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* y[t][n] = sum_k W[n][k] * x[t][k]   (W is [N][K], "out x in", no bias) */
static void linear(const void *W, int dt, int N, int K, const double *x, int T, int ldx, double *y, int ldy)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int t = 0; t < T; ++t) {
            double acc = 0.0;
            const double *xr = x + (size_t)t * ldx;
            for (int k = 0; k < K; ++k)
                acc += wget(W, (size_t)n * K + k, dt) * xr[k];
            y[(size_t)t * ldy + n] = acc;
        }
    }
}

/* RMSNorm: y_i = g_i * x_i / sqrt(mean(x^2) + eps) */
static void rmsnorm(const double *x, const void *g, int dt, int d, double eps, double *y)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i)
        ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)d + eps);
    for (int i = 0; i < d; ++i)
        y[i] = wget(g, (size_t)i, dt) * (x[i] * r);
}

static inline double silu(double u) { return u / (1.0 + exp(-u)); }

/* Rotary embedding on one head vector of length D at integer position pos:
 * element i is paired with i + D/2, angle = pos * theta^(-2i/D). */
static void rope(double *v, int D, int64_t pos, double theta)
{
    int half = D / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(theta, -2.0 * (double)i / (double)D);
        double c = cos(ang), s = sin(ang);
        double a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = b * c + a * s;
    }
}

/* ------------------------------------------------------------------ trees */

/* order on rank tuples: element-wise, a proper prefix sorts before its extensions */
static int tuple_cmp(const int32_t *a, int la, const int32_t *b, int lb)
{
    int m = la < lb ? la : lb;
    for (int i = 0; i < m; ++i) {
        if (a[i] != b[i])
            return a[i] < b[i] ? -1 : 1;
    }
    if (la != lb)
        return la < lb ? -1 : 1;
    return 0;
}

static int tuple_len(const int32_t *p, int max_depth)
{
    int l = 0;
    while (l < max_depth && p[l] >= 0)
        ++l;
    return l;
}

/*
 * The sparse tree of Sec. 2.3.3 with the surrogate accuracy a_k^(i) = 1/(i+1):
 * start from the root and repeatedly add the not-yet-added node whose parent is
 * already in the tree and whose estimated accuracy prod_j a_j^(i_j) is highest,
 * until the tree has n_nodes nodes (root included).  Ties go to the smaller
 * tuple.  Accuracies are compared exactly through their integer denominators
 * prod_j (i_j+1).  paths_out: [n_nodes-1][depth], -1 padded, in order of insertion.
 * Returns the number of paths written, or -1 on bad arguments.
 */
int32_t ora_default_tree_paths(const int32_t *per_depth_topk, int32_t depth, int32_t n_nodes, int32_t *paths_out)
{
    if (depth < 1 || depth > ORA_MAX_DEPTH || n_nodes < 1)
        return -1;
    /* enumerate every node of the full Cartesian tree */
    size_t total = 0, level = 1;
    for (int k = 0; k < depth; ++k) {
        level *= (size_t)per_depth_topk[k];
        total += level;
    }
    if ((size_t)(n_nodes - 1) > total)
        return -1;
    int32_t *all = (int32_t *)malloc(total * depth * sizeof(int32_t));
    int *len = (int *)malloc(total * sizeof(int));
    char *in_tree = (char *)calloc(total, 1);
    size_t cnt = 0;
    for (int k = 1; k <= depth; ++k) {
        int32_t idx[ORA_MAX_DEPTH] = {0};
        for (;;) {
            for (int j = 0; j < depth; ++j)
                all[cnt * depth + j] = j < k ? idx[j] : -1;
            len[cnt++] = k;
            int j = k - 1;
            while (j >= 0 && ++idx[j] == per_depth_topk[j]) {
                idx[j] = 0;
                --j;
            }
            if (j < 0)
                break;
        }
    }
    int added = 0;
    while (added < n_nodes - 1) {
        long best = -1;
        int64_t best_den = 0;
        for (size_t c = 0; c < cnt; ++c) {
            if (in_tree[c])
                continue;
            /* connected: parent (the tuple minus its last element) already added, or depth 1 */
            int ok = (len[c] == 1);
            if (!ok) {
                for (size_t p = 0; p < cnt && !ok; ++p)
                    if (in_tree[p] && len[p] == len[c] - 1 &&
                        tuple_cmp(all + p * depth, len[p], all + c * depth, len[c] - 1) == 0)
                        ok = 1;
            }
            if (!ok)
                continue;
            int64_t den = 1;
            for (int j = 0; j < len[c]; ++j)
                den *= (int64_t)(all[c * depth + j] + 1);
            if (best < 0 || den < best_den ||
                (den == best_den && tuple_cmp(all + c * depth, len[c], all + best * depth, len[best]) < 0)) {
                best = (long)c;
                best_den = den;
            }
        }
        in_tree[best] = 1;
        memcpy(paths_out + (size_t)added * depth, all + (size_t)best * depth, depth * sizeof(int32_t));
        ++added;
    }
    free(all);
    free(len);
    free(in_tree);
    return added;
}

/*
 * Sparse-tree construction from measured accuracies (Sec. 2.3.3).  acc[k][i] (row-major [depth][topk]) is the
 * estimated probability that the rank-i prediction of head k+1 is the right token.  Under the section's
 * independence assumption a node (i_1..i_k) is accepted with probability prod_j acc[j][i_j], and the expected
 * number of accepted speculated tokens of a tree is the sum of that product over its nodes.  Starting from the
 * root alone, the node with the largest product among those whose parent is already in the tree is added,
 * n_nodes - 1 times (ties: the smaller tuple in tuple_cmp order).  The product is formed left to right in double.
 * paths_out: [n_nodes-1][depth] in the order the nodes were added, -1 padded.  *expect_out (nullable): the sum.
 * Returns the number of paths or -1 (bad sizes, an accuracy outside [0, 1] or not a number, tree too large).
 */
int32_t ora_tree_paths_from_accuracies(const double *acc, int32_t depth, int32_t topk, int32_t n_nodes,
                                       int32_t *paths_out, double *expect_out)
{
    if (!acc || !paths_out || depth < 1 || depth > ORA_MAX_DEPTH || topk < 1 || n_nodes < 1 || n_nodes > ORA_MAX_T)
        return -1;
    for (int i = 0; i < depth * topk; ++i)
        if (!(acc[i] >= 0.0 && acc[i] <= 1.0))
            return -1;
    double total = 0.0, level = 1.0;
    for (int k = 0; k < depth; ++k) {
        level *= (double)topk;
        total += level;
    }
    if ((double)(n_nodes - 1) > total)
        return -1;
    int32_t tree[ORA_MAX_T][ORA_MAX_DEPTH]; /* tree[0] = root (length 0) */
    int tlen[ORA_MAX_T];
    double tacc[ORA_MAX_T];
    int n = 1;
    tlen[0] = 0;
    tacc[0] = 1.0;
    double expect = 0.0;
    while (n < n_nodes) {
        int have = 0, best_len = 0;
        int32_t best[ORA_MAX_DEPTH];
        double best_acc = 0.0;
        for (int p = 0; p < n; ++p) {           /* every node already in the tree ... */
            if (tlen[p] == depth)
                continue;
            for (int32_t i = 0; i < topk; ++i) { /* ... and each of its possible children */
                int32_t c[ORA_MAX_DEPTH];
                memcpy(c, tree[p], sizeof(int32_t) * (size_t)tlen[p]);
                c[tlen[p]] = i;
                int cl = tlen[p] + 1, present = 0;
                for (int q = 0; q < n && !present; ++q)
                    present = tuple_cmp(tree[q], tlen[q], c, cl) == 0;
                if (present)
                    continue;
                double a = 1.0;
                for (int j = 0; j < cl; ++j)
                    a = a * acc[j * topk + c[j]];
                if (!have || a > best_acc || (a == best_acc && tuple_cmp(c, cl, best, best_len) < 0)) {
                    have = 1;
                    best_acc = a;
                    best_len = cl;
                    memcpy(best, c, sizeof(int32_t) * (size_t)cl);
                }
            }
        }
        if (!have)
            return -1;
        memcpy(tree[n], best, sizeof(int32_t) * (size_t)best_len);
        tlen[n] = best_len;
        tacc[n] = best_acc;
        for (int j = 0; j < depth; ++j)
            paths_out[(size_t)(n - 1) * depth + j] = j < best_len ? best[j] : -1;
        expect += best_acc;
        ++n;
    }
    (void)tacc;
    if (expect_out)
        *expect_out = expect;
    return n - 1;
}

/*
 * Static tree buffers (Sec. 2.1.2, Fig. 2).  paths: [n_paths][max_depth] rank tuples, -1 padded,
 * distinct and prefix-closed.  Node 0 is the root (the LM head's own token); the other nodes are
 * sorted by (depth, tuple).  For node i:
 *   mask[i]     bit j set iff node j is i itself or one of its ancestors (root included); ceil(T/64) words per node
 *   pos[i]      depth of i  (its rotary position is cache_len + pos[i])
 *   parent[i]   node index of the parent (-1 for the root)
 *   tree_idx[i] index into the candidate pool [root, head-1 ranks 0..topk-1, head-2 ranks ...]
 *   retrieve    one row per leaf (ascending tuple order): node indices root..leaf, -1 padded
 * dims_out = {T, P, depth, topk}.  Returns 0, or a negative code on invalid input.
 */
int32_t ora_build_tree_buffers(const int32_t *paths, int32_t n_paths, int32_t max_depth, int32_t *dims_out,
                               uint64_t *mask, int32_t *pos, int32_t *tree_idx, int32_t *parent,
                               int32_t *retrieve /* [P][depth+1], caller sizes it [T][max_depth+1] */)
{
    int T = n_paths + 1;
    if (n_paths < 0 || T > ORA_MAX_T || max_depth < 1 || max_depth > ORA_MAX_DEPTH)
        return -1;
    int order[ORA_MAX_T]; /* order[i-1] = index into paths of node i */
    int lens[ORA_MAX_T];
    for (int p = 0; p < n_paths; ++p) {
        lens[p] = tuple_len(paths + (size_t)p * max_depth, max_depth);
        if (lens[p] == 0)
            return -2;
        for (int j = lens[p]; j < max_depth; ++j)
            if (paths[(size_t)p * max_depth + j] >= 0)
                return -2; /* hole in the padding */
        order[p] = p;
    }
    /* insertion sort by (depth, tuple) */
    for (int a = 1; a < n_paths; ++a) {
        int cur = order[a], b = a - 1;
        while (b >= 0) {
            int o = order[b];
            int c = lens[o] != lens[cur] ? (lens[o] < lens[cur] ? -1 : 1)
                                         : tuple_cmp(paths + (size_t)o * max_depth, lens[o],
                                                     paths + (size_t)cur * max_depth, lens[cur]);
            if (c <= 0)
                break;
            order[b + 1] = o;
            --b;
        }
        order[b + 1] = cur;
    }
    int depth = 0, topk = 0;
    const int W = mask_words(T);
    memset(mask, 0, (size_t)T * W * sizeof(uint64_t));
    mask_set(mask, W, 0, 0);
    pos[0] = 0;
    parent[0] = -1;
    tree_idx[0] = 0;
    for (int i = 1; i < T; ++i) {
        const int32_t *ti = paths + (size_t)order[i - 1] * max_depth;
        int li = lens[order[i - 1]];
        if (i > 1) {
            const int32_t *tp = paths + (size_t)order[i - 2] * max_depth;
            if (lens[order[i - 2]] == li && tuple_cmp(tp, li, ti, li) == 0)
                return -3; /* duplicate */
        }
        if (li > depth)
            depth = li;
        for (int j = 0; j < li; ++j)
            if (ti[j] + 1 > topk)
                topk = ti[j] + 1;
        pos[i] = li;
    }
    for (int i = 1; i < T; ++i) {
        const int32_t *ti = paths + (size_t)order[i - 1] * max_depth;
        int li = lens[order[i - 1]];
        mask_set(mask, W, i, 0);
        mask_set(mask, W, i, i);
        int par = li == 1 ? 0 : -1;
        for (int j = 1; j < i; ++j) {
            const int32_t *tj = paths + (size_t)order[j - 1] * max_depth;
            int lj = lens[order[j - 1]];
            if (lj < li && tuple_cmp(tj, lj, ti, lj) == 0) { /* tj is a proper prefix of ti */
                mask_set(mask, W, i, j);
                if (lj == li - 1)
                    par = j;
            }
        }
        if (par < 0)
            return -4; /* not prefix-closed */
        parent[i] = par;
        tree_idx[i] = 1 + (li - 1) * topk + ti[li - 1];
    }
    /* leaves in ascending tuple order */
    int leaves[ORA_MAX_T], P = 0;
    for (int i = 0; i < T; ++i) {
        int has_child = 0;
        for (int j = 1; j < T; ++j)
            if (parent[j] == i)
                has_child = 1;
        if (!has_child)
            leaves[P++] = i;
    }
    for (int a = 1; a < P; ++a) {
        int cur = leaves[a], b = a - 1;
        while (b >= 0) {
            int o = leaves[b];
            int c = (o == 0 || cur == 0)
                        ? 0
                        : tuple_cmp(paths + (size_t)order[o - 1] * max_depth, lens[order[o - 1]],
                                    paths + (size_t)order[cur - 1] * max_depth, lens[order[cur - 1]]);
            if (c <= 0)
                break;
            leaves[b + 1] = o;
            --b;
        }
        leaves[b + 1] = cur;
    }
    for (int r = 0; r < P; ++r) {
        int chain[ORA_MAX_DEPTH + 1], n = 0;
        for (int v = leaves[r]; v >= 0; v = parent[v])
            chain[n++] = v;
        for (int j = 0; j <= depth; ++j)
            retrieve[(size_t)r * (depth + 1) + j] = j < n ? chain[n - 1 - j] : -1;
    }
    dims_out[0] = T;
    dims_out[1] = P;
    dims_out[2] = depth;
    dims_out[3] = topk;
    return 0;
}

/* ------------------------------------------------------------------ heads, top-k, candidates */

/*
 * Medusa heads (Sec. 2.1.1): for k = 1..K,  x_k = h + SiLU(W1_k h),  z_k = W2_k x_k.
 * W1: [K][d][d] (out x in), W2: [K][V][d].  The softmax is omitted: ranking is monotone in z.
 * x_out [K][d] and logits_out [K][V] are doubles.
 */
void ora_medusa_heads(const double *h, const void *W1, const void *W2, int32_t wdtype, int32_t K, int32_t d, int32_t V,
                      double *x_out, double *logits_out)
{
    double *u = (double *)malloc((size_t)d * sizeof(double));
    for (int k = 0; k < K; ++k) {
        const char *w1 = (const char *)W1 + (size_t)k * d * d * (wdtype ? 2 : 4);
        const char *w2 = (const char *)W2 + (size_t)k * V * d * (wdtype ? 2 : 4);
        linear(w1, wdtype, d, d, h, 1, d, u, d);
        for (int i = 0; i < d; ++i)
            x_out[(size_t)k * d + i] = h[i] + silu(u[i]);
        linear(w2, wdtype, V, d, x_out + (size_t)k * d, 1, d, logits_out + (size_t)k * V, V);
    }
    free(u);
}

/* indices of the k largest values, ordered by (value descending, index ascending); compares only */
void ora_topk(const float *v, int32_t n, int32_t k, int32_t *idx_out)
{
    for (int r = 0; r < k; ++r) {
        int best = -1;
        for (int i = 0; i < n; ++i) {
            int taken = 0;
            for (int q = 0; q < r; ++q)
                if (idx_out[q] == i)
                    taken = 1;
            if (taken)
                continue;
            if (best < 0 || v[i] > v[best])
                best = i;
        }
        idx_out[r] = best;
    }
}

/* Candidate pool = [root, head-1 top-`topk`, head-2 top-`topk`, ...]; tree_tok[i] = pool[tree_idx[i]];
 * cand[r][j] = tree_tok[retrieve[r][j]] (or -1 where the row is padded). */
void ora_expand_candidates(int32_t root, const int32_t *topk_idx /* [K][topk] */, int32_t topk, const int32_t *tree_idx,
                           int32_t T, const int32_t *retrieve, int32_t P, int32_t depth, int32_t *tree_tok,
                           int32_t *cand)
{
    for (int i = 0; i < T; ++i)
        tree_tok[i] = tree_idx[i] == 0 ? root : topk_idx[tree_idx[i] - 1];
    if (cand)
        for (int r = 0; r < P; ++r)
            for (int j = 0; j <= depth; ++j) {
                int nd = retrieve[(size_t)r * (depth + 1) + j];
                cand[(size_t)r * (depth + 1) + j] = nd < 0 ? -1 : tree_tok[nd];
            }
}

/* ------------------------------------------------------------------ tree attention */

/*
 * Tree attention for one layer (Sec. 2.1.2; App. G Table 5).  All arrays double.
 *   q, k_new, v_new : [T][H][D]  (already rotated)
 *   kc, vc          : [H][L_max][D], positions 0..L-1 valid (keys stored rotated)
 * Query i of head h sees every cache position 0..L-1 and then, in index order, the tree nodes
 * j with bit j of mask row i set (its ancestors and itself; ceil(T/64) words per row).  out[i][h] = softmax(q.k/sqrt(D)) V.
 * lse (nullable): [T][H] log-sum-exp of the scaled scores.
 */
static void tree_attention_core(const double *q, const double *k_new, const double *v_new, const double *kc,
                                const double *vc, int T, int H, int Hkv, int D, int L, int L_max, const uint64_t *mask,
                                double *out, double *lse)
{
    /* grouped-query attention: query head h reads key/value head h / (H / Hkv); Hkv == H is the ordinary case */
    const int group = H / Hkv;
    const int W = mask_words(T);
    double scale = 1.0 / sqrt((double)D);
#pragma omp parallel for collapse(2) schedule(static)
    for (int h = 0; h < H; ++h) {
        for (int i = 0; i < T; ++i) {
            int nk = L + T;
            double *s = (double *)malloc((size_t)nk * sizeof(double));
            const double *qi = q + ((size_t)i * H + h) * D;
            const int hk = h / group;
            double m = -INFINITY;
            for (int j = 0; j < nk; ++j) {
                int visible = j < L || mask_bit(mask, W, i, j - L);
                if (!visible) {
                    s[j] = -INFINITY;
                    continue;
                }
                const double *kj = j < L ? kc + ((size_t)hk * L_max + j) * D : k_new + ((size_t)(j - L) * Hkv + hk) * D;
                double acc = 0.0;
                for (int e = 0; e < D; ++e)
                    acc += qi[e] * kj[e];
                s[j] = acc * scale;
                if (s[j] > m)
                    m = s[j];
            }
            double den = 0.0;
            for (int j = 0; j < nk; ++j) {
                s[j] = s[j] == -INFINITY ? 0.0 : exp(s[j] - m);
                den += s[j];
            }
            double *o = out + ((size_t)i * H + h) * D;
            for (int e = 0; e < D; ++e) {
                double acc = 0.0;
                for (int j = 0; j < nk; ++j) {
                    if (s[j] == 0.0)
                        continue;
                    const double *vj =
                        j < L ? vc + ((size_t)hk * L_max + j) * D : v_new + ((size_t)(j - L) * Hkv + hk) * D;
                    acc += s[j] * vj[e];
                }
                o[e] = acc / den;
            }
            if (lse)
                lse[(size_t)i * H + h] = m + log(den);
            free(s);
        }
    }
}

/*
 * Stand-alone operator on float32 inputs.  If apply_rope != 0, q[i] and k_new[i] are rotated at
 * position L + pos[i] first (cache keys are taken as already rotated).  out: [T][H][D] doubles.
 */
void ora_tree_attention(const float *q, const float *k_new, const float *v_new, const float *k_cache,
                        const float *v_cache, int32_t T, int32_t H, int32_t Hkv, int32_t D, int32_t L, int32_t L_max,
                        const uint64_t *mask, const int32_t *pos, int32_t apply_rope, double rope_theta, double *out,
                        double *lse)
{
    /* q: [T][H][D]; k_new, v_new: [T][Hkv][D]; caches: [Hkv][L_max][D] */
    size_t nq = (size_t)T * H * D, nk = (size_t)T * Hkv * D, nc = (size_t)Hkv * L_max * D;
    double *qd = (double *)malloc(nq * sizeof(double)), *kd = (double *)malloc(nk * sizeof(double));
    double *vd = (double *)malloc(nk * sizeof(double));
    double *kcd = (double *)malloc((nc ? nc : 1) * sizeof(double)), *vcd = (double *)malloc((nc ? nc : 1) * sizeof(double));
    for (size_t i = 0; i < nq; ++i)
        qd[i] = q[i];
    for (size_t i = 0; i < nk; ++i) {
        kd[i] = k_new[i];
        vd[i] = v_new[i];
    }
    for (size_t i = 0; i < nc; ++i) {
        kcd[i] = k_cache[i];
        vcd[i] = v_cache[i];
    }
    if (apply_rope)
        for (int i = 0; i < T; ++i) {
            for (int h = 0; h < H; ++h)
                rope(qd + ((size_t)i * H + h) * D, D, (int64_t)L + pos[i], rope_theta);
            for (int h = 0; h < Hkv; ++h)
                rope(kd + ((size_t)i * Hkv + h) * D, D, (int64_t)L + pos[i], rope_theta);
        }
    tree_attention_core(qd, kd, vd, kcd, vcd, T, H, Hkv, D, L, L_max, mask, out, lse);
    free(qd);
    free(kd);
    free(vd);
    free(kcd);
    free(vcd);
}

/* ------------------------------------------------------------------ backbone */

typedef struct {
    int32_t n_layers, d, n_heads, head_dim, ffn, vocab, n_medusa, wdtype; /* wdtype 0 f32, 1 bf16 bits */
    int32_t n_kv_heads;  /* key/value heads (grouped-query attention); 0 means n_heads */
    int32_t kv_bf16;     /* != 0: every pass holds its tree keys (after rotation) and values as a bfloat16 KV cache holds
                          * them (a property of the workload's storage, see layer_forward); 0: unrounded */
    double rms_eps, rope_theta;
    const void *embed;        /* [V][d] */
    const void *final_norm;   /* [d] */
    const void *lm_head;      /* [V][d] */
    const void *const *layers; /* n_layers*9: attn_norm[d], wq[H*D][d], wk[Hkv*D][d], wv[Hkv*D][d], wo[d][H*D], ffn_norm[d], w_gate[F][d], w_up[F][d], w_down[d][F] */
    const void *medusa_w1;    /* [K][d][d] */
    const void *medusa_w2;    /* [K][V][d] */
} ora_model;

static inline int kv_heads(const void *model)
{
    const ora_model *m = (const ora_model *)model;
    return m->n_kv_heads > 0 ? m->n_kv_heads : m->n_heads;
}

/*
 * One backbone pass over T tree tokens against a cache of length L (App. G Table 5, "parallel decoding"):
 * pre-norm Llama block  x += Wo Attn(RMSNorm(x));  x += Wd (SiLU(Wg n) * (Wu n)), n = RMSNorm(x);
 * final RMSNorm; LM head.  K/V of tree node i are computed at rotary position L + pos[i].
 *   kc, vc        : [N_L][H][L_max][D] doubles (read only)
 *   tree_k,tree_v : [N_L][T][H][D] doubles (written: this pass's rotated K and V)
 *   hidden        : [T][d]  final-norm output (the LM head's input, and the Medusa heads' input)
 *   logits        : [T][V]  (nullable)
 */
/* A value as a bfloat16 store holds it: rounded to float, then to the nearest bfloat16 (ties to even). */
static double round_bf16(double v)
{
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7f800000u) == 0x7f800000u)
        return (double)f; /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Scratch of one layer evaluation. */
typedef struct {
    double *n, *q, *att, *o, *g, *u;
} layer_scratch;

static void layer_scratch_alloc(layer_scratch *s, int T, int d, int hd, int F)
{
    s->n = (double *)malloc((size_t)T * d * sizeof(double));
    s->q = (double *)malloc((size_t)T * hd * sizeof(double));
    s->att = (double *)malloc((size_t)T * hd * sizeof(double));
    s->o = (double *)malloc((size_t)T * d * sizeof(double));
    s->g = (double *)malloc((size_t)T * F * sizeof(double));
    s->u = (double *)malloc((size_t)T * F * sizeof(double));
}

static void layer_scratch_free(layer_scratch *s)
{
    free(s->n); free(s->q); free(s->att); free(s->o); free(s->g); free(s->u);
}

/*
 * One pre-norm Llama block on T tree tokens (App. G Table 5, "parallel decoding"), in place on x [T][d]:
 *   x += Wo Attn(RMSNorm(x));  x += Wd (SiLU(Wg n) * (Wu n)), n = RMSNorm(x).
 * kc, vc: this layer's cache [Hkv][L_max][D]; tk, tv: this layer's rotated tree keys and values [T][Hkv][D] (written).
 * kv_bf16 != 0: the tree keys (after rotation) and values are held as a bfloat16 KV cache holds them -- the rounding
 * belongs to the workload's definition of its cache storage, not to the method.  The attention output is left in
 * s->att.
 */
static void layer_forward(const ora_model *m, int l, double *x, const uint64_t *mask, const int32_t *pos, int T, int L,
                          int L_max, const double *kc, const double *vc, double *tk, double *tv, int kv_bf16,
                          layer_scratch *s)
{
    int d = m->d, H = m->n_heads, Hkv = kv_heads(m), D = m->head_dim, F = m->ffn, dt = m->wdtype;
    int hd = H * D, hkd = Hkv * D;
    const void *const *w = m->layers + (size_t)l * 9;
    double *n = s->n, *q = s->q, *att = s->att, *o = s->o, *g = s->g, *u = s->u;
    for (int t = 0; t < T; ++t)
        rmsnorm(x + (size_t)t * d, w[0], dt, d, m->rms_eps, n + (size_t)t * d);
    linear(w[1], dt, hd, d, n, T, d, q, hd);
    linear(w[2], dt, hkd, d, n, T, d, tk, hkd);
    linear(w[3], dt, hkd, d, n, T, d, tv, hkd);
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h)
            rope(q + ((size_t)t * H + h) * D, D, (int64_t)L + pos[t], m->rope_theta);
        for (int h = 0; h < Hkv; ++h)
            rope(tk + ((size_t)t * Hkv + h) * D, D, (int64_t)L + pos[t], m->rope_theta);
    }
    if (kv_bf16)
        for (size_t i = 0; i < (size_t)T * hkd; ++i) {
            tk[i] = round_bf16(tk[i]);
            tv[i] = round_bf16(tv[i]);
        }
    tree_attention_core(q, tk, tv, kc, vc, T, H, Hkv, D, L, L_max, mask, att, NULL);
    linear(w[4], dt, d, hd, att, T, hd, o, d);
    for (size_t i = 0; i < (size_t)T * d; ++i)
        x[i] += o[i];
    for (int t = 0; t < T; ++t)
        rmsnorm(x + (size_t)t * d, w[5], dt, d, m->rms_eps, n + (size_t)t * d);
    linear(w[6], dt, F, d, n, T, d, g, F);
    linear(w[7], dt, F, d, n, T, d, u, F);
    for (size_t i = 0; i < (size_t)T * F; ++i)
        g[i] = silu(g[i]) * u[i];
    linear(w[8], dt, d, F, g, T, F, o, d);
    for (size_t i = 0; i < (size_t)T * d; ++i)
        x[i] += o[i];
}

void ora_tree_pass(const ora_model *m, const int32_t *tokens, const uint64_t *mask, const int32_t *pos, int32_t T,
                   int32_t L, int32_t L_max, const double *kc, const double *vc, double *tree_k, double *tree_v,
                   double *hidden, double *logits)
{
    int d = m->d, H = m->n_heads, Hkv = kv_heads(m), D = m->head_dim, F = m->ffn, dt = m->wdtype;
    int hd = H * D, hkd = Hkv * D;
    double *x = (double *)malloc((size_t)T * d * sizeof(double));
    layer_scratch s;
    layer_scratch_alloc(&s, T, d, hd, F);
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < d; ++i)
            x[(size_t)t * d + i] = wget(m->embed, (size_t)tokens[t] * d + i, dt);
    for (int l = 0; l < m->n_layers; ++l)
        layer_forward(m, l, x, mask, pos, T, L, L_max, kc + (size_t)l * Hkv * L_max * D, vc + (size_t)l * Hkv * L_max * D,
                      tree_k + (size_t)l * T * hkd, tree_v + (size_t)l * T * hkd, m->kv_bf16, &s);
    for (int t = 0; t < T; ++t)
        rmsnorm(x + (size_t)t * d, m->final_norm, dt, d, m->rms_eps, hidden + (size_t)t * d);
    if (logits)
        linear(m->lm_head, dt, m->vocab, d, hidden, T, d, logits, m->vocab);
    free(x);
    layer_scratch_free(&s);
}

/*
 * Layer l alone on a given layer input (the same code the pass above runs): x [T][d] in/out, att_out [T][H*D]
 * (nullable) receives the attention output, kc/vc are THIS layer's cache [Hkv][L_max][D], tk/tv [T][Hkv][D] are written.
 * Used to check an implementation layer by layer on that implementation's own layer inputs and cache.
 */
void ora_layer(const ora_model *m, int32_t l, double *x, const uint64_t *mask, const int32_t *pos, int32_t T, int32_t L,
               int32_t L_max, const double *kc, const double *vc, double *tk, double *tv, int32_t kv_bf16, double *att_out)
{
    layer_scratch s;
    layer_scratch_alloc(&s, T, m->d, m->n_heads * m->head_dim, m->ffn);
    layer_forward(m, l, x, mask, pos, T, L, L_max, kc, vc, tk, tv, kv_bf16, &s);
    if (att_out)
        memcpy(att_out, s.att, (size_t)T * m->n_heads * m->head_dim * sizeof(double));
    layer_scratch_free(&s);
}

/* The closing steps of a pass on a given residual stream x [T][d]: hidden = final RMSNorm(x) (nullable out), then the
 * LM head on `hidden_in` if that is given, else on the hidden just computed; logits [T][V] (nullable). */
void ora_final_norm_lm_head(const ora_model *m, const double *x, const double *hidden_in, int32_t T, double *hidden,
                            double *logits)
{
    int d = m->d;
    double *hn = (double *)malloc((size_t)T * d * sizeof(double));
    if (x)
        for (int t = 0; t < T; ++t)
            rmsnorm(x + (size_t)t * d, m->final_norm, m->wdtype, d, m->rms_eps, hn + (size_t)t * d);
    if (hidden && x)
        memcpy(hidden, hn, (size_t)T * d * sizeof(double));
    if (logits)
        linear(m->lm_head, m->wdtype, m->vocab, d, hidden_in ? hidden_in : hn, T, d, logits, m->vocab);
    free(hn);
}

/* ------------------------------------------------------------------ acceptance */

static int argmax_f(const float *v, int n)
{
    int b = 0;
    for (int i = 1; i < n; ++i)
        if (v[i] > v[b])
            b = i;
    return b;
}

/*
 * Acceptance (Sec. 2.3.1; Fig. 1 "longest accepted candidate prefix").  logits: [T][V] float32.
 * For each retrieve row r and depth j >= 1 with node c = r[j] and parent p = r[j-1]:
 *   mode 0 (greedy) : ok iff tree_tok[c] == argmax logits[p]          (ties -> lower index)
 *   mode 1 (typical): with l = logits[p]/tau, P = softmax(l), Hn = entropy(P) in nats,
 *                     ok iff P[tree_tok[c]] > min(eps, delta * exp(-Hn))   (strict)
 * tau <= 0 selects greedy.  The accepted length of a row is its number of leading ok's; accept_len is
 * the maximum over rows, best the lowest row attaining it, acc_nodes = retrieve[best][0..accept_len]
 * (-1 beyond).  The next root is the greedy token after the last accepted node (the paper's
 * unconditionally accepted first token): argmax logits[last]; or, if gumbel != NULL, the Gumbel-max
 * sample argmax_v fl32(fl32(logits[last][v] * inv_tau) + gumbel[v]) with inv_tau = fl32(1/tau).
 * min_margin (nullable): smallest |P - thr| / thr over all typical decisions taken (conditioning report).
 */
/*
 * One typical-acceptance decision (Sec. 2.3.1): with l = row/tau, P = softmax(l) and Hn its entropy in nats,
 * the candidate token passes iff P[token] > min(eps, delta * exp(-Hn)) (strict).  The three quantities of the
 * criterion are returned so that hand-worked vectors can pin each of them, not only the decision.
 */
static int typical_decision(const float *lp, int V, double tau, double eps, double delta, int token, double *p_out,
                            double *ent_out, double *thr_out)
{
    double mx = -INFINITY;
    for (int v = 0; v < V; ++v) {
        double l = (double)lp[v] / tau;
        if (l > mx)
            mx = l;
    }
    double se = 0.0;
    for (int v = 0; v < V; ++v)
        se += exp((double)lp[v] / tau - mx);
    double lse = mx + log(se);
    double ent = 0.0; /* H = -sum p log p */
    for (int v = 0; v < V; ++v) {
        double l = (double)lp[v] / tau;
        double pv = exp(l - lse);
        if (pv > 0.0)
            ent -= pv * (l - lse);
    }
    double pc = exp((double)lp[token] / tau - lse);
    double thr = fmin(eps, delta * exp(-ent));
    *p_out = pc;
    *ent_out = ent;
    *thr_out = thr;
    return pc > thr;
}

/* The same decision for one logits row, exported for the pins: returns 1 if `token` passes. */
int32_t ora_typical_decision(const float *row, int32_t V, double tau, double eps, double delta, int32_t token,
                             double *p_out, double *entropy_out, double *threshold_out)
{
    return typical_decision(row, V, tau, eps, delta, token, p_out, entropy_out, threshold_out);
}

void ora_evaluate_posterior(const float *logits, int32_t V, const int32_t *tree_tok, const int32_t *retrieve, int32_t P,
                            int32_t depth, int32_t mode, double tau, double eps, double delta, const float *gumbel,
                            int32_t *best, int32_t *accept_len, int32_t *next_root, int32_t *acc_nodes,
                            double *min_margin)
{
    int W = depth + 1;
    int best_r = 0, best_len = -1;
    double mm = INFINITY;
    if (tau <= 0.0)
        mode = 0;
    for (int r = 0; r < P; ++r) {
        int len = 0;
        for (int j = 1; j < W; ++j) {
            int c = retrieve[(size_t)r * W + j];
            if (c < 0)
                break;
            int p = retrieve[(size_t)r * W + j - 1];
            const float *lp = logits + (size_t)p * V;
            int ok;
            if (mode == 0) {
                ok = tree_tok[c] == argmax_f(lp, V);
            } else {
                double pc, ent, thr;
                ok = typical_decision(lp, V, tau, eps, delta, tree_tok[c], &pc, &ent, &thr);
                if (thr > 0.0) {
                    double mg = fabs(pc - thr) / thr;
                    if (mg < mm)
                        mm = mg;
                }
            }
            if (!ok)
                break;
            ++len;
        }
        if (len > best_len) {
            best_len = len;
            best_r = r;
        }
    }
    *best = best_r;
    *accept_len = best_len;
    for (int j = 0; j < W; ++j)
        acc_nodes[j] = j <= best_len ? retrieve[(size_t)best_r * W + j] : -1;
    const float *ll = logits + (size_t)acc_nodes[best_len] * V;
    if (gumbel && tau > 0.0) {
        float inv_tau = (float)(1.0 / tau);
        int b = 0;
        float bs = 0.f;
        for (int v = 0; v < V; ++v) {
            volatile float sc = ll[v] * inv_tau; /* volatile: one rounding per operation, no fused multiply-add */
            volatile float s = sc + gumbel[v];
            if (v == 0 || s > bs) {
                bs = s;
                b = v;
            }
        }
        *next_root = b;
    } else {
        *next_root = argmax_f(ll, V);
    }
    if (min_margin)
        *min_margin = mm;
}

/*
 * Rejection-sampling acceptance (Sec. 1 and Sec. 2.3.1, first paragraph: the rejection sampling scheme of
 * speculative decoding can be reused so that the output follows the original model's distribution).  The paper
 * gives no algorithm for its candidate tree; the reading taken here is speculative sampling with the tree's
 * candidates as DETERMINISTIC drafts (they are top-k picks, not samples, so a draft's proposal distribution is a
 * point mass q = 1 on its token):
 *   at node n with P = softmax(logits[n] / tau), its children c_1, c_2, ... in node order, R = 0:
 *     child c_i with token x_i is accepted iff uniform[c_i] < P[x_i] / (1 - R)       (min(1, P/q) of the residual)
 *     otherwise x_i is struck out, R += P[x_i], and the next sibling is tried against the renormalised residual;
 *   an accepted child becomes n; when every child of n was rejected (or n is a leaf) the next token is drawn from
 *   the residual of n: the Gumbel-max sample argmax_v fl32(fl32(logits[n][v] * inv_tau) + gumbel[v]) over the
 *   tokens v that were not struck out at n (ties -> lower index).
 * Each emitted token then has exactly the backbone's sampling distribution: P(x_i emitted) =
 * prod_{j<i} (1 - a_j) * a_i = P[x_i], and a token outside the children keeps its mass P[v].
 * uniform: [T] numbers in [0, 1), one per node (the entry of a node is used when that node is tried).
 * Outputs as ora_evaluate_posterior; best = the lowest retrieve row that starts with the accepted path;
 * rejected_tok (nullable, [T]) / n_rejected: the tokens struck out at the last node;
 * min_margin (nullable): smallest |u - a| / a over the decisions taken.  Requires tau > 0.
 */
void ora_evaluate_rejection(const float *logits, int32_t V, const int32_t *tree_tok, const int32_t *parent, int32_t T,
                            const int32_t *retrieve, int32_t P, int32_t depth, double tau, const float *gumbel,
                            const float *uniform, int32_t *best, int32_t *accept_len, int32_t *next_root,
                            int32_t *acc_nodes, int32_t *rejected_tok, int32_t *n_rejected, double *min_margin)
{
    int W = depth + 1;
    int n = 0, len = 0, nrej = 0;
    double mm = INFINITY;
    int32_t *rej = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    acc_nodes[0] = 0;
    for (;;) {
        const float *lp = logits + (size_t)n * V;
        double mx = -INFINITY;
        for (int v = 0; v < V; ++v) {
            double l = (double)lp[v] / tau;
            if (l > mx)
                mx = l;
        }
        double se = 0.0;
        for (int v = 0; v < V; ++v)
            se += exp((double)lp[v] / tau - mx);
        double lse = mx + log(se);
        double R = 0.0;
        int accepted = -1;
        nrej = 0;
        for (int c = 0; c < T; ++c) {
            if (c == n || parent[c] != n)
                continue;
            double pc = exp((double)lp[tree_tok[c]] / tau - lse);
            double rem = 1.0 - R;
            double a = rem > 0.0 ? pc / rem : 1.0;
            double u = (double)uniform[c];
            if (a > 0.0) {
                double mg = fabs(u - a) / a;
                if (mg < mm)
                    mm = mg;
            }
            if (u < a) {
                accepted = c;
                break;
            }
            R += pc;
            rej[nrej++] = tree_tok[c];
        }
        if (accepted < 0)
            break;
        n = accepted; /* a tree of this depth has no node deeper than W - 1, so len stays below W */
        acc_nodes[++len] = n;
    }
    for (int j = len + 1; j < W; ++j)
        acc_nodes[j] = -1;
    *accept_len = len;
    int b = 0;
    for (int r = 0; r < P; ++r) {
        int same = 1;
        for (int j = 0; j <= len; ++j)
            if (retrieve[(size_t)r * W + j] != acc_nodes[j]) {
                same = 0;
                break;
            }
        if (same) {
            b = r;
            break;
        }
    }
    *best = b;
    {
        const float *ll = logits + (size_t)n * V;
        float inv_tau = (float)(1.0 / tau);
        int bi = -1;
        float bs = 0.f;
        for (int v = 0; v < V; ++v) {
            int struck = 0;
            for (int q = 0; q < nrej; ++q)
                if (rej[q] == v)
                    struck = 1;
            if (struck)
                continue;
            volatile float sc = ll[v] * inv_tau; /* one rounding per operation, no fused multiply-add */
            volatile float s = sc + gumbel[v];
            if (bi < 0 || s > bs) {
                bs = s;
                bi = v;
            }
        }
        *next_root = bi < 0 ? 0 : bi;
    }
    if (rejected_tok)
        for (int q = 0; q < nrej; ++q)
            rejected_tok[q] = rej[q];
    if (n_rejected)
        *n_rejected = nrej;
    if (min_margin)
        *min_margin = mm;
    free(rej);
}

/*
 * Commit the accepted path.  n_commit = min(1 + accept_len, max_commit).  For every layer, K and V:
 * cache[L + j] <- tree[acc_nodes[j]], j = 0..n_commit-1;  emitted[j] = tree_tok[acc_nodes[j]];
 * h_last <- hidden[acc_nodes[n_commit-1]];  returns the new cache length L + n_commit, or -1 if that
 * would exceed L_max (nothing is written then).  moved_src/moved_dst (nullable, [depth+1]): the absolute
 * positions L + acc_nodes[j] -> L + j ("gathered KV positions").
 */
int32_t ora_accept_and_update_kv(int32_t n_layers, int32_t H, int32_t D, int32_t T, int32_t L_max, const double *tree_k,
                                 const double *tree_v, double *kc, double *vc, const int32_t *acc_nodes,
                                 int32_t accept_len, int32_t max_commit, int32_t L, const double *hidden, int32_t d,
                                 double *h_last, const int32_t *tree_tok, int32_t *emitted, int32_t *n_emitted,
                                 int32_t *moved_src, int32_t *moved_dst)
{
    int n = 1 + accept_len;
    if (n > max_commit)
        n = max_commit;
    if (n < 0)
        n = 0;
    if (L + n > L_max)
        return -1;
    for (int l = 0; l < n_layers; ++l)
        for (int j = 0; j < n; ++j)
            for (int h = 0; h < H; ++h) {
                size_t dst = (((size_t)l * H + h) * L_max + (size_t)(L + j)) * D;
                size_t src = (((size_t)l * T + acc_nodes[j]) * H + h) * D;
                memcpy(kc + dst, tree_k + src, (size_t)D * sizeof(double));
                memcpy(vc + dst, tree_v + src, (size_t)D * sizeof(double));
            }
    for (int j = 0; j < n; ++j) {
        emitted[j] = tree_tok[acc_nodes[j]];
        if (moved_src)
            moved_src[j] = L + acc_nodes[j];
        if (moved_dst)
            moved_dst[j] = L + j;
    }
    *n_emitted = n;
    if (n > 0)
        memcpy(h_last, hidden + (size_t)acc_nodes[n - 1] * d, (size_t)d * sizeof(double));
    return L + n;
}

/* ------------------------------------------------------------------ drivers */

typedef struct {
    int32_t T, P, depth, topk;
    const uint64_t *mask;
    const int32_t *pos, *tree_idx, *parent, *retrieve;
} ora_tree;

static int argmax_d_as_f(const double *v, int n, float *tmp)
{
    for (int i = 0; i < n; ++i)
        tmp[i] = (float)v[i];
    return argmax_f(tmp, n);
}

/*
 * Prefill: the same pass with a chain "tree" (node i's parent is i-1, so the mask is lower-triangular
 * and the attention is ordinary causal attention), up to 64 tokens per call, every token committed.
 * Returns the cache length (= n_prompt); writes h_last [d] and *root = argmax of the last logits.
 */
static int prefill(const ora_model *m, const int32_t *prompt, int n_prompt, int L_max, double *kc, double *vc,
                   double *h_last, int32_t *root)
{
    int d = m->d, H = kv_heads(m), D = m->head_dim, V = m->vocab, NL = m->n_layers; /* H: key/value heads */
    int L = 0;
    double *tk = (double *)malloc((size_t)NL * 64 * H * D * sizeof(double));
    double *tv = (double *)malloc((size_t)NL * 64 * H * D * sizeof(double));
    double *hid = (double *)malloc((size_t)64 * d * sizeof(double));
    double *lg = (double *)malloc((size_t)64 * V * sizeof(double));
    float *tmp = (float *)malloc((size_t)V * sizeof(float));
    while (L < n_prompt) {
        int T = n_prompt - L < 64 ? n_prompt - L : 64;
        uint64_t mask[64];
        int32_t pos[64], acc[64], tok_dummy[64], emitted[64], n_em;
        for (int i = 0; i < T; ++i) {
            mask[i] = i == 63 ? ~0ull : ((1ull << (i + 1)) - 1ull);
            pos[i] = i;
            acc[i] = i;
            tok_dummy[i] = prompt[L + i];
        }
        ora_tree_pass(m, prompt + L, mask, pos, T, L, L_max, kc, vc, tk, tv, hid, lg);
        *root = argmax_d_as_f(lg + (size_t)(T - 1) * V, V, tmp);
        L = ora_accept_and_update_kv(NL, H, D, T, L_max, tk, tv, kc, vc, acc, T - 1, T, L, hid, d, h_last, tok_dummy,
                                     emitted, &n_em, NULL, NULL);
    }
    free(tk);
    free(tv);
    free(hid);
    free(lg);
    free(tmp);
    return L;
}

/*
 * Medusa decoding (Sec. 2: generate candidates -> process them with tree attention -> accept).
 * Prefill the prompt, then repeat { heads on h_last -> top-k -> tree tokens -> tree pass ->
 * acceptance -> commit } until G tokens are emitted.  out_tokens [G]; accept_hist (nullable) [G] gets
 * the number of tokens emitted per step; returns the number of steps.  gumbel (nullable): [max_steps][V]
 * noise, row s used at step s; only read when mode == 1.
 */
int32_t ora_generate(const ora_model *m, const ora_tree *tr, const int32_t *prompt, int32_t n_prompt, int32_t G,
                     int32_t L_max, int32_t mode, double tau, double eps, double delta, const float *gumbel,
                     int32_t *out_tokens, int32_t *accept_hist, double *kc_out, double *vc_out)
{
    int d = m->d, H = kv_heads(m), D = m->head_dim, V = m->vocab, NL = m->n_layers, K = m->n_medusa, T = tr->T; /* H: key/value heads */
    size_t csz = (size_t)NL * H * L_max * D;
    double *kc = kc_out ? kc_out : (double *)calloc(csz, sizeof(double));
    double *vc = vc_out ? vc_out : (double *)calloc(csz, sizeof(double));
    double *h_last = (double *)malloc((size_t)d * sizeof(double));
    double *xk = (double *)malloc((size_t)K * d * sizeof(double));
    double *hl = (double *)malloc((size_t)K * V * sizeof(double));
    float *hlf = (float *)malloc((size_t)V * sizeof(float));
    double *tk = (double *)malloc((size_t)NL * T * H * D * sizeof(double));
    double *tv = (double *)malloc((size_t)NL * T * H * D * sizeof(double));
    double *hid = (double *)malloc((size_t)T * d * sizeof(double));
    double *lg = (double *)malloc((size_t)T * V * sizeof(double));
    float *lgf = (float *)malloc((size_t)T * V * sizeof(float));
    int32_t *topk_idx = (int32_t *)malloc((size_t)K * tr->topk * sizeof(int32_t));
    int32_t tree_tok[ORA_MAX_T], acc[ORA_MAX_DEPTH + 1], emitted[ORA_MAX_DEPTH + 1];
    int32_t root, n_out = 0, steps = 0;
    int L = prefill(m, prompt, n_prompt, L_max, kc, vc, h_last, &root);
    while (n_out < G) {
        ora_medusa_heads(h_last, m->medusa_w1, m->medusa_w2, m->wdtype, K, d, V, xk, hl);
        for (int k = 0; k < K; ++k) {
            for (int v = 0; v < V; ++v)
                hlf[v] = (float)hl[(size_t)k * V + v];
            ora_topk(hlf, V, tr->topk, topk_idx + (size_t)k * tr->topk);
        }
        ora_expand_candidates(root, topk_idx, tr->topk, tr->tree_idx, T, tr->retrieve, tr->P, tr->depth, tree_tok,
                              NULL);
        ora_tree_pass(m, tree_tok, tr->mask, tr->pos, T, L, L_max, kc, vc, tk, tv, hid, lg);
        for (size_t i = 0; i < (size_t)T * V; ++i)
            lgf[i] = (float)lg[i];
        int32_t best, alen, next_root, n_em;
        ora_evaluate_posterior(lgf, V, tree_tok, tr->retrieve, tr->P, tr->depth, mode, tau, eps, delta,
                               (gumbel && mode == 1) ? gumbel + (size_t)steps * V : NULL, &best, &alen, &next_root,
                               acc, NULL);
        int max_commit = G - n_out < L_max - L ? G - n_out : L_max - L;
        if (max_commit <= 0)
            break;
        L = ora_accept_and_update_kv(NL, H, D, T, L_max, tk, tv, kc, vc, acc, alen, max_commit, L, hid, d, h_last,
                                     tree_tok, emitted, &n_em, NULL, NULL);
        for (int j = 0; j < n_em; ++j)
            out_tokens[n_out++] = emitted[j];
        if (accept_hist)
            accept_hist[steps] = n_em;
        root = next_root;
        ++steps;
    }
    if (!kc_out)
        free(kc);
    if (!vc_out)
        free(vc);
    free(h_last);
    free(xk);
    free(hl);
    free(hlf);
    free(tk);
    free(tv);
    free(hid);
    free(lg);
    free(lgf);
    free(topk_idx);
    return steps;
}

/* Plain greedy autoregressive decoding of the backbone: the same pass with T = 1 per step. */
int32_t ora_generate_plain(const ora_model *m, const int32_t *prompt, int32_t n_prompt, int32_t G, int32_t L_max,
                           int32_t *out_tokens, double *kc_out, double *vc_out)
{
    int d = m->d, H = kv_heads(m), D = m->head_dim, V = m->vocab, NL = m->n_layers; /* H: key/value heads */
    size_t csz = (size_t)NL * H * L_max * D;
    double *kc = kc_out ? kc_out : (double *)calloc(csz, sizeof(double));
    double *vc = vc_out ? vc_out : (double *)calloc(csz, sizeof(double));
    double *h_last = (double *)malloc((size_t)d * sizeof(double));
    double *tk = (double *)malloc((size_t)NL * H * D * sizeof(double));
    double *tv = (double *)malloc((size_t)NL * H * D * sizeof(double));
    double *hid = (double *)malloc((size_t)d * sizeof(double));
    double *lg = (double *)malloc((size_t)V * sizeof(double));
    float *tmp = (float *)malloc((size_t)V * sizeof(float));
    int32_t root;
    int L = prefill(m, prompt, n_prompt, L_max, kc, vc, h_last, &root);
    for (int n = 0; n < G && L < L_max; ++n) {
        uint64_t mask = 1ull;
        int32_t pos = 0, acc = 0, em, n_em;
        out_tokens[n] = root;
        ora_tree_pass(m, &root, &mask, &pos, 1, L, L_max, kc, vc, tk, tv, hid, lg);
        int32_t tok = root;
        root = argmax_d_as_f(lg, V, tmp);
        L = ora_accept_and_update_kv(NL, H, D, 1, L_max, tk, tv, kc, vc, &acc, 0, 1, L, hid, d, h_last, &tok, &em, &n_em,
                                     NULL, NULL);
    }
    if (!kc_out)
        free(kc);
    if (!vc_out)
        free(vc);
    free(h_last);
    free(tk);
    free(tv);
    free(hid);
    free(lg);
    free(tmp);
    return L;
}

/* small exported wrappers so the pins can reach the building blocks directly */
void ora_rmsnorm(const double *x, const float *g, int32_t d, double eps, double *y) { rmsnorm(x, g, 0, d, eps, y); }
void ora_rope(double *v, int32_t D, int64_t pos, double theta) { rope(v, D, pos, theta); }
double ora_silu(double u) { return silu(u); }

// Acceptance (paper Sec. 2.3.1; Fig. 1: the longest accepted candidate prefix wins) and the KV-cache commit
// of the accepted path.  Three small kernels: per-node statistics of the backbone logits (argmax; for
// typical acceptance also log-sum-exp and entropy, in double so that threshold decisions do not depend on
// the reduction order), the walk over the retrieve rows, and the 16-byte gather of accepted K/V rows.
#include "common.cuh"
#include "pdl.cuh"
#include "kernels.h"

namespace medusa {

__device__ __forceinline__ bool better_f(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// block-wide argmax with (value desc, index asc); result valid in thread 0
__device__ int block_argmax(float bv, int bi, float *sv, int *si)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better_f(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (warp == 0) {
        int nw = blockDim.x >> 5;
        bv = lane < nw ? sv[lane] : -INFINITY;
        bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (better_f(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
    }
    return bi == 0x7fffffff ? 0 : bi;  // no finite candidate (all NaN): still a valid index
}

// per-thread part of an argmax over lp[0..V): 16-byte loads, four of them in flight, when the row allows it
__device__ __forceinline__ void scan_argmax(const float *__restrict__ lp, int V, float &bv, int &bi)
{
    if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(lp) & 15u) == 0) {
        const float4 *p4 = reinterpret_cast<const float4 *>(lp);
        const int n4 = V >> 2, stride = blockDim.x;
        for (int c = threadIdx.x; c < n4; c += stride * 4) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (c + u * stride < n4) v[u] = p4[c + u * stride];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int q = c + u * stride;
                if (q < n4) {
                    const float e[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (better_f(e[k], q * 4 + k, bv, bi)) { bv = e[k]; bi = q * 4 + k; }
                }
            }
        }
    } else {
        for (int v = threadIdx.x; v < V; v += blockDim.x) {
            float x = lp[v];
            if (better_f(x, v, bv, bi)) { bv = x; bi = v; }
        }
    }
}

__device__ double block_sum_d(double v, double *sd)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) sd[warp] = v;
    __syncthreads();
    double t = 0.0;
    int nw = blockDim.x >> 5;
    for (int w = 0; w < nw; ++w)  // every thread sums the warp partials in the same order
        t += sd[w];
    return t;
}

// What one block knows about its slice of a node's logits: the best (value, index) and, for typical acceptance, the
// slice's own maximum m of x = l / tau, se = sum exp(x - m) and sx = sum exp(x - m) * x.  From these the node's
// statistics follow without another pass: with M = max m, SE = sum se * exp(m - M), SX = sum sx * exp(m - M):
// log-sum-exp = M + log SE, and the entropy H = -sum p log p = -sum p (x - lse) = lse - SX / SE.
struct NodePart {
    float bv;
    int bi;
    double m, se, sx;
};
static_assert(sizeof(NodePart) == NODE_PART_BYTES, "scratch size of the node statistics");

// grid (tree nodes, slices of the vocabulary).  Greedy acceptance (typical == 0) runs with one slice and writes the
// node's argmax directly; typical acceptance writes a NodePart per slice, merged by select_path_kernel.
__global__ void __launch_bounds__(1024)
node_stats_kernel(const float *__restrict__ logits, int V, int typical, double tau, int32_t *__restrict__ node_argmax,
                  NodePart *__restrict__ part)
{
    pdl_enter();
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ double sd[32];
    __shared__ float s_max;
    const int slices = gridDim.y, slice = blockIdx.y;
    const int chunk = (((V + slices - 1) / slices) + 3) & ~3;  // multiple of 4: slices keep the row's alignment
    const int v0 = min(V, slice * chunk), v1 = min(V, v0 + chunk);
    const float *lp = logits + (size_t)blockIdx.x * V + v0;  // this block's slice
    const int n = v1 - v0;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    scan_argmax(lp, n, bv, bi);
    const int am = block_argmax(bv, bi, sv, si);  // index inside the slice (0 if it holds no comparable value)
    if (threadIdx.x == 0)
        s_max = n > 0 ? lp[am] : -INFINITY;
    if (!typical) {
        if (threadIdx.x == 0)
            node_argmax[blockIdx.x] = v0 + am;
        return;
    }
    __syncthreads();
    const float best = s_max;
    const double mx = (double)best / tau;
    // four elements of a thread in flight at a time: the double-precision exponentials are long dependent chains
    double se4[4] = {0.0, 0.0, 0.0, 0.0}, sx4[4] = {0.0, 0.0, 0.0, 0.0};
    for (int i0 = threadIdx.x; i0 < n; i0 += 4 * blockDim.x) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * blockDim.x;
            if (i < n) {
                const double x = (double)lp[i] / tau;
                const double e = exp(x - mx);
                se4[u] += e;
                if (e > 0.0)
                    sx4[u] += e * x;  // (a term that underflowed contributes nothing, also when x is -inf)
            }
        }
    }
    const double se = block_sum_d((se4[0] + se4[1]) + (se4[2] + se4[3]), sd);
    const double sx = block_sum_d((sx4[0] + sx4[1]) + (sx4[2] + sx4[3]), sd);
    if (threadIdx.x == 0) {
        NodePart p;
        p.bv = best;
        p.bi = n > 0 && !(best != best) ? v0 + am : 0x7fffffff;
        p.m = mx;
        p.se = se;
        p.sx = sx;
        part[(size_t)blockIdx.x * slices + slice] = p;
    }
}

// one block: thread r walks retrieve row r; thread 0 picks the longest (lowest row on ties).
// rejection != 0 (rejection sampling with the candidates as deterministic drafts; needs the typical statistics):
// the block walks down from the root instead -- per level every thread evaluates p of "its" node if that node is a
// child of the current one, thread 0 tries the children in node order against the renormalised residual -- and the
// next token is the Gumbel-max sample over the tokens that were not rejected at the last node.
__global__ void __launch_bounds__(256)
select_path_kernel(PosteriorArgs a, int typical, double tau, double eps, double delta, int rejection)
{
    pdl_enter();
    __shared__ int s_len[MAX_T];
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ int s_last;
    __shared__ double s_pc[MAX_T];
    __shared__ int s_rej[MAX_T];
    __shared__ int s_nrej, s_cur, s_stop;
    const int W = a.depth + 1;
    const int r = threadIdx.x;
    if (typical && threadIdx.x < a.T) {
        // merge the vocabulary slices of node threadIdx.x (slice order, so the result does not depend on timing)
        const NodePart *p = reinterpret_cast<const NodePart *>(a.node_part) + (size_t)threadIdx.x * a.stat_slices;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        double M = -INFINITY;
        for (int q = 0; q < a.stat_slices; ++q) {
            if (better_f(p[q].bv, p[q].bi, bv, bi)) { bv = p[q].bv; bi = p[q].bi; }
            if (p[q].se > 0.0 && p[q].m > M) M = p[q].m;
        }
        double SE = 0.0, SX = 0.0;
        for (int q = 0; q < a.stat_slices; ++q)
            if (p[q].se > 0.0) {
                const double w = exp(p[q].m - M);
                SE += p[q].se * w;
                SX += p[q].sx * w;
            }
        const double lse = M + log(SE);
        a.node_argmax[threadIdx.x] = bi == 0x7fffffff ? 0 : bi;
        a.node_lse[threadIdx.x] = lse;
        a.node_ent[threadIdx.x] = lse - SX / SE;
    }
    if (typical)
        __syncthreads();  // the statistics written above are read by other threads of this (only) block
    if (rejection) {
        const int W1 = a.depth + 1;
        if (threadIdx.x == 0) {
            s_cur = 0;
            s_stop = 0;
            s_nrej = 0;
            a.acc_nodes[0] = 0;
            *a.accept_len = 0;
        }
        __syncthreads();
        int len = 0;  // kept by every thread: all of them see the same s_cur / s_stop
        for (int lvl = 0; lvl < W1; ++lvl) {
            const int n = s_cur;
            if (threadIdx.x < a.T) {
                const int cnode = threadIdx.x;
                s_pc[cnode] = cnode != n && a.parent[cnode] == n
                                  ? exp((double)a.logits[(size_t)n * a.V + a.tree_tok[cnode]] / tau - a.node_lse[n])
                                  : -1.0;  // not a child of the current node
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                double R = 0.0;
                int accepted = -1, nrej = 0;
                for (int cnode = 0; cnode < a.T; ++cnode) {
                    const double pc = s_pc[cnode];
                    if (pc < 0.0)
                        continue;
                    const double rem = 1.0 - R;
                    const double acc_p = rem > 0.0 ? pc / rem : 1.0;
                    if ((double)a.uniform[cnode] < acc_p) {
                        accepted = cnode;
                        break;
                    }
                    R += pc;
                    s_rej[nrej++] = a.tree_tok[cnode];
                }
                s_nrej = nrej;
                if (accepted < 0 || len + 1 >= W1) {
                    s_stop = 1;
                } else {
                    s_cur = accepted;
                    a.acc_nodes[len + 1] = accepted;
                }
            }
            __syncthreads();
            if (s_stop)
                break;
            ++len;
        }
        const int last_node = s_cur, nrej = s_nrej;
        if (threadIdx.x == 0) {
            *a.accept_len = len;
            for (int j = len + 1; j < W1; ++j)
                a.acc_nodes[j] = -1;
        }
        // the lowest retrieve row that starts with the accepted path
        if (r < a.P) {
            int same = 1;
            for (int j = 0; j <= len; ++j)
                same &= a.retrieve[r * W1 + j] == (j == 0 ? 0 : a.acc_nodes[j]);
            s_len[r] = same;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int b = 0;
            for (int q = 0; q < a.P; ++q)
                if (s_len[q]) { b = q; break; }
            *a.best = b;
        }
        // Gumbel-max over the tokens that were not struck out at the last node
        const float inv_tau = (float)(1.0 / tau);
        const float *lp = a.logits + (size_t)last_node * a.V;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int v = threadIdx.x; v < a.V; v += blockDim.x) {
            bool struck = false;
            for (int q = 0; q < nrej; ++q)
                struck |= s_rej[q] == v;
            if (struck)
                continue;
            const float sc = __fadd_rn(__fmul_rn(lp[v], inv_tau), a.gumbel[v]);
            if (better_f(sc, v, bv, bi)) { bv = sc; bi = v; }
        }
        const int am = block_argmax(bv, bi, sv, si);
        if (threadIdx.x == 0)
            *a.next_root = am;
        return;
    }
    if (r < a.P) {
        int len = 0;
        for (int j = 1; j < W; ++j) {
            int c = a.retrieve[r * W + j];
            if (c < 0)
                break;
            int p = a.retrieve[r * W + j - 1];
            bool ok;
            if (!typical) {
                ok = a.tree_tok[c] == a.node_argmax[p];
            } else {
                double pc = exp((double)a.logits[(size_t)p * a.V + a.tree_tok[c]] / tau - a.node_lse[p]);
                double thr = fmin(eps, delta * exp(-a.node_ent[p]));
                ok = pc > thr;
            }
            if (!ok)
                break;
            ++len;
        }
        s_len[r] = len;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0, bl = -1;
        for (int q = 0; q < a.P; ++q)
            if (s_len[q] > bl) { bl = s_len[q]; best = q; }
        *a.best = best;
        *a.accept_len = bl;
        for (int j = 0; j < W; ++j)
            a.acc_nodes[j] = j <= bl ? a.retrieve[best * W + j] : -1;
        s_last = a.retrieve[best * W + bl];
    }
    __syncthreads();
    const int last = s_last;
    if (a.gumbel != nullptr && typical) {
        // Gumbel-max sample of softmax(logits/tau): one float multiply, one float add, never fused
        const float inv_tau = (float)(1.0 / tau);
        const float *lp = a.logits + (size_t)last * a.V;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        if ((a.V & 3) == 0 && ((reinterpret_cast<uintptr_t>(lp) | reinterpret_cast<uintptr_t>(a.gumbel)) & 15u) == 0) {
            // 16-byte loads of both rows, four of each in flight per thread
            const float4 *l4 = reinterpret_cast<const float4 *>(lp), *g4 = reinterpret_cast<const float4 *>(a.gumbel);
            const int n4 = a.V >> 2, stride = blockDim.x;
            for (int c = threadIdx.x; c < n4; c += stride * 4) {
                float4 x[4], y[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (c + u * stride < n4) { x[u] = l4[c + u * stride]; y[u] = g4[c + u * stride]; }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = c + u * stride;
                    if (q < n4) {
                        const float xs[4] = {x[u].x, x[u].y, x[u].z, x[u].w}, ys[4] = {y[u].x, y[u].y, y[u].z, y[u].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float sc = __fadd_rn(__fmul_rn(xs[k], inv_tau), ys[k]);
                            if (better_f(sc, q * 4 + k, bv, bi)) { bv = sc; bi = q * 4 + k; }
                        }
                    }
                }
            }
        } else {
            for (int v = threadIdx.x; v < a.V; v += blockDim.x) {
                float sc = __fadd_rn(__fmul_rn(lp[v], inv_tau), a.gumbel[v]);
                if (better_f(sc, v, bv, bi)) { bv = sc; bi = v; }
            }
        }
        int am = block_argmax(bv, bi, sv, si);
        if (threadIdx.x == 0)
            *a.next_root = am;
    } else if (threadIdx.x == 0) {
        *a.next_root = a.node_argmax[last];
    }
}

void launch_evaluate_posterior(const PosteriorArgs &a, cudaStream_t s)
{
    const int rejection = (a.mode == MEDUSA_REJECTION && a.temperature > 0.f) ? 1 : 0;
    int typical = ((a.mode == MEDUSA_TYPICAL && a.temperature > 0.f) || rejection) ? 1 : 0;
    double tau = typical ? (double)a.temperature : 1.0;
    launch_pdl(node_stats_kernel, dim3(a.T, typical ? a.stat_slices : 1), dim3(1024), 0, s, a.logits, a.V, typical, tau, a.node_argmax,
               reinterpret_cast<NodePart *>(a.node_part));
    launch_pdl(select_path_kernel, dim3(1), dim3(256), 0, s, a, typical, tau, (double)a.eps, (double)a.delta, rejection);
}

__global__ void __launch_bounds__(1024) argmax_row_kernel(const float *__restrict__ logits, int V, int row, int32_t *out)
{
    pdl_enter();
    __shared__ float sv[32];
    __shared__ int si[32];
    const float *lp = logits + (size_t)row * V;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    scan_argmax(lp, V, bv, bi);
    int am = block_argmax(bv, bi, sv, si);
    if (threadIdx.x == 0)
        *out = am;
}

void launch_argmax_row(const float *logits, int V, int row, int32_t *out, cudaStream_t s)
{
    launch_pdl(argmax_row_kernel, dim3(1), dim3(1024), 0, s, logits, V, row, out);
}

// ---------------------------------------------------------------------------------------- commit
// grid (n_layers, 2): block (l, 0) moves K rows, (l, 1) moves V rows, 16 bytes per thread per step.
template <typename AT>
__global__ void __launch_bounds__(256) commit_rows_kernel(CommitArgs a)
{
    pdl_enter();
    const int L = *a.cache_len;
    int n = min(1 + *a.accept_len, a.max_commit);
    if (n <= 0 || L + n > a.L_max)
        return;
    constexpr int VN = Vec16<AT>::N;
    const int l = blockIdx.x;
    const AT *src = (const AT *)(blockIdx.y == 0 ? a.tree_k : a.tree_v) + (size_t)l * a.tree_rows * a.H * a.D;
    AT *dst = (AT *)(blockIdx.y == 0 ? a.k_cache : a.v_cache) + (size_t)l * a.H * a.L_max * a.D;
    const int cpr = a.D / VN;  // 16-byte chunks per head row
    const int per_node = a.H * cpr;
    for (int i = threadIdx.x; i < n * per_node; i += blockDim.x) {
        int j = i / per_node, rem = i % per_node, h = rem / cpr, c = rem % cpr;
        int node = a.acc_nodes[j];
        const uint4 *sp = reinterpret_cast<const uint4 *>(src + ((size_t)node * a.H + h) * a.D) + c;
        uint4 *dp = reinterpret_cast<uint4 *>(dst + ((size_t)h * a.L_max + (L + j)) * a.D) + c;
        *dp = *sp;
    }
}

template <typename AT>
__global__ void __launch_bounds__(256) commit_finalize_kernel(CommitArgs a)
{
    pdl_enter();
    const int L = *a.cache_len;
    int n = min(1 + *a.accept_len, a.max_commit);
    if (n < 0) n = 0;
    if (L + n > a.L_max) {
        if (threadIdx.x == 0) {
            *a.status = MEDUSA_ERR_CACHE_FULL;
            *a.n_emitted = 0;
        }
        return;
    }
    if (n > 0) {
        const float *hs = a.hidden + (size_t)a.acc_nodes[n - 1] * a.d;
        for (int i = threadIdx.x; i < a.d; i += blockDim.x)
            a.h_last[i] = hs[i];
    }
    if (threadIdx.x < a.depth_plus1)
        a.emitted[threadIdx.x] = threadIdx.x < n ? a.tree_tok[a.acc_nodes[threadIdx.x]] : -1;
    __syncthreads();
    if (threadIdx.x == 0) {
        *a.n_emitted = n;
        *a.cache_len = L + n;
        // The next step's root is the successor of the last COMMITTED token.  When max_commit cut the accepted path
        // short (n < 1 + accept_len) that successor is the path's next node, which was already accepted; otherwise it
        // is the token chosen after the whole path.
        if (a.root_out && a.next_root)
            *a.root_out = n > 0 && n < 1 + *a.accept_len ? a.tree_tok[a.acc_nodes[n]] : *a.next_root;
    }
}

void launch_commit(int dtype, const CommitArgs &a, cudaStream_t s)
{
    dim3 grid(a.n_layers, 2);
    if (dtype == MEDUSA_BF16) {
        launch_pdl(commit_rows_kernel<bf16>, dim3(grid), dim3(256), 0, s, a);
        launch_pdl(commit_finalize_kernel<bf16>, dim3(1), dim3(256), 0, s, a);
    } else {
        launch_pdl(commit_rows_kernel<float>, dim3(grid), dim3(256), 0, s, a);
        launch_pdl(commit_finalize_kernel<float>, dim3(1), dim3(256), 0, s, a);
    }
}

}  // namespace medusa

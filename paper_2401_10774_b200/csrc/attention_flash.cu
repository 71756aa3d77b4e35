// Split-KV flash-decode kernel for tree attention (paper Sec. 2.1.2, Fig. 2; App. G Table 5: QK^T and PV with
// q candidate tokens against s cached positions), bf16, head_dim 128, up to 64 tree queries.
//
// Every K/V byte of a head serves all 64 tree queries, so the operator is an HBM streamer (about 60 flops
// per byte) as long as the two products run on tensor cores.  One CTA owns one (head, key range): it streams
// 64-key K/V tiles into swizzled shared memory (16-byte asynchronous copies, 3-stage ring), each of its four
// warps keeps 16 query rows in registers (Q fragments, score and output accumulators), the softmax is the
// online form with row reductions by warp shuffles inside a quad.  The tree mask is one 64-bit word per
// query held in registers and touches only the single tile that holds the tree's own keys; cache tiles are
// unmasked except for the ragged end.  Key ranges are combined by log-sum-exp: each CTA writes an
// unnormalised partial (O, m, l); the CTA that finishes last for a head (atomic ticket, nobody waits) adds
// the partials in split order, normalises and writes the output, optionally as a split (hi, lo) activation.
// Caches of at most 8 tiles (512 keys) skip all of that: two CTAs per head take 32 query rows each over all the
// keys (attention_rows_mode; measured 8.6 vs 11.5 us at 256 keys, 11.7 vs 12.4 us at 512, slower from 768 on).
// Which of the two forms runs, and with how many key ranges, is decided on the device from the cache length.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "pdl.cuh"
#include "kernels.h"

namespace medusa {

namespace {

constexpr int D = 128;          // head dim
constexpr int BQ = 64;          // query rows per CTA (4 warps x 16)
constexpr int BKEY = 64;        // keys per tile
constexpr int STAGES = 3;
constexpr int THREADS = 256;     // 8 warps: warp w owns query rows 16*(w&3).. and key half (w>>2) of every tile
constexpr int TILE_BYTES = BKEY * D * 2;           // 16 KiB for K, same for V
constexpr int STAGE_BYTES = 2 * TILE_BYTES;
// Q tile (and its second plane, if q comes as two planes), then the K/V ring
constexpr int smem_bytes(bool qlo) { return (qlo ? 2 : 1) * TILE_BYTES + STAGES * STAGE_BYTES; }
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk c (0..15) of row r in a [64][128] bf16 tile; XOR swizzle on the low 3 chunk bits
__device__ __forceinline__ uint32_t tile_off(int r, int c) { return (uint32_t)(r * 256 + ((c ^ (r & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    int sz = valid ? 16 : 0;  // size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *c, const uint32_t *a, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

struct Args {
    const bf16 *q, *k_new, *v_new;   // [T][H][D]
    const bf16 *q_lo;                // [T][H][D] second plane of q (kernels instantiated with QLO): scores are q.k + q_lo.k
    const bf16 *k_cache, *v_cache;   // [H][L_max][D]
    const int32_t *cache_len;
    const uint64_t *mask;            // [T][mask_words]: bit j of row i -- tree node j visible to query i
    int mask_words;                  // 64 tree nodes per word (1 unless the kernel is instantiated with LARGE)
    // LARGE instantiation only.  batch != 0: blockIdx.z is a SEQUENCE (one tile of 64 query rows each, all with the same
    // tree of T nodes): its keys are its own cache (cache_seq_stride elements after the previous sequence's), its own
    // cache length (len_stride ints after the previous one's) and its own tile of tree keys.
    int batch, len_stride;
    long long cache_seq_stride;
    bf16 *out, *out_lo;              // [T][H][D]; out_lo nullable
    float *lse;                      // nullable [T][H]
    float *ws_o;                     // [q tiles][H][max_splits][64][128] unnormalised partial outputs
    float *ws_ml;                    // [q tiles][H][max_splits][2][64]  running max (log2 domain) and sum
    int *counters;                   // [q tiles][H] arrival tickets, zero between launches
    int T, H, L_max, tiles_per_split, max_splits;
    int Hkv;                         // key/value heads; query head h reads key/value head h / (H / Hkv)
    int rows_max_tiles;              // caches of up to this many tiles run in row-split mode (0: never)
};

// loads one 64-key tile pair (K and V) into a stage; rows >= n_valid are zero-filled
__device__ __forceinline__ void load_tile(uint8_t *stage, const bf16 *ksrc, const bf16 *vsrc, size_t row_stride, int n_valid)
{
    const uint32_t kb = smem_u32(stage), vb = kb + TILE_BYTES;
#pragma unroll
    for (int i = 0; i < 1024 / THREADS; ++i) {
        int idx = threadIdx.x + i * THREADS;   // 1024 chunks per tile
        int r = idx >> 4, c = idx & 15;
        bool ok = r < n_valid;
        size_t off = (size_t)(ok ? r : 0) * row_stride + c * 8;
        cp_async16(kb + tile_off(r, c), ksrc + off, ok);
        cp_async16(vb + tile_off(r, c), vsrc + off, ok);
    }
}

// Row-split mode for short caches: CTA (h, half) owns 32 query rows of head h and walks ALL keys, so no partial
// results cross CTAs and nothing is combined through global memory.  Warp w owns query rows 16*(w&1).. of the half
// and keys 16*(w>>1).. of every 64-key tile; the four key quarters meet once, in shared memory, at the end.
// (Twice the CTAs of one key range per head at half the tensor work per tile each; K/V are read twice, the second
// time from L2.)  Its tile loop repeats the key-range form's with 16 instead of 32 keys per warp; the two are kept
// spelled out because one template for both measured 2-10 % slower (register allocation of the longer form).
template <bool QLO>
__device__ __forceinline__ void attention_rows_mode(const Args &a, uint8_t *smem_all, int h, int half, int L, int nt)
{
    uint8_t *smem = smem_all + (QLO ? 2 : 1) * TILE_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
    const int wq = warp & 1, kq = warp >> 1;
    const int rbase = half * 32;
    if (rbase >= a.T)
        return;
    const int n_tiles = nt + 1;  // the tree's own keys are the last tile
    const size_t HD = (size_t)a.H * D, HkvD = (size_t)a.Hkv * D;
    const int hk = h / (a.H / a.Hkv);
    auto issue = [&](int i) {
        uint8_t *stage = smem + (i % STAGES) * STAGE_BYTES;
        if (i < nt) {
            const size_t base = ((size_t)hk * a.L_max + (size_t)i * BKEY) * D;
            load_tile(stage, a.k_cache + base, a.v_cache + base, D, min(BKEY, L - i * BKEY));
        } else {
            load_tile(stage, a.k_new + (size_t)hk * D, a.v_new + (size_t)hk * D, HkvD, a.T);
        }
    };
    {
        const uint32_t qb = smem_u32(smem_all);
#pragma unroll
        for (int i = 0; i < 512 / THREADS; ++i) {
            const int idx = threadIdx.x + i * THREADS;
            const int r = idx >> 4, c = idx & 15;
            const bool ok = rbase + r < a.T;
            cp_async16(qb + tile_off(r, c), a.q + (size_t)(ok ? rbase + r : 0) * HD + (size_t)h * D + c * 8, ok);
            if (QLO)
                cp_async16(qb + TILE_BYTES + tile_off(r, c), a.q_lo + (size_t)(ok ? rbase + r : 0) * HD + (size_t)h * D + c * 8, ok);
        }
        cp_async_commit();
    }
    for (int i = 0; i < STAGES - 1; ++i) {
        if (i < n_tiles)
            issue(i);
        cp_async_commit();
    }
    cp_async_wait<STAGES - 1>();
    __syncthreads();
    uint32_t qf[8][4];
    const int q_row = wq * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
    const uint32_t q_lo_addr = smem_u32(smem_all) + TILE_BYTES;  // second plane's tile (QLO): fragments are re-read per tile
    {
        const uint32_t qb = smem_u32(smem_all);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            ldsm_x4(qb + tile_off(q_row, 2 * ks + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    const int lr0 = wq * 16 + g, lr1 = lr0 + 8;      // rows inside the half
    const int row0 = rbase + lr0, row1 = rbase + lr1;  // tree rows
    const uint64_t mask0 = row0 < a.T ? a.mask[row0] : 0ull, mask1 = row1 < a.T ? a.mask[row1] : 0ull;
    const float sc = rsqrtf((float)D) * LOG2E;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
        o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    for (int i = 0; i < n_tiles; ++i) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (i + STAGES - 1 < n_tiles)
            issue(i + STAGES - 1);
        cp_async_commit();
        const uint32_t kb = smem_u32(smem + (i % STAGES) * STAGE_BYTES), vb = kb + TILE_BYTES;
        const bool tree_tile = i >= nt;
        // ---- S = Q K^T  (16 rows x this warp's 16 keys of the tile)
        float s[2][4];
        s[0][0] = s[0][1] = s[0][2] = s[0][3] = 0.f;
        s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t b0, b1, b2, b3;
            const int kr = kq * 16 + (lane & 7) + 8 * (lane >> 4);
            ldsm_x4(kb + tile_off(kr, 2 * ks + ((lane >> 3) & 1)), b0, b1, b2, b3);
            mma_bf16(s[0], qf[ks], b0, b1);
            mma_bf16(s[1], qf[ks], b2, b3);
            if (QLO) {  // the second plane's fragments come from shared memory: there are no registers to hold them
                uint32_t ql[4];
                ldsm_x4(q_lo_addr + tile_off(q_row, 2 * ks + (lane >> 4)), ql[0], ql[1], ql[2], ql[3]);
                mma_bf16(s[0], ql, b0, b1);
                mma_bf16(s[1], ql, b2, b3);
            }
        }
        // ---- mask + online softmax (log2 domain)
        float mx0 = -INFINITY, mx1 = -INFINITY;
        const int key_base = i * BKEY;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int j = (2 * kq + n) * 8 + 2 * t4 + e;  // key inside the tile
                bool v0, v1;
                if (tree_tile) {
                    v0 = (mask0 >> j) & 1ull;
                    v1 = (mask1 >> j) & 1ull;
                } else {
                    v0 = v1 = key_base + j < L;
                }
                s[n][e] = v0 ? s[n][e] * sc : -INFINITY;
                s[n][2 + e] = v1 ? s[n][2 + e] * sc : -INFINITY;
                mx0 = fmaxf(mx0, s[n][e]);
                mx1 = fmaxf(mx1, s[n][2 + e]);
            }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
        const float c0 = exp2f(m0 - ms0), c1 = exp2f(m1 - ms1);  // m = -inf gives 0
        m0 = mn0;
        m1 = mn1;
        float ps0 = 0.f, ps1 = 0.f;
        uint32_t pf[4];
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            const float p00 = exp2f(s[n][0] - ms0), p01 = exp2f(s[n][1] - ms0);
            const float p10 = exp2f(s[n][2] - ms1), p11 = exp2f(s[n][3] - ms1);
            ps0 += p00 + p01;
            ps1 += p10 + p11;
            pf[n * 2] = pack_bf16(p00, p01);
            pf[n * 2 + 1] = pack_bf16(p10, p11);
        }
        l0 = l0 * c0 + ps0;
        l1 = l1 * c1 + ps1;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            o[dn][0] *= c0;
            o[dn][1] *= c0;
            o[dn][2] *= c1;
            o[dn][3] *= c1;
        }
        // ---- O += P V
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
            uint32_t b0, b1, b2, b3;
            const int kr = kq * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
            ldsm_x4_t(vb + tile_off(kr, 2 * dp + (lane >> 4)), b0, b1, b2, b3);
            mma_bf16(o[2 * dp], pf, b0, b1);
            mma_bf16(o[2 * dp + 1], pf, b2, b3);
        }
    }
    cp_async_wait<0>();
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- the key quarters meet: warps of quarters 1-3 hand (m, l, O) to the warps of quarter 0, added in quarter order
    __syncthreads();  // every warp is done with the K/V ring
    float *mo = reinterpret_cast<float *>(smem);  // [3][32][128]
    float *mml = mo + 3 * 32 * D;                 // [3][2][32]
    if (kq > 0) {
        float *po = mo + (size_t)(kq - 1) * 32 * D;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            *reinterpret_cast<float2 *>(po + lr0 * D + dn * 8 + 2 * t4) = make_float2(o[dn][0], o[dn][1]);
            *reinterpret_cast<float2 *>(po + lr1 * D + dn * 8 + 2 * t4) = make_float2(o[dn][2], o[dn][3]);
        }
        if (t4 == 0) {
            float *pm = mml + (kq - 1) * 64;
            pm[lr0] = m0; pm[lr1] = m1; pm[32 + lr0] = l0; pm[32 + lr1] = l1;
        }
    }
    __syncthreads();
    if (kq != 0)
        return;
#pragma unroll 1
    for (int p = 0; p < 3; ++p) {
        const float *po = mo + (size_t)p * 32 * D;
        const float *pm = mml + p * 64;
        const float mb0 = pm[lr0], mb1 = pm[lr1], lb0 = pm[32 + lr0], lb1 = pm[32 + lr1];
        const float mn0 = fmaxf(m0, mb0), mn1 = fmaxf(m1, mb1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
        const float ca0 = exp2f(m0 - ms0), cb0 = exp2f(mb0 - ms0), ca1 = exp2f(m1 - ms1), cb1 = exp2f(mb1 - ms1);
        l0 = l0 * ca0 + lb0 * cb0;
        l1 = l1 * ca1 + lb1 * cb1;
        m0 = mn0;
        m1 = mn1;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            const float2 p0 = *reinterpret_cast<const float2 *>(po + lr0 * D + dn * 8 + 2 * t4);
            const float2 p1 = *reinterpret_cast<const float2 *>(po + lr1 * D + dn * 8 + 2 * t4);
            o[dn][0] = o[dn][0] * ca0 + p0.x * cb0;
            o[dn][1] = o[dn][1] * ca0 + p0.y * cb0;
            o[dn][2] = o[dn][2] * ca1 + p1.x * cb1;
            o[dn][3] = o[dn][3] * ca1 + p1.y * cb1;
        }
    }
    // ---- normalise and write straight from the accumulators
    const float i0 = l0 > 0.f ? 1.0f / l0 : 0.f, i1 = l1 > 0.f ? 1.0f / l1 : 0.f;
#pragma unroll
    for (int dn = 0; dn < 16; ++dn) {
        const int col = dn * 8 + 2 * t4;
        if (row0 < a.T) {
            const size_t idx = (size_t)row0 * HD + (size_t)h * D + col;
            const float y0 = o[dn][0] * i0, y1 = o[dn][1] * i0;
            const __nv_bfloat162 hi = __floats2bfloat162_rn(y0, y1);
            *reinterpret_cast<__nv_bfloat162 *>(a.out + idx) = hi;
            if (a.out_lo)
                *reinterpret_cast<__nv_bfloat162 *>(a.out_lo + idx) =
                    __floats2bfloat162_rn(y0 - __low2float(hi), y1 - __high2float(hi));
        }
        if (row1 < a.T) {
            const size_t idx = (size_t)row1 * HD + (size_t)h * D + col;
            const float y0 = o[dn][2] * i1, y1 = o[dn][3] * i1;
            const __nv_bfloat162 hi = __floats2bfloat162_rn(y0, y1);
            *reinterpret_cast<__nv_bfloat162 *>(a.out + idx) = hi;
            if (a.out_lo)
                *reinterpret_cast<__nv_bfloat162 *>(a.out_lo + idx) =
                    __floats2bfloat162_rn(y0 - __low2float(hi), y1 - __high2float(hi));
        }
    }
    if (a.lse && t4 == 0) {
        if (row0 < a.T) a.lse[(size_t)row0 * a.H + h] = m0 / LOG2E + logf(l0);
        if (row1 < a.T) a.lse[(size_t)row1 * a.H + h] = m1 / LOG2E + logf(l1);
    }
}

// QLO: q comes as two bf16 planes (the decode step's rotation kernel writes them), and the scores are q.k + q_lo.k, so
// that q's rounding to one plane does not reach the softmax.  LARGE: trees of more than 64 nodes -- blockIdx.z is the
// tile of 64 query rows, which sees the tree's key tiles 0..z (ancestors have smaller indices) through one 64-bit mask
// word per key tile.  The plain instantiation is the 64-node kernel unchanged.
template <bool QLO, bool LARGE>
__global__ void __launch_bounds__(THREADS, 1) tree_attention_flash_kernel(Args a)
{
    pdl_enter();
    extern __shared__ __align__(1024) uint8_t smem_all[];
    uint8_t *smem = smem_all + (QLO ? 2 : 1) * TILE_BYTES;  // K/V ring; the Q tile(s) sit in front of it
    __shared__ int s_ticket;
    const int h = blockIdx.x, sp = blockIdx.y;
    const bool batch = LARGE && a.batch != 0;
    const int q0 = LARGE ? (int)blockIdx.z * BQ : 0;            // first query row of this CTA's tile
    const int Tq = LARGE && !batch ? min(BQ, a.T - q0) : a.T;   // its query rows
    const int tree_tiles = LARGE && !batch ? (int)blockIdx.z + 1 : 1;  // key tiles of the tree this query tile can see
    const int tree_tile0 = batch ? (int)blockIdx.z : 0;         // the first of them (a sequence's own tile in a batch)
    const int mrow0 = batch ? 0 : q0;                           // mask row of the tile's first query
    const size_t slot = LARGE ? (size_t)blockIdx.z * a.H + h : (size_t)h;  // (query tile, head)
    const bf16 *const kc_base = a.k_cache + (batch ? (size_t)blockIdx.z * a.cache_seq_stride : 0);
    const bf16 *const vc_base = a.v_cache + (batch ? (size_t)blockIdx.z * a.cache_seq_stride : 0);
    const int32_t *const len_ptr = a.cache_len + (batch ? (size_t)blockIdx.z * a.len_stride : 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
    const int wq = warp & 3, kh = warp >> 2;  // query-row group, key half
    // a length outside [0, L_max] would index past the caches: clamp (the driver's own state never leaves that range)
    const int L = min(max(*len_ptr, 0), a.L_max);
    const int nt = (L + BKEY - 1) / BKEY;
    if (!LARGE && nt <= a.rows_max_tiles && gridDim.y >= 2) {
        if (sp < 2)
            attention_rows_mode<QLO>(a, smem_all, h, sp, L, nt);
        return;
    }
    // Key ranges: fixed by the launch (tiles_per_split > 0), or chosen here from the true cache length, so that
    // the result does not depend on what the host knew about the length when it launched.  A CTA's time grows
    // with its tiles, the combine with the number of ranges: about sqrt(tiles) ranges balances the two, and never
    // more ranges than the grid has rows.
    int tps = a.tiles_per_split;
    if (tps <= 0) {
        int want = 1;
        while (want * want < nt) ++want;
        if (want > (int)gridDim.y) want = (int)gridDim.y;
        tps = nt > 0 ? (nt + want - 1) / want : 1;
    }
    const int n_cache_splits = (nt + tps - 1) / tps;
    // never more ranges than the grid has rows: when the launch's fixed range size was chosen for a shorter cache than
    // the one found here, the last range takes all the remaining tiles (slower, still complete)
    const int n_active = min(n_cache_splits > 0 ? n_cache_splits : 1, (int)gridDim.y);
    if (sp >= n_active)
        return;
    const int tile0 = sp * tps;
    const bool has_tree = sp == n_active - 1;
    const int tile1 = has_tree ? nt : min(nt, tile0 + tps);
    const int n_tiles = (tile1 - tile0) + (has_tree ? tree_tiles : 0);
    const size_t HD = (size_t)a.H * D, HkvD = (size_t)a.Hkv * D;
    const int hk = h / (a.H / a.Hkv);

    auto issue = [&](int i) {
        // tile i of this CTA: a cache tile, or (last, if has_tree) the tree's own keys
        uint8_t *stage = smem + (i % STAGES) * STAGE_BYTES;
        const int ct = tile0 + i;
        if (ct < tile1) {
            const size_t base = ((size_t)hk * a.L_max + (size_t)ct * BKEY) * D;
            load_tile(stage, kc_base + base, vc_base + base, D, min(BKEY, L - ct * BKEY));
        } else {
            const int w = LARGE ? tree_tile0 + ct - tile1 : 0;  // key tile of the tree (row tile of k_new / v_new)
            const size_t tb = ((size_t)w * BKEY * a.Hkv + hk) * D;
            load_tile(stage, a.k_new + tb, a.v_new + tb, HkvD, batch ? a.T : min(BKEY, a.T - w * BKEY));
        }
    };
    // ---- Q and the first K/V tiles are requested together; Q is copy group 0
    {
        const uint32_t qb = smem_u32(smem_all);
#pragma unroll
        for (int i = 0; i < 1024 / THREADS; ++i) {
            int idx = threadIdx.x + i * THREADS;
            int r = idx >> 4, c = idx & 15;
            bool ok = r < Tq;
            cp_async16(qb + tile_off(r, c), a.q + (size_t)(ok ? q0 + r : 0) * HD + (size_t)h * D + c * 8, ok);
            if (QLO)
                cp_async16(qb + TILE_BYTES + tile_off(r, c), a.q_lo + (size_t)(ok ? q0 + r : 0) * HD + (size_t)h * D + c * 8, ok);
        }
        cp_async_commit();
    }
    for (int i = 0; i < STAGES - 1; ++i) {
        if (i < n_tiles)
            issue(i);
        cp_async_commit();
    }
    cp_async_wait<STAGES - 1>();  // everything but the K/V groups just issued: Q has landed
    __syncthreads();
    uint32_t qf[8][4];
    const int q_row = wq * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
    const uint32_t q_lo_addr = smem_u32(smem_all) + TILE_BYTES;  // second plane's tile (QLO): fragments are re-read per tile
    {
        const uint32_t qb = smem_u32(smem_all);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            ldsm_x4(qb + tile_off(q_row, 2 * ks + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }

    const int row0 = wq * 16 + g, row1 = row0 + 8;  // rows inside the query tile
    // mask words of this thread's two rows for the tree's first key tile; with LARGE the words of the following key tiles
    // are fetched one tile ahead inside the loop
    uint64_t mask0 = row0 < Tq ? a.mask[(size_t)(mrow0 + row0) * (LARGE ? a.mask_words : 1)] : 0ull;
    uint64_t mask1 = row1 < Tq ? a.mask[(size_t)(mrow0 + row1) * (LARGE ? a.mask_words : 1)] : 0ull;
    uint64_t next_mask0 = 0ull, next_mask1 = 0ull;
    const float sc = rsqrtf((float)D) * LOG2E;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
        o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    for (int i = 0; i < n_tiles; ++i) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (i + STAGES - 1 < n_tiles)
            issue(i + STAGES - 1);
        cp_async_commit();
        const uint32_t kb = smem_u32(smem + (i % STAGES) * STAGE_BYTES), vb = kb + TILE_BYTES;
        const int ct = tile0 + i;
        const bool tree_tile = ct >= tile1;

        // ---- S = Q K^T  (16 rows x this warp's 32 keys of the tile)
        float s[4][4];
#pragma unroll
        for (int n = 0; n < 4; ++n)
            s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t ql[4];
            if (QLO)  // the second plane's fragments come from shared memory: there are no registers to hold them
                ldsm_x4(q_lo_addr + tile_off(q_row, 2 * ks + (lane >> 4)), ql[0], ql[1], ql[2], ql[3]);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t b0, b1, b2, b3;
                const int kr = (2 * kh + np) * 16 + (lane & 7) + 8 * (lane >> 4);
                ldsm_x4(kb + tile_off(kr, 2 * ks + ((lane >> 3) & 1)), b0, b1, b2, b3);
                mma_bf16(s[2 * np], qf[ks], b0, b1);
                mma_bf16(s[2 * np + 1], qf[ks], b2, b3);
                if (QLO) {
                    mma_bf16(s[2 * np], ql, b0, b1);
                    mma_bf16(s[2 * np + 1], ql, b2, b3);
                }
            }
        }
        // ---- mask + online softmax (log2 domain)
        float mx0 = -INFINITY, mx1 = -INFINITY;
        const int key_base = ct * BKEY;
        if (LARGE && tree_tile) {
            // this key tile's words were fetched a tile ago (the first one before the loop); ask for the next tile's now
            const int w = ct - tile1;
            if (w > 0) { mask0 = next_mask0; mask1 = next_mask1; }
            if (w + 1 < tree_tiles) {
                if (row0 < Tq) next_mask0 = a.mask[(size_t)(mrow0 + row0) * a.mask_words + w + 1];
                if (row1 < Tq) next_mask1 = a.mask[(size_t)(mrow0 + row1) * a.mask_words + w + 1];
            }
        }
#pragma unroll
        for (int n = 0; n < 4; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int j = (4 * kh + n) * 8 + 2 * t4 + e;  // key inside the tile
                bool v0, v1;
                if (tree_tile) {
                    v0 = (mask0 >> j) & 1ull;
                    v1 = (mask1 >> j) & 1ull;
                } else {
                    v0 = v1 = key_base + j < L;
                }
                s[n][e] = v0 ? s[n][e] * sc : -INFINITY;
                s[n][2 + e] = v1 ? s[n][2 + e] * sc : -INFINITY;
                mx0 = fmaxf(mx0, s[n][e]);
                mx1 = fmaxf(mx1, s[n][2 + e]);
            }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
        const float c0 = exp2f(m0 - ms0), c1 = exp2f(m1 - ms1);  // m = -inf gives 0
        m0 = mn0;
        m1 = mn1;
        float ps0 = 0.f, ps1 = 0.f;
        uint32_t pf[2][4];
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            const float p00 = exp2f(s[n][0] - ms0), p01 = exp2f(s[n][1] - ms0);
            const float p10 = exp2f(s[n][2] - ms1), p11 = exp2f(s[n][3] - ms1);
            ps0 += p00 + p01;
            ps1 += p10 + p11;
            pf[n >> 1][(n & 1) * 2] = pack_bf16(p00, p01);
            pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p10, p11);
        }
        l0 = l0 * c0 + ps0;
        l1 = l1 * c1 + ps1;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            o[dn][0] *= c0;
            o[dn][1] *= c0;
            o[dn][2] *= c1;
            o[dn][3] *= c1;
        }
        // ---- O += P V
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                uint32_t b0, b1, b2, b3;
                const int kr = (2 * kh + j) * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
                ldsm_x4_t(vb + tile_off(kr, 2 * dp + (lane >> 4)), b0, b1, b2, b3);
                mma_bf16(o[2 * dp], pf[j], b0, b1);
                mma_bf16(o[2 * dp + 1], pf[j], b2, b3);
            }
        }
    }
    cp_async_wait<0>();
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- merge the two key halves of the CTA: warps 4-7 hand (m, l, O) to warps 0-3 through shared memory
    {
        __syncthreads();  // every warp is done with the K/V ring
        float *mo = reinterpret_cast<float *>(smem);  // [64][128]
        float *mml = mo + BQ * D;                     // [2][64]
        if (kh == 1) {
#pragma unroll
            for (int dn = 0; dn < 16; ++dn) {
                *reinterpret_cast<float2 *>(mo + row0 * D + dn * 8 + 2 * t4) = make_float2(o[dn][0], o[dn][1]);
                *reinterpret_cast<float2 *>(mo + row1 * D + dn * 8 + 2 * t4) = make_float2(o[dn][2], o[dn][3]);
            }
            if (t4 == 0) {
                mml[row0] = m0; mml[row1] = m1; mml[BQ + row0] = l0; mml[BQ + row1] = l1;
            }
        }
        __syncthreads();
        if (kh == 0) {
            const float mb0 = mml[row0], mb1 = mml[row1], lb0 = mml[BQ + row0], lb1 = mml[BQ + row1];
            const float mn0 = fmaxf(m0, mb0), mn1 = fmaxf(m1, mb1);
            const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
            const float ca0 = exp2f(m0 - ms0), cb0 = exp2f(mb0 - ms0), ca1 = exp2f(m1 - ms1), cb1 = exp2f(mb1 - ms1);
            l0 = l0 * ca0 + lb0 * cb0;
            l1 = l1 * ca1 + lb1 * cb1;
            m0 = mn0;
            m1 = mn1;
#pragma unroll
            for (int dn = 0; dn < 16; ++dn) {
                const float2 p0 = *reinterpret_cast<const float2 *>(mo + row0 * D + dn * 8 + 2 * t4);
                const float2 p1 = *reinterpret_cast<const float2 *>(mo + row1 * D + dn * 8 + 2 * t4);
                o[dn][0] = o[dn][0] * ca0 + p0.x * cb0;
                o[dn][1] = o[dn][1] * ca0 + p0.y * cb0;
                o[dn][2] = o[dn][2] * ca1 + p1.x * cb1;
                o[dn][3] = o[dn][3] * ca1 + p1.y * cb1;
            }
        }
        __syncthreads();  // the ring is reused below
    }
    const bool owner = kh == 0;  // warps 0-3 now hold the CTA's result

    if (n_active == 1) {
        // a single key range: normalise and write straight from the accumulators
        const float i0 = l0 > 0.f ? 1.0f / l0 : 0.f, i1 = l1 > 0.f ? 1.0f / l1 : 0.f;
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            const int col = dn * 8 + 2 * t4;
            if (owner && row0 < Tq) {
                const size_t idx = (size_t)(q0 + row0) * HD + (size_t)h * D + col;
                const float y0 = o[dn][0] * i0, y1 = o[dn][1] * i0;
                const __nv_bfloat162 hi = __floats2bfloat162_rn(y0, y1);
                *reinterpret_cast<__nv_bfloat162 *>(a.out + idx) = hi;
                if (a.out_lo)
                    *reinterpret_cast<__nv_bfloat162 *>(a.out_lo + idx) =
                        __floats2bfloat162_rn(y0 - __low2float(hi), y1 - __high2float(hi));
            }
            if (owner && row1 < Tq) {
                const size_t idx = (size_t)(q0 + row1) * HD + (size_t)h * D + col;
                const float y0 = o[dn][2] * i1, y1 = o[dn][3] * i1;
                const __nv_bfloat162 hi = __floats2bfloat162_rn(y0, y1);
                *reinterpret_cast<__nv_bfloat162 *>(a.out + idx) = hi;
                if (a.out_lo)
                    *reinterpret_cast<__nv_bfloat162 *>(a.out_lo + idx) =
                        __floats2bfloat162_rn(y0 - __low2float(hi), y1 - __high2float(hi));
            }
        }
        if (a.lse && t4 == 0 && owner) {
            if (row0 < Tq) a.lse[(size_t)(q0 + row0) * a.H + h] = m0 / LOG2E + logf(l0);
            if (row1 < Tq) a.lse[(size_t)(q0 + row1) * a.H + h] = m1 / LOG2E + logf(l1);
        }
        return;
    }
    // ---- partial result of this key range
    float *wo = a.ws_o + (slot * a.max_splits + sp) * BQ * D;
    float *wml = a.ws_ml + (slot * a.max_splits + sp) * 2 * BQ;
    if (owner) {
#pragma unroll
        for (int dn = 0; dn < 16; ++dn) {
            *reinterpret_cast<float2 *>(wo + (size_t)row0 * D + dn * 8 + 2 * t4) = make_float2(o[dn][0], o[dn][1]);
            *reinterpret_cast<float2 *>(wo + (size_t)row1 * D + dn * 8 + 2 * t4) = make_float2(o[dn][2], o[dn][3]);
        }
    }
    if (t4 == 0 && owner) {
        wml[row0] = m0;
        wml[row1] = m1;
        wml[BQ + row0] = l0;
        wml[BQ + row1] = l1;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0)
        s_ticket = atomicAdd(a.counters + slot, 1);
    __syncthreads();
    if (s_ticket != n_active - 1)
        return;
    // ---- last CTA of this head: combine the key ranges in split order
    __threadfence();
    float (*s_w)[BQ] = reinterpret_cast<float (*)[BQ]>(smem);  // [max_splits + 1][64] weights; the ring is idle now
    float *s_ml = reinterpret_cast<float *>(smem) + (FLASH_MAX_SPLITS + 1) * BQ;  // staged (max, sum) pairs [split][2][64]
    const float *__restrict__ mlh = a.ws_ml + slot * a.max_splits * 2 * BQ;
    {
        // one batch of independent loads: thread t fetches element t of every key range's 128-float record
        float t[FLASH_MAX_SPLITS];
        const bool mine = threadIdx.x < 2 * BQ;
#pragma unroll
        for (int s2 = 0; s2 < FLASH_MAX_SPLITS; ++s2)
            if (mine && s2 < n_active) t[s2] = mlh[(size_t)s2 * 2 * BQ + threadIdx.x];
#pragma unroll
        for (int s2 = 0; s2 < FLASH_MAX_SPLITS; ++s2)
            if (mine && s2 < n_active) s_ml[s2 * 2 * BQ + threadIdx.x] = t[s2];
    }
    __syncthreads();
    if (threadIdx.x < BQ) {
        const int r = threadIdx.x;
        float mstar = -INFINITY;
        for (int s2 = 0; s2 < n_active; ++s2)
            mstar = fmaxf(mstar, s_ml[s2 * 2 * BQ + r]);
        const float msafe = mstar == -INFINITY ? 0.f : mstar;
        float lstar = 0.f;
        for (int s2 = 0; s2 < n_active; ++s2) {
            const float w = exp2f(s_ml[s2 * 2 * BQ + r] - msafe);
            s_w[s2][r] = w;
            lstar += w * s_ml[s2 * 2 * BQ + BQ + r];
        }
        s_w[FLASH_MAX_SPLITS][r] = lstar > 0.f ? 1.0f / lstar : 0.f;
        if (a.lse && r < Tq)
            a.lse[(size_t)(q0 + r) * a.H + h] = mstar / LOG2E + logf(lstar);
    }
    __syncthreads();
    // thread -> 4 adjacent columns of 8 rows; per key range the 8 row loads are in flight together
    const float *__restrict__ oh = a.ws_o + slot * a.max_splits * BQ * D;
    const int c4 = (threadIdx.x & 31) * 4, rg = (threadIdx.x >> 5) * 8;
    float4 acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
        acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s2 = 0; s2 < n_active; s2 += 2) {
        // two key ranges (16 independent 16-byte loads per thread) in flight per round; always added in range order
        float4 v[8], v2[8];
        const bool two = s2 + 1 < n_active;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            v[u] = *reinterpret_cast<const float4 *>(oh + ((size_t)s2 * BQ + rg + u) * D + c4);
        if (two) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
                v2[u] = *reinterpret_cast<const float4 *>(oh + ((size_t)(s2 + 1) * BQ + rg + u) * D + c4);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float w = s_w[s2][rg + u];
            acc[u].x += w * v[u].x; acc[u].y += w * v[u].y; acc[u].z += w * v[u].z; acc[u].w += w * v[u].w;
        }
        if (two) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float w = s_w[s2 + 1][rg + u];
                acc[u].x += w * v2[u].x; acc[u].y += w * v2[u].y; acc[u].z += w * v2[u].z; acc[u].w += w * v2[u].w;
            }
        }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int r = rg + u;
        if (r >= Tq)
            continue;
        const float inv = s_w[FLASH_MAX_SPLITS][r];
        const float y[4] = {acc[u].x * inv, acc[u].y * inv, acc[u].z * inv, acc[u].w * inv};
        const size_t idx = (size_t)(q0 + r) * HD + (size_t)h * D + c4;
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(y[0], y[1]), h1 = __floats2bfloat162_rn(y[2], y[3]);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t *>(&h0);
        pk.y = *reinterpret_cast<const uint32_t *>(&h1);
        *reinterpret_cast<uint2 *>(a.out + idx) = pk;
        if (a.out_lo) {
            const __nv_bfloat162 q0 = __floats2bfloat162_rn(y[0] - __low2float(h0), y[1] - __high2float(h0));
            const __nv_bfloat162 q1 = __floats2bfloat162_rn(y[2] - __low2float(h1), y[3] - __high2float(h1));
            pk.x = *reinterpret_cast<const uint32_t *>(&q0);
            pk.y = *reinterpret_cast<const uint32_t *>(&q1);
            *reinterpret_cast<uint2 *>(a.out_lo + idx) = pk;
        }
    }
    if (threadIdx.x == 0)
        a.counters[slot] = 0;  // ready for the next launch
}

}  // namespace

// Caches of up to this many 64-key tiles run in row-split mode (MEDUSA_ATTN_ROWS_MAX_TILES overrides, 0 = never).
static int rows_mode_max_tiles()
{
    static const int v = tuning_env("MEDUSA_ATTN_ROWS_MAX_TILES") ? atoi(tuning_env("MEDUSA_ATTN_ROWS_MAX_TILES")) : 8;
    return v;
}

size_t tree_attention_flash_workspace_bytes(int H, int q_tiles)
{
    const size_t slots = (size_t)H * (q_tiles > 0 ? q_tiles : 1);
    return slots * FLASH_MAX_SPLITS * (BQ * D + 2 * BQ) * sizeof(float) + slots * sizeof(int);
}

// The kernel's instantiations and their dynamic shared memory; the limit is raised once per device.
typedef void (*FlashKernel)(Args);
static FlashKernel flash_kernel(bool qlo, bool large)
{
    return qlo ? (large ? tree_attention_flash_kernel<true, true> : tree_attention_flash_kernel<true, false>)
               : (large ? tree_attention_flash_kernel<false, true> : tree_attention_flash_kernel<false, false>);
}
static cudaError_t flash_set_limits()
{
    static bool done[64] = {};
    if (!first_use_on_current_device(done))
        return cudaSuccess;
    for (int q = 0; q < 2; ++q)
        for (int l = 0; l < 2; ++l) {
            cudaError_t e = cudaFuncSetAttribute(flash_kernel(q, l), cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(q));
            if (e != cudaSuccess)
                return e;
        }
    return cudaSuccess;
}

cudaError_t launch_tree_attention_flash(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                        const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                        void *out_lo, float *lse, void *workspace, int T, int H, int Hkv, int L_max,
                                        int L_hint, cudaStream_t s, const void *q_lo, int mask_words, int n_seq,
                                        long long cache_seq_stride, int len_stride)
{
    {
        cudaError_t e = flash_set_limits();
        if (e != cudaSuccess)
            return e;
    }
    // One CTA per SM: the grid offers every head as many key ranges as fit one wave, the kernel uses the number
    // the true cache length asks for (the other CTAs leave at once).  L_hint is not needed for that.
    (void)L_hint;
    int splits = 148 / H > 0 ? 148 / H : 1;
    if (splits > FLASH_MAX_SPLITS) splits = FLASH_MAX_SPLITS;
    int tps = 0;
    if (const char *e = tuning_env("MEDUSA_ATTN_SPLITS")) {  // tuning aid: a fixed number of key ranges
        const int want = atoi(e);
        if (want > 0) {
            const int nt = ((L_hint < 0 || L_hint > L_max ? L_max : L_hint) + BKEY - 1) / BKEY;
            if (want < splits) splits = want;
            tps = nt > 0 ? (nt + splits - 1) / splits : 1;
        }
    }
    Args a;
    // n_seq > 1: a batch of sequences, one tile of 64 query rows each (T <= 64 is then the tree size of every sequence)
    const int q_tiles = n_seq > 1 ? n_seq : (T + BQ - 1) / BQ;
    const bool large = q_tiles > 1, qlo = q_lo != nullptr;
    a.batch = n_seq > 1 ? 1 : 0;
    a.cache_seq_stride = cache_seq_stride;
    a.len_stride = len_stride;
    const size_t slots = (size_t)H * q_tiles;
    a.q = (const bf16 *)q; a.k_new = (const bf16 *)k_new; a.v_new = (const bf16 *)v_new;
    a.q_lo = (const bf16 *)q_lo;
    a.k_cache = (const bf16 *)k_cache; a.v_cache = (const bf16 *)v_cache;
    a.cache_len = cache_len; a.mask = mask; a.mask_words = mask_words > 0 ? mask_words : 1;
    a.out = (bf16 *)out; a.out_lo = (bf16 *)out_lo; a.lse = lse;
    a.ws_o = (float *)workspace;
    a.ws_ml = a.ws_o + slots * FLASH_MAX_SPLITS * BQ * D;
    a.counters = (int *)(a.ws_ml + slots * FLASH_MAX_SPLITS * 2 * BQ);
    a.T = T; a.H = H; a.Hkv = Hkv; a.L_max = L_max; a.tiles_per_split = tps; a.max_splits = FLASH_MAX_SPLITS;
    a.rows_max_tiles = rows_mode_max_tiles();
    dim3 grid(H, splits, q_tiles);
    launch_pdl(flash_kernel(qlo, large), dim3(grid), dim3(THREADS), (size_t)smem_bytes(qlo), s, a);
    return cudaGetLastError();
}

}  // namespace medusa

// ------------------------------------------------------------------------------------------------------
// Allocation-free entry point (declared in include/medusa.h as medusa_tree_attention_static).
//
// Some callers cannot allocate device memory when they want to run tree attention: a serving runtime that
// has handed its whole memory budget to a pool of its own, code running where cudaMalloc would implicitly
// synchronise the device at a bad moment, or a caller that simply has no context object of this library.
// For them the split-KV partials live in the fixed array below instead of a context's workspace.  The array
// is part of the library image: every GPU that loads the library holds these bytes until the process exits.
namespace medusa {
namespace {

constexpr int STATIC_MAX_HEADS = 64;   // largest head count the fixed scratch can serve
constexpr int STATIC_MAX_SPLITS = 4;   // key ranges per head (a context's workspace allows FLASH_MAX_SPLITS)
constexpr size_t STATIC_O_FLOATS = (size_t)STATIC_MAX_HEADS * STATIC_MAX_SPLITS * BQ * D;
constexpr size_t STATIC_ML_FLOATS = (size_t)STATIC_MAX_HEADS * STATIC_MAX_SPLITS * 2 * BQ;
constexpr size_t STATIC_SCRATCH_BYTES = (STATIC_O_FLOATS + STATIC_ML_FLOATS) * sizeof(float) + STATIC_MAX_HEADS * sizeof(int);

// about 8.1 MiB: partial outputs, their (max, sum) pairs, and one arrival counter per head
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
unsigned char *g_static_scratch_addr[STATIC_MAX_DEVICES] = {};  // device address of the array, per device

}  // namespace
}  // namespace medusa

extern "C" int32_t medusa_tree_attention_static(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                                const void *v_cache, const int32_t *cache_len, const uint64_t *mask,
                                                int32_t T, int32_t H, int32_t L_max, int32_t L_hint, void *out, float *lse,
                                                void *stream)
{
    using namespace medusa;
    if (!q || !k_new || !v_new || !cache_len || !mask || !out || (L_max > 0 && (!k_cache || !v_cache)))
        return MEDUSA_ERR_INVALID_ARG;
    const uintptr_t al = (uintptr_t)q | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)out;
    if (al & 15u)
        return MEDUSA_ERR_INVALID_ARG;
    if (T < 1 || T > BQ || H < 1 || L_max < 0) {
        fprintf(stderr, "medusa_tree_attention_static: T must be 1..%d, H >= 1, L_max >= 0 (got T=%d H=%d L_max=%d)\n", BQ, T, H, L_max);
        return MEDUSA_ERR_SHAPE;
    }
    if (H > STATIC_MAX_HEADS) {
        fprintf(stderr, "medusa_tree_attention_static: %d heads exceed the fixed scratch, which serves at most %d heads; "
                        "use medusa_tree_attention with a context instead\n", H, STATIC_MAX_HEADS);
        return MEDUSA_ERR_SHAPE;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES)
        return MEDUSA_ERR_CUDA;
    if (!g_static_scratch_addr[dev]) {
        // One-time set-up on this device (the current one): in host code the array's name is only a stand-in,
        // the kernel needs the address the runtime resolves for this device.
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) {
            fprintf(stderr, "medusa_tree_attention_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
            return MEDUSA_ERR_CUDA;
        }
        e = flash_set_limits();
        if (e != cudaSuccess) {
            fprintf(stderr, "medusa_tree_attention_static: cudaFuncSetAttribute failed: %s\n", cudaGetErrorString(e));
            return MEDUSA_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = (unsigned char *)p;
    }
    cudaStream_t s = (cudaStream_t)stream;
    float *base = (float *)g_static_scratch_addr[dev];
    Args a;
    a.q = (const bf16 *)q; a.k_new = (const bf16 *)k_new; a.v_new = (const bf16 *)v_new;
    a.q_lo = nullptr;
    a.batch = 0; a.len_stride = 0; a.cache_seq_stride = 0;
    a.k_cache = (const bf16 *)k_cache; a.v_cache = (const bf16 *)v_cache;
    a.cache_len = cache_len; a.mask = mask; a.mask_words = 1; a.out = (bf16 *)out; a.out_lo = nullptr; a.lse = lse;
    a.ws_o = base;
    a.ws_ml = base + STATIC_O_FLOATS;
    a.counters = (int *)(base + STATIC_O_FLOATS + STATIC_ML_FLOATS);
    // the arrival counters must start at zero; the partials are fully rewritten before they are read
    if (cudaMemsetAsync(a.counters, 0, STATIC_MAX_HEADS * sizeof(int), s) != cudaSuccess)
        return MEDUSA_ERR_CUDA;
    if (L_hint > L_max || L_hint < 0) L_hint = L_max;
    const int nt = (L_hint + BKEY - 1) / BKEY;
    int tps = (nt * H + 2 * 148 - 1) / (2 * 148);
    if (tps < 1) tps = 1;
    int splits = nt > 0 ? (nt + tps - 1) / tps : 1;
    if (splits > STATIC_MAX_SPLITS) {
        tps = (nt + STATIC_MAX_SPLITS - 1) / STATIC_MAX_SPLITS;
        splits = (nt + tps - 1) / tps;
    }
    a.T = T; a.H = H; a.Hkv = H; a.L_max = L_max; a.tiles_per_split = tps; a.max_splits = STATIC_MAX_SPLITS;
    a.rows_max_tiles = rows_mode_max_tiles();
    cudaError_t e = launch_pdl(flash_kernel(false, false), dim3(H, splits), dim3(THREADS), (size_t)smem_bytes(false), s, a);
    return e == cudaSuccess ? MEDUSA_OK : MEDUSA_ERR_CUDA;
}

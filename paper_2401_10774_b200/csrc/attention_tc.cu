// Tree attention on the tcgen05 tensor cores (paper Sec. 2.1.2 "Tree Attention"; App. G Table 5 rows QK^T / PV
// for "parallel decoding"), bf16, head dim 128, T <= 64 tree queries per head against {cache 0..L-1} + {tree}.
//
// One CTA = one head x one contiguous range of 128-key cache tiles (split-KV; the last range also takes the
// tree's own keys under the ancestor mask).  Per tile two MMAs run entirely out of tensor memory on the A side:
//     S[128][128]  = Qp[128][128 dims] (TMEM) * K_tile[128 keys][128 dims]^T (shared memory, K-major)
//     O'[128][128] = P[128][128 keys] (TMEM) * V_tile[128 keys][128 dims]    (shared memory, MN-major)
// Q is a split activation: both bf16 planes sit in tensor memory and S = Q_hi K^T + Q_lo K^T, so the rounding of q to
// one plane does not reach the softmax (same accuracy as the mma.sync kernel).  Tensor memory is used to the last
// column -- two score buffers, the P V accumulator, the two planes of Q -- so P has no region of its own: P of tile
// i is written over the first 64 columns of the score buffer it was computed from, once both threads of a lane have
// read their scores, and that buffer takes new scores only after the P V MMA has read P out of it.
// The 64 query rows are stored twice (TMEM lanes r and 64 + r), and the two copies split every tile's keys: copy 0
// owns keys 0..63, copy 1 keys 64..127; the other half of a copy's P columns is written as zero.  Each copy keeps
// its own running maximum and sum, so the copies never talk during the loop and are merged once at the end like two
// key ranges.  Two threads share a lane (32 of the copy's 64 keys, 64 of the 128 output columns each) and exchange
// one partial maximum per tile through shared memory.  The running output stays in registers:
// o = o * 2^(m_old - m_new) + O', with O' read back from TMEM after every tile (no TMEM read-modify-write).
//
// Warp roles (352 threads): warps 0..7 softmax (warp w: lane quadrant w % 4, half w / 4), warp 8 issues the score
// MMAs one tile ahead, warp 10 the P V MMAs, warp 9 feeds a 3-stage K/V ring: full cache tiles by TMA (tensor maps
// over [H * L_max][128]), the ragged last cache tile and the tree's keys by 16-byte cp.async with zero fill, so no
// row past the cache length is ever read.  All hand-offs are mbarriers; every wait is bounded, and after an expired
// wait all further waits return at once (the loops keep their trip counts, so no barrier is left short), the CTA
// reports MEDUSA_ERR_TIMEOUT and stores nothing.
// The partial results of the key ranges ([column quad][row][4] floats, so that warps write and read 512 contiguous
// bytes) are combined by the last CTA of a head to arrive (ticket), in range order; the workspace has the size of
// the mma.sync kernel's (attention_flash.cu).  In steady state the loop streams K/V at ~6 TB/s; the kernel is the
// faster of the two from about 2048 cached keys on as a stand-alone operation and from about 1536 inside a decode step.
#include <cuda.h>

#include <unordered_map>

#include "common.cuh"
#include "gemm_tc.h"
#include "kernels.h"
#include "pdl.cuh"

namespace medusa {

namespace {

constexpr int D = 128;
constexpr int BQ = 64;           // query rows
constexpr int BKEY = 128;        // keys per tile
constexpr int STAGES = 3;
constexpr int THREADS = 352;     // 8 softmax warps, 2 MMA warps (scores / P V), 1 producer warp
constexpr int KSUB_BYTES = BKEY * 128;   // [128 keys][64 dims]
constexpr int K_BYTES = 2 * KSUB_BYTES;
constexpr int STAGE_BYTES = 2 * K_BYTES; // K then V
constexpr int TAIL_BYTES = 4096;         // barriers and exchange buffers (struct Smem)
constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + TAIL_BYTES;
constexpr float LOG2E = 1.4426950408889634f;
constexpr uint32_t TMEM_COLS = 512;
// S0: 0..127, S1: 128..255, O': 256..383, Q lo plane: 384..447, Q hi plane: 448..511.  P of tile i is written over the
// first 64 columns of the score buffer S(i & 1) it was computed from, once both threads of a lane have read their scores.
constexpr uint32_t O_COL = 256, QLO_COL = 384, Q_COL = 448;
constexpr int MAX_SPLITS = FLASH_MAX_SPLITS;

struct Smem {
    uint64_t kv_full[STAGES], kv_empty[STAGES], s_full[2], s_empty[2], p_full, o_full, o_empty, q_full, done;
    uint32_t tmem_base;
    volatile int failed;
    int ticket;
    float mx[2][2][2][BQ];  // [tile parity][row copy][key half][row] partial row maxima
    float lx[2][2][BQ];     // [row copy][key half][row] partial row sums
    float mm[BQ], ml[BQ];   // second copy's (max, sum) for the final merge
};
static_assert(sizeof(Smem) <= TAIL_BYTES, "Smem must fit its slot");

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :
                 : "r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait.  Once any wait of the CTA has expired (`*failed`), every later wait returns immediately.
__device__ __forceinline__ void mbar_wait(uint64_t *bar, uint32_t parity, volatile int *failed, uint32_t limit)
{
    const uint32_t addr = smem_u32(bar);
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok)
                     : "r"(addr), "r"(parity)
                     : "memory");
        if (ok)
            return;
        if (*failed)
            return;
    }
    *failed = 1;
}

// 16-byte chunk c8 (0..7) of 128-byte row r inside a 1024-byte-aligned sub-tile: the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int r, int c8) { return (uint32_t)(r * 128 + ((c8 ^ (r & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int sz = valid ? 16 : 0;  // 0: zero fill
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// makes this thread's completed shared-memory writes visible to the tensor core's (asynchronous proxy) reads
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// shared-memory operand descriptors, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;              // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;    // stride between 8-row groups
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// MN-major operand (V: rows are keys = the MMA's K, 64 output dims per 128-byte row): the next 64 dims are
// KSUB_BYTES further, the next 8 keys 1024 bytes further
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(KSUB_BYTES >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// instruction descriptors: D fp32, A and B bf16, M = 128
constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BKEY >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);  // N = 128 keys
constexpr uint32_t IDESC_O = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) /* B is MN-major */ | ((uint32_t)(D >> 3) << 17) |
                             ((uint32_t)(128 >> 4) << 24);

// The whole MMA warp runs the issue loop convergently (descriptor arithmetic stays warp-uniform); the instructions
// themselves are predicated on `leader` (lane 0) instead of sitting in a divergent branch.
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred p, q;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "setp.ne.b32 q, %5, 0;\n\t"
                 "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :
                 : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred q;\n\t"
                 "setp.ne.b32 q, %1, 0;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                 ::"r"(smem_u32(bar)), "r"(leader) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v)
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i)
        v[i] = __uint_as_float(r[i]);
}
// the four warps that work on one copy of the rows (128 threads) meet on barrier 1 + copy
__device__ __forceinline__ void copy_bar(int copy) { asm volatile("bar.sync %0, 128;" ::"r"(1 + copy) : "memory"); }
// MMA with the A operand in tensor memory (lane = row, two bf16 per 32-bit column)
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred p, q;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "setp.ne.b32 q, %5, 0;\n\t"
                 "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 :
                 : "r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
                 : "memory");
}
// 16 / 32 columns of this warp's 32 TMEM lanes, one row per thread
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
                   "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x)  // 2^x, -inf -> 0
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 16 columns of this warp's 32 TMEM lanes
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i)
        v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

struct Args {
    const bf16 *q, *q_lo, *k_new, *v_new;   // [T][H][D]; q_lo (nullable): the second bf16 plane of a split q
    const bf16 *k_cache, *v_cache;   // [H][L_max][D]
    const int32_t *cache_len;
    const uint64_t *mask;            // [T]
    bf16 *out, *out_lo;              // [T][H][D]; out_lo nullable
    float *lse;                      // nullable [T][H]
    float *ws_o;                     // [H][MAX_SPLITS][64][128] unnormalised partial outputs
    float *ws_ml;                    // [H][MAX_SPLITS][2][64] running max (log2 domain) and sum
    int *counters;                   // [H] arrival tickets, zero between launches
    int32_t *status;                 // device status word
    int T, H, L_max, tiles_per_split;
    int Hkv;                         // key/value heads; query head h reads key/value head h / (H / Hkv)
    uint32_t spin_limit;             // polls before a bounded wait gives up
    int withhold;                    // test hook: CTA (0, 0)'s producer delivers no tile, so its consumers' waits expire
};

__global__ void __launch_bounds__(THREADS, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, Args a)
{
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Smem *sm = (Smem *)(ring + STAGES * STAGE_BYTES);
    const int h = blockIdx.x, sp = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int L = min(max(*a.cache_len, 0), a.L_max);  // a length outside [0, L_max] would index past the caches
    const int nt = (L + BKEY - 1) / BKEY;
    const int n_cache_splits = (nt + a.tiles_per_split - 1) / a.tiles_per_split;
    // the range size was chosen on the host from an upper bound of the length; should the cache be longer than that,
    // the grid's last row takes all the remaining tiles (slower, still complete)
    const int n_active = min(n_cache_splits > 0 ? n_cache_splits : 1, (int)gridDim.y);
    if (sp >= n_active)
        return;
    const int tile0 = sp * a.tiles_per_split;
    const bool has_tree = sp == n_active - 1;
    const int tile1 = has_tree ? nt : min(nt, tile0 + a.tiles_per_split);
    const int n_tiles = (tile1 - tile0) + (has_tree ? 1 : 0);  // >= 1
    const size_t HD = (size_t)a.H * D;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm->kv_full[s], 1);   // the stage's producer warp
            mbar_init(&sm->kv_empty[s], 1);  // tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm->s_full[b], 1);
            mbar_init(&sm->s_empty[b], 1);   // tcgen05.commit of the P V MMA that read this buffer's P
        }
        mbar_init(&sm->p_full, 8);
        mbar_init(&sm->o_full, 1);
        mbar_init(&sm->o_empty, 8);
        mbar_init(&sm->q_full, 8);
        mbar_init(&sm->done, 2);  // one tcgen05.commit per MMA warp
        sm->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();  // barriers are initialised: the producer warp starts copying at once
    // what the softmax threads carry out of the tile loop
    const bool softmax_warp = warp < 8;
    const int quad = warp & 3;             // TMEM lane quadrant
    const int copy = quad >> 1;            // copy 0 (lanes 0..63) takes keys 0..63 of every tile, copy 1 keys 64..127
    const int hf = warp >> 2;              // half of the copy's 64 keys / half of the 128 output columns
    const int r = (quad & 1) * 32 + lane;  // query row of a softmax thread
    float m = -INFINITY, l = 0.f;
    float o[64];
#pragma unroll
    for (int i = 0; i < 64; ++i)
        o[i] = 0.f;
    // Q row r, dims hf*64..: requested now, stored to tensor memory once that is allocated
    uint32_t qv[32], qlv[32];
    const bool has_qlo = a.q_lo != nullptr;
    if (softmax_warp) {
        const size_t qoff = (size_t)min(r, a.T - 1) * HD + (size_t)h * D + hf * 64;
        const uint4 *src = reinterpret_cast<const uint4 *>(a.q + qoff);
        const uint4 *src_lo = reinterpret_cast<const uint4 *>((has_qlo ? a.q_lo : a.q) + qoff);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = r < a.T ? src[j] : make_uint4(0u, 0u, 0u, 0u);
            qv[4 * j] = v.x; qv[4 * j + 1] = v.y; qv[4 * j + 2] = v.z; qv[4 * j + 3] = v.w;
            const uint4 u = r < a.T && has_qlo ? src_lo[j] : make_uint4(0u, 0u, 0u, 0u);
            qlv[4 * j] = u.x; qlv[4 * j + 1] = u.y; qlv[4 * j + 2] = u.z; qlv[4 * j + 3] = u.w;
        }
    }
    uint32_t tmem = 0;
    volatile int *failed = &sm->failed;
    if (warp != 9) {
        // everyone but the producer meets again once warp 8 has allocated the tensor memory
        if (warp == 8) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(TMEM_COLS));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync 3, %0;" ::"n"(THREADS - 32) : "memory");
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem = sm->tmem_base;
    }

    if (warp == 9) {
        // ------------------------------------------------------------ producer warp
        // Full 128-key cache tiles come by TMA (four boxes of 64 dims x 128 keys: K and V, two dim halves each;
        // rows = head * L_max + key); the ragged last cache tile and the tree's own keys by 16-byte asynchronous
        // copies with zero fill, so that no row beyond the cache length is ever read.
        const int hk = h / (a.H / a.Hkv);
        const int n_deliver = a.withhold && h == 0 && sp == 0 ? 0 : n_tiles;
        for (int i = 0; i < n_deliver; ++i) {
            const int st = i % STAGES;
            uint8_t *stage = ring + st * STAGE_BYTES;
            if (i >= STAGES)
                mbar_wait(&sm->kv_empty[st], ((i / STAGES) - 1) & 1, failed, a.spin_limit);
            const int ct = tile0 + i;
            if (ct < tile1 && (ct + 1) * BKEY <= L) {
                if (lane == 0) {
                    const int row = hk * a.L_max + ct * BKEY;
                    mbar_expect_tx(&sm->kv_full[st], STAGE_BYTES);
                    tma_load_2d(stage, &mapK, 0, row, &sm->kv_full[st]);
                    tma_load_2d(stage + KSUB_BYTES, &mapK, 64, row, &sm->kv_full[st]);
                    tma_load_2d(stage + K_BYTES, &mapV, 0, row, &sm->kv_full[st]);
                    tma_load_2d(stage + K_BYTES + KSUB_BYTES, &mapV, 64, row, &sm->kv_full[st]);
                }
                __syncwarp();
                continue;
            }
            const bf16 *ksrc, *vsrc;
            size_t stride;
            int n_valid;
            if (ct < tile1) {
                const size_t o0 = ((size_t)hk * a.L_max + (size_t)ct * BKEY) * D;
                ksrc = a.k_cache + o0; vsrc = a.v_cache + o0; stride = D; n_valid = min(BKEY, L - ct * BKEY);
            } else {
                ksrc = a.k_new + (size_t)hk * D; vsrc = a.v_new + (size_t)hk * D; stride = (size_t)a.Hkv * D; n_valid = a.T;
            }
            const uint32_t kb = smem_u32(stage), vb = kb + K_BYTES;
#pragma unroll 8
            for (int idx = lane; idx < BKEY * 16; idx += 32) {
                const int row = idx >> 4, c = idx & 15;
                const bool ok = row < n_valid;
                const size_t off = (size_t)(ok ? row : 0) * stride + c * 8;
                const uint32_t dst = (uint32_t)((c >> 3) * KSUB_BYTES) + sw128(row, c & 7);
                cp_async16(kb + dst, ksrc + off, ok);
                cp_async16(vb + dst, vsrc + off, ok);
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_async_smem();
            __syncwarp();
            if (lane == 0)
                mbar_arrive(&sm->kv_full[st]);
        }
    } else if (warp == 8 || warp == 10) {
        // ------------------------------------------------------------ MMA issuers (lane 0 of a convergent warp each)
        // warp 8 issues the score MMAs one tile ahead, warp 10 the P V MMAs: an MMA costs its issuing thread about
        // as long as it takes the tensor core at these shapes, so two threads issue side by side.
        const uint32_t leader = lane == 0 ? 1u : 0u;
        if (warp == 8) {
            mbar_wait(&sm->q_full, 0, failed, a.spin_limit);  // Q sits in tensor memory
            for (int i = 0; i < n_tiles; ++i) {
                mbar_wait(&sm->kv_full[i % STAGES], (i / STAGES) & 1, failed, a.spin_limit);
                if (i >= 2)  // the P V MMA of tile i - 2 has read its P out of this buffer
                    mbar_wait(&sm->s_empty[i & 1], ((i >> 1) - 1) & 1, failed, a.spin_limit);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t dk = desc_kmajor(smem_u32(ring + (i % STAGES) * STAGE_BYTES));
                const uint32_t td = tmem + (uint32_t)((i & 1) * BKEY);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {  // 16 dims per step: 8 packed columns of Q, 32 bytes inside a K row
                    const uint64_t ko = (uint64_t)(((ks >> 2) * KSUB_BYTES + (ks & 3) * 32) >> 4);
                    umma_ts(td, tmem + Q_COL + (uint32_t)(ks * 8), dk + ko, IDESC_S, ks ? 1u : 0u, leader);
                }
                if (has_qlo) {  // S += Q_lo K^T: q's rounding to one bf16 plane does not reach the softmax
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t ko = (uint64_t)(((ks >> 2) * KSUB_BYTES + (ks & 3) * 32) >> 4);
                        umma_ts(td, tmem + QLO_COL + (uint32_t)(ks * 8), dk + ko, IDESC_S, 1u, leader);
                    }
                }
                umma_commit(&sm->s_full[i & 1], leader);
            }
        } else {
            for (int i = 0; i < n_tiles; ++i) {
                mbar_wait(&sm->p_full, i & 1, failed, a.spin_limit);
                if (i >= 1)
                    mbar_wait(&sm->o_empty, (i - 1) & 1, failed, a.spin_limit);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t dv = desc_mnmajor(smem_u32(ring + (i % STAGES) * STAGE_BYTES) + K_BYTES);
#pragma unroll
                for (int kk = 0; kk < BKEY / 16; ++kk)  // 16 keys per step: 8 packed columns of P, 16 V rows of 128 bytes
                    umma_ts(tmem + O_COL, tmem + (uint32_t)((i & 1) * BKEY + kk * 8), dv + (uint64_t)((kk * 2048) >> 4), IDESC_O,
                            kk ? 1u : 0u, leader);
                umma_commit(&sm->s_empty[i & 1], leader);  // P has been read: the buffer may take the scores of tile i + 2
                umma_commit(&sm->o_full, leader);
                umma_commit(&sm->kv_empty[i % STAGES], leader);  // the scores of this stage were read before its P existed
            }
        }
        // every MMA of both warps has retired before the accumulators are freed, also after an expired wait
        umma_commit(&sm->done, leader);
        const uint32_t addr = smem_u32(&sm->done);
        for (uint32_t it = 0; it < a.spin_limit; ++it) {
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(addr) : "memory");
            if (ok)
                break;
        }
    } else if (softmax_warp) {
        // ------------------------------------------------------------ softmax: thread = (row r, row copy, half hf)
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint64_t mask_r = r < a.T ? a.mask[r] : 0ull;
        const float sc = rsqrtf((float)D) * LOG2E;
        {
            // Q: 32 packed columns of this thread's lane in each plane
            tmem_st16(tmem + lane_addr + Q_COL + (uint32_t)(hf * 32), qv);
            tmem_st16(tmem + lane_addr + Q_COL + (uint32_t)(hf * 32 + 16), qv + 16);
            tmem_st16(tmem + lane_addr + QLO_COL + (uint32_t)(hf * 32), qlv);
            tmem_st16(tmem + lane_addr + QLO_COL + (uint32_t)(hf * 32 + 16), qlv + 16);
            tmem_st_wait();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                mbar_arrive(&sm->q_full);
        }
        float c_prev = 0.f;  // rescale factor that belongs to the tile whose P V is still in TMEM
        for (int i = 0; i <= n_tiles; ++i) {
            float c = 0.f;
            if (i < n_tiles) {
                float s[32];
                mbar_wait(&sm->s_full[i & 1], (i >> 1) & 1, failed, a.spin_limit);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                tmem_ld32(tmem + lane_addr + (uint32_t)((i & 1) * BKEY + copy * 64 + hf * 32), s);
                const int ct = tile0 + i;
                const bool tree_tile = ct >= tile1;
                const int kj0 = copy * 64 + hf * 32;  // first key of this thread inside the tile
                const int key0 = ct * BKEY + kj0;
                if (tree_tile || key0 + 32 > L) {  // warp-uniform: only the tree tile and the last cache tile mask
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int kj = kj0 + j;  // the tree has at most 64 keys: all of them belong to copy 0
                        const bool v = tree_tile ? (kj < 64 && ((mask_r >> (kj & 63)) & 1ull) != 0ull) : key0 + j < L;
                        s[j] = v ? s[j] : -INFINITY;
                    }
                }
                float t8[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    t8[j] = fmaxf(fmaxf(s[j], s[j + 8]), fmaxf(s[j + 16], s[j + 24]));
                const float lmax = fmaxf(fmaxf(fmaxf(t8[0], t8[4]), fmaxf(t8[1], t8[5])), fmaxf(fmaxf(t8[2], t8[6]), fmaxf(t8[3], t8[7]))) * sc;
                sm->mx[i & 1][copy][hf][r] = lmax;
                copy_bar(copy);
                const float mn = fmaxf(m, fmaxf(lmax, sm->mx[i & 1][copy][hf ^ 1][r]));
                const float ms = mn == -INFINITY ? 0.f : mn;
                c = ex2(m - ms);  // m = -inf gives 0
                m = mn;
                float ps0 = 0.f, ps1 = 0.f;
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float p0 = ex2(fmaf(s[2 * j], sc, -ms)), p1 = ex2(fmaf(s[2 * j + 1], sc, -ms));
                    ps0 += p0;
                    ps1 += p1;
                    pk[j] = pack_bf16(p0, p1);
                }
                l = l * c + (ps0 + ps1);
                // P goes over the first 64 columns of the score buffer it came from: both threads of this lane have read
                // their scores (they met on the copy's barrier above), and the buffer is not written again before the
                // P V MMA of this tile has read P.  The half that belongs to the other copy's keys is zero.
                {
                    uint32_t z[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        z[j] = 0u;
                    tmem_st16(tmem + lane_addr + (uint32_t)((i & 1) * BKEY + copy * 32 + hf * 16), pk);
                    tmem_st16(tmem + lane_addr + (uint32_t)((i & 1) * BKEY + (1 - copy) * 32 + hf * 16), z);
                }
                tmem_st_wait();
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(&sm->p_full);
            }
            if (i > 0) {
                // o = o * 2^(m_old - m_new) + P V of tile i - 1 (its MMA ran while this tile's scores were processed)
                mbar_wait(&sm->o_full, (i - 1) & 1, failed, a.spin_limit);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int q2 = 0; q2 < 2; ++q2) {
                    float t[32];
                    tmem_ld32(tmem + lane_addr + O_COL + (uint32_t)(hf * 64 + q2 * 32), t);
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        o[q2 * 32 + j] = o[q2 * 32 + j] * c_prev + t[j];
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(&sm->o_empty);
            }
            c_prev = c;
        }
        sm->lx[copy][hf][r] = l;
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 8)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS));
    if (sm->failed && threadIdx.x == 0)
        atomicExch(a.status, MEDUSA_ERR_TIMEOUT);
    const bool stores_ok = !sm->failed;
    // ---- merge the two row copies (each saw half of every tile's keys): copy 1 hands (m, l, o) to copy 0
    // [32 column quads][64 rows][4]: a warp's lanes are consecutive rows, 16 bytes each (no bank conflicts); the ring is idle
    float *mo = reinterpret_cast<float *>(ring);
    if (softmax_warp) {
        l = sm->lx[copy][0][r] + sm->lx[copy][1][r];
        if (copy == 1) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
                *reinterpret_cast<float4 *>(mo + ((size_t)(hf * 16 + j) * BQ + r) * 4) = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
            if (hf == 0) {
                sm->mm[r] = m;
                sm->ml[r] = l;
            }
        }
    }
    __syncthreads();
    const bool owner = softmax_warp && copy == 0;
    if (owner) {
        const float mb = sm->mm[r], lb = sm->ml[r];
        const float mn = fmaxf(m, mb);
        const float ms = mn == -INFINITY ? 0.f : mn;
        const float ca = ex2(m - ms), cb = ex2(mb - ms);
        l = l * ca + lb * cb;
        m = mn;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float4 v = *reinterpret_cast<const float4 *>(mo + ((size_t)(hf * 16 + j) * BQ + r) * 4);
            o[4 * j] = o[4 * j] * ca + v.x * cb;
            o[4 * j + 1] = o[4 * j + 1] * ca + v.y * cb;
            o[4 * j + 2] = o[4 * j + 2] * ca + v.z * cb;
            o[4 * j + 3] = o[4 * j + 3] * ca + v.w * cb;
        }
    }
    __syncthreads();  // the ring is reused by the combine below

    if (n_active == 1) {
        // a single key range: normalise and write straight from the registers (64 columns = 128 bytes per thread)
        if (owner && r < a.T && stores_ok) {
            const float inv = l > 0.f ? 1.0f / l : 0.f;
            const size_t idx = (size_t)r * HD + (size_t)h * D + hf * 64;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float y0 = o[8 * j + 2 * e] * inv, y1 = o[8 * j + 2 * e + 1] * inv;
                    const __nv_bfloat162 hv = __floats2bfloat162_rn(y0, y1);
                    hi[e] = *reinterpret_cast<const uint32_t *>(&hv);
                    lo[e] = pack_bf16(y0 - __low2float(hv), y1 - __high2float(hv));
                }
                *reinterpret_cast<uint4 *>(a.out + idx + 8 * j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                if (a.out_lo)
                    *reinterpret_cast<uint4 *>(a.out_lo + idx + 8 * j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
            if (a.lse && hf == 0)
                a.lse[(size_t)r * a.H + h] = m / LOG2E + logf(l);
        }
        return;
    }
    // ---- partial result of this key range
    float *wo = a.ws_o + ((size_t)h * MAX_SPLITS + sp) * BQ * D;
    float *wml = a.ws_ml + ((size_t)h * MAX_SPLITS + sp) * 2 * BQ;
    if (owner) {
#pragma unroll
        for (int j = 0; j < 16; ++j)  // [column quad][row][4]: a warp writes 512 consecutive bytes per store
            *reinterpret_cast<float4 *>(wo + ((size_t)(hf * 16 + j) * BQ + r) * 4) = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        if (hf == 0) {
            wml[r] = m;
            wml[BQ + r] = l;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0)
        sm->ticket = atomicAdd(a.counters + h, 1);
    __syncthreads();
    if (sm->ticket != n_active - 1)
        return;
    // ---- last CTA of this head: combine the key ranges in range order.  Thread -> row tid % 64, columns
    // 32 * (tid / 64)..; every thread works out its row's weights itself from the (max, sum) records (no staging, no
    // barrier), and the lanes of a warp read consecutive rows of a column quad (512 contiguous bytes).
    __threadfence();
    const int tid = threadIdx.x;
    if (tid < 256) {
        const float *__restrict__ mlh = a.ws_ml + (size_t)h * MAX_SPLITS * 2 * BQ;
        const float *__restrict__ oh = a.ws_o + (size_t)h * MAX_SPLITS * BQ * D;
        const int row = tid & (BQ - 1), cg = tid >> 6;
        float mstar = -INFINITY;
        for (int s2 = 0; s2 < n_active; ++s2)
            mstar = fmaxf(mstar, mlh[(size_t)s2 * 2 * BQ + row]);
        const float msafe = mstar == -INFINITY ? 0.f : mstar;
        float lstar = 0.f;
        float acc[32];
#pragma unroll
        for (int j = 0; j < 32; ++j)
            acc[j] = 0.f;
        for (int s2 = 0; s2 < n_active; ++s2) {
            const float4 *src = reinterpret_cast<const float4 *>(oh + (size_t)s2 * BQ * D) + (size_t)(cg * 8) * BQ + row;
            float4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[j] = src[(size_t)j * BQ];
            const float w = ex2(mlh[(size_t)s2 * 2 * BQ + row] - msafe);
            lstar += w * mlh[(size_t)s2 * 2 * BQ + BQ + row];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                acc[4 * j] += w * v[j].x;
                acc[4 * j + 1] += w * v[j].y;
                acc[4 * j + 2] += w * v[j].z;
                acc[4 * j + 3] += w * v[j].w;
            }
        }
        if (a.lse && cg == 0 && row < a.T && stores_ok)
            a.lse[(size_t)row * a.H + h] = mstar / LOG2E + logf(lstar);
        if (row < a.T && stores_ok) {
            const float inv = lstar > 0.f ? 1.0f / lstar : 0.f;
            const size_t idx = (size_t)row * HD + (size_t)h * D + cg * 32;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float y0 = acc[8 * j + 2 * e] * inv, y1 = acc[8 * j + 2 * e + 1] * inv;
                    const __nv_bfloat162 hv = __floats2bfloat162_rn(y0, y1);
                    hi[e] = *reinterpret_cast<const uint32_t *>(&hv);
                    lo[e] = pack_bf16(y0 - __low2float(hv), y1 - __high2float(hv));
                }
                *reinterpret_cast<uint4 *>(a.out + idx + 8 * j) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                if (a.out_lo)
                    *reinterpret_cast<uint4 *>(a.out_lo + idx + 8 * j) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
    }
    if (tid == 0)
        a.counters[h] = 0;  // ready for the next launch
}

}  // namespace

cudaError_t launch_tree_attention_tc(const void *q, const void *k_new, const void *v_new, const void *k_cache,
                                     const void *v_cache, const int32_t *cache_len, const uint64_t *mask, void *out,
                                     void *out_lo, float *lse, void *workspace, int T, int H, int Hkv, int L_max,
                                     int L_hint, int32_t *status, cudaStream_t s, uint32_t spin_limit, int withhold,
                                     const void *q_lo)
{
    // TMA descriptors of the two caches ([Hkv * L_max rows][128 dims] bf16, boxes of 64 dims x 128 rows), encoded once
    // per distinct cache
    static std::unordered_map<uint64_t, TensorMap> maps;
    auto map_of = [&](const void *base) -> const TensorMap * {
        const uint64_t key = (uint64_t)(uintptr_t)base ^ ((uint64_t)Hkv << 52) ^ ((uint64_t)L_max << 40);
        auto it = maps.find(key);
        if (it == maps.end()) {
            TensorMap tm;
            if (!make_weight_map(&tm, base, Hkv * L_max, D))
                return nullptr;
            it = maps.emplace(key, tm).first;
        }
        return &it->second;
    };
    const TensorMap *mk = map_of(k_cache), *mv = map_of(v_cache);
    if (!mk || !mv)
        return cudaErrorInvalidValue;
    static bool attr_set[64] = {};
    if (first_use_on_current_device(attr_set)) {
        cudaError_t e = cudaFuncSetAttribute(tree_attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess)
            return e;
    }
    if (L_hint > L_max) L_hint = L_max;
    if (L_hint < 0) L_hint = 0;
    const int nt = (L_hint + BKEY - 1) / BKEY;
    // A CTA's time grows with its tiles, the combine with the number of key ranges: about sqrt(tiles) ranges
    // balances the two; one CTA per SM, so never more ranges than fill one wave.
    int want = 1;
    while (want * want < nt) ++want;
    const int one_wave = 148 / H > 0 ? 148 / H : 1;
    if (want > one_wave) want = one_wave;
    if (const char *e = tuning_env("MEDUSA_ATTN_SPLITS")) want = atoi(e) > 0 ? atoi(e) : want;
    int tps = nt > 0 ? (nt + want - 1) / want : 1;
    if (tps < 1) tps = 1;
    int splits = nt > 0 ? (nt + tps - 1) / tps : 1;
    if (splits > MAX_SPLITS) {
        tps = (nt + MAX_SPLITS - 1) / MAX_SPLITS;
        splits = (nt + tps - 1) / tps;
    }
    Args a;
    a.q = (const bf16 *)q; a.q_lo = (const bf16 *)q_lo; a.k_new = (const bf16 *)k_new; a.v_new = (const bf16 *)v_new;
    a.k_cache = (const bf16 *)k_cache; a.v_cache = (const bf16 *)v_cache;
    a.cache_len = cache_len; a.mask = mask; a.out = (bf16 *)out; a.out_lo = (bf16 *)out_lo; a.lse = lse;
    a.ws_o = (float *)workspace;
    a.ws_ml = a.ws_o + (size_t)H * MAX_SPLITS * BQ * D;
    a.counters = (int *)(a.ws_ml + (size_t)H * MAX_SPLITS * 2 * BQ);
    a.status = status;
    a.T = T; a.H = H; a.Hkv = Hkv; a.L_max = L_max; a.tiles_per_split = tps;
    a.spin_limit = spin_limit ? spin_limit : DEFAULT_SPIN_LIMIT;
    a.withhold = withhold;
    launch_pdl(tree_attention_tc_kernel, dim3(H, splits), dim3(THREADS), (size_t)SMEM_BYTES, s, *(const CUtensorMap *)mk,
               *(const CUtensorMap *)mv, a);
    return cudaGetLastError();
}

}  // namespace medusa

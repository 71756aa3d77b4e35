// Tensor-core GEMM for the backbone linears at M = tree size (paper App. G Table 5: "parallel decoding"
// XW_Q/K/V, XW_u/g/d on q candidate tokens).  With 64 tokens the product does 64 flops per weight byte: far
// left of the B200 ridge, so the kernel is an HBM streamer whose arithmetic must merely keep up -- which the
// CUDA cores cannot, hence tcgen05.
//
// Shape of the computation ("swap AB"): the weight rows are the MMA's M dimension, the tokens its N:
//     D[128 weight rows][128] (fp32, in TMEM) += W_tile[128][64 k] * [X_hi; X_lo][128][64 k]^T
// (one MMA of N = 128 per 16 k: columns t and 64 + t of a row are added in the epilogue).  Launches over more than 64
// tokens put up to four token tiles (two with both planes) behind one another in a stage; they form ONE B operand of up
// to 256 rows, so a k step is still a single MMA (N up to 256) and the weight tile is read once for all of them.  At
// 256 rows the kernel is no longer bound by HBM but by what an SM can take in: every CTA fetches its own copy of the
// activation tiles from the L2 (twice the bytes of its weight tile), about 4.7 TB/s over the chip, which caps the
// contraction near 400 (one plane) to 560 (two planes) TFLOP/s.
// W tiles come straight from HBM by TMA (128-byte swizzle, evict-first), the two bf16 planes of the split
// activation come from L2.
//
// Work distribution ("stream-K"): the (weight tile, k block) pairs of a launch form one flat sequence that is
// cut into gridDim.x equal contiguous ranges, one per persistent CTA.  Every SM therefore streams the same
// number of weight bytes whatever the matrix shape, and the TMA producer never drains between tiles.  A tile
// whose k blocks fall into several CTAs is produced as several fp32 partial planes ("pieces", numbered by
// CTA order); the kernel that consumes the projection adds a tile's pieces in that order (deterministic).
// The LM head writes straight into the logits, so it is distributed by whole tiles instead.
//
// Roles inside a CTA (192 threads, two CTAs per SM): warp 0 lane 0 issues TMA loads into a 3-stage ring, warp 1 lane 0 issues
// tcgen05.mma into one of two TMEM accumulators, warps 2-5 drain a finished accumulator with tcgen05.ld
// while the next one fills.  The weight loads of the first ring fill are issued before the kernel waits for
// its predecessor in the stream (programmatic dependent launch): weights never depend on it.
// Every mbarrier wait is bounded; on expiry the CTA records MEDUSA_ERR_TIMEOUT, stops storing, waits
// (bounded) for its loads in flight, frees its TMEM and returns.
#include <cuda.h>
#include <cstdlib>

#include "common.cuh"
#include "gemm_tc.h"

namespace medusa {

namespace {

constexpr int BM = 128;                 // weight rows per tile (UMMA M)
constexpr int BN = 64;                  // tokens
// MMA N per token tile: PL * BN -- the hi plane's 64 token rows, followed by the lo plane's when the activations come as
// two planes (PL = 2)
constexpr int BK = 64;                  // k elements per stage: one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int MAX_STAGES = 8;         // ring depth is a launch parameter (a.stages)
constexpr int A_BYTES = BM * BK * 2;    // 16 KiB
constexpr int B_BYTES = BN * BK * 2;    // 8 KiB per plane
// a stage: one weight tile and, for each of the launch's RT token tiles, the PL activation planes
constexpr int stage_bytes(int rt, int pl) { return A_BYTES + rt * pl * B_BYTES; }
constexpr int smem_bytes(int stages, int rt, int pl) { return stages * stage_bytes(rt, pl) + 1024 /* alignment slack */ + 256 /* barriers */; }
constexpr int THREADS = 192;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// bounded wait: false if the phase did not complete within `limit` polls
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, uint32_t limit)
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
            return true;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar, uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%2, %3}], [%4], %5;"
                 :
                 : "r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
                 : "memory");
}

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                     // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                     // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                     // layout: 128-byte swizzle
    return d;
}

// instruction descriptor: D fp32, A and B bf16, both K-major, N = n, M = 128
constexpr uint32_t idesc(int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24); }

// The MMA warp runs its loop convergently (descriptor arithmetic stays warp-uniform); the tcgen05 instructions
// are predicated on `leader` (lane 0) instead of sitting in a divergent branch.
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t IDESC, uint32_t accumulate,
                                     uint32_t leader)
{
    asm volatile("{\n\t.reg .pred p, q;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "setp.ne.b32 q, %5, 0;\n\t"
                 "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :
                 : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate), "r"(leader)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar, uint32_t leader)
{
    asm volatile("{\n\t.reg .pred q;\n\t"
                 "setp.ne.b32 q, %1, 0;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                 ::"r"(smem_u32(bar)), "r"(leader) : "memory");
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

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

struct Smem {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    volatile int failed;
};

// One contiguous run of k blocks inside one weight tile, and the partial plane it is written to.
struct Segment {
    int tile, kb0, nkb, piece;
};

// Iterates the segments of CTA `c` in order; every role of the CTA walks the same sequence.
struct SegmentIter {
    int KB, G, tiles, whole, c;
    long long total, x, x1;
    int tile_next;
    __device__ SegmentIter(const GemmTcArgs &a, int c_) : KB(a.KB), G(a.G), tiles(a.seg0_tiles + (a.n_seg - 1) * a.seg_tiles), whole(a.whole_tiles), c(c_)
    {
        total = (long long)tiles * KB;
        x = ((long long)c * total) / G;
        x1 = ((long long)(c + 1) * total) / G;
        tile_next = c;
    }
    __device__ bool next(Segment &s)
    {
        if (whole) {
            if (tile_next >= tiles) return false;
            s.tile = tile_next; s.kb0 = 0; s.nkb = KB; s.piece = 0;
            tile_next += G;
            return true;
        }
        if (x >= x1) return false;
        s.tile = (int)(x / KB);
        s.kb0 = (int)(x % KB);
        const long long end = min((long long)(s.tile + 1) * KB, x1);
        s.nkb = (int)(end - x);
        s.piece = c - gemm_tc_first_cta((long long)s.tile * KB, G, total);
        x = end;
        return true;
    }
};

// RT = token tiles (64 rows each) per launch, PL = activation planes (2: hi + lo, the default; 1: hi only).  The weight
// tile of a stage feeds RT MMAs of N = 64 PL, one per token tile, into RT accumulators of 64 PL columns; the accumulators
// are double-buffered, so a CTA holds 2 RT 64 PL tensor-memory columns: up to 256 leaves room for two CTAs per SM,
// 512 (RT PL = 4) means one CTA per SM with a deeper ring.
// OT: the result may be stored or accumulated transposed (a.out_t; the gradient projections of the heads' training)
template <int RT, int PL, bool OT = false>
__global__ void __launch_bounds__(THREADS, RT * PL <= 2 ? 2 : 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW0,
               const __grid_constant__ CUtensorMap mapW1, const __grid_constant__ CUtensorMap mapW2, GemmTcArgs a)
{
    constexpr int STAGE_BYTES = stage_bytes(RT, PL);
    constexpr int UMMA_N = PL * BN;              // MMA N of one token tile
    constexpr uint32_t IDESC = idesc(UMMA_N);
    constexpr uint32_t ACC_COLS = RT * UMMA_N;   // columns of one accumulator set (all token tiles of a segment)
    const int rt_n = min(RT, (a.T + BN - 1) / BN);  // token tiles that hold rows in this launch
    const uint32_t stage_tx = (uint32_t)(A_BYTES + rt_n * PL * B_BYTES);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the next kernel may start its prologue
    extern __shared__ uint8_t smem_raw[];
    // tiles must sit on 1024-byte boundaries for the 128-byte swizzle pattern
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int STAGES = a.stages;
    Smem *sm = (Smem *)(tiles + STAGES * STAGE_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm->full[s], 1);
            mbar_init(&sm->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm->acc_full[b], 1);
            mbar_init(&sm->acc_empty[b], 4);  // one arrival per epilogue warp
        }
        sm->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();  // barriers are initialised: the producer warp starts loading at once
    // The other warps meet again once warp 1 has allocated both accumulators (2 x 128 fp32 columns x 128 lanes): the
    // allocation can have to wait for tensor memory that a CTA of the preceding kernel still holds on this SM, and the
    // weight loads must not wait with it.
    uint32_t tmem_base = 0;
    if (warp != 0) {
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(2 * ACC_COLS));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync 1, %0;" ::"n"(THREADS - 32) : "memory");
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem_base = sm->tmem_base;
    }

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            // the activation planes of k block `k` for every token tile of the launch: hi rows, then lo rows
            auto load_x = [&](uint8_t *st, int k, uint64_t *bar) {
                for (int rt = 0; rt < rt_n; ++rt) {
                    tma_load_2d(st + A_BYTES + rt * PL * B_BYTES, &mapX, k, a.x_row_hi + rt * BN, bar, pol_keep);
                    if (PL == 2)
                        tma_load_2d(st + A_BYTES + rt * PL * B_BYTES + B_BYTES, &mapX, k, a.x_row_lo + rt * BN, bar, pol_keep);
                }
            };
            SegmentIter it(a, blockIdx.x);
            Segment sg;
            int n = 0;          // k blocks issued so far by this CTA
            int rs = 0;         // ring stage of k block n, and the parity of that stage's release one lap earlier
            uint32_t ph = 1;
            bool waited = false;  // has this thread waited for the preceding kernel yet
            int pend_k[MAX_STAGES], pend_n = 0;
            bool ok = !(a.withhold && blockIdx.x == 0);  // test hook: this CTA's loads are withheld, nothing is in flight
            while (ok && it.next(sg)) {
                // the first weight matrix may have its own number of tiles (a wider q beside narrower k and v)
                const int rest = sg.tile - a.seg0_tiles;
                const int seg = rest < 0 ? 0 : 1 + rest / a.seg_tiles;
                const int trow = (rest < 0 ? sg.tile : rest % a.seg_tiles) * BM;
                const CUtensorMap *mapW = seg == 0 ? &mapW0 : (seg == 1 ? &mapW1 : &mapW2);
                for (int i = 0; i < sg.nkb; ++i, ++n) {
                    const int s = rs;
                    if (n >= STAGES) {
                        if (!waited) {
                            // the ring is full of weight tiles: now wait for the producer of X, then add the X tiles
                            asm volatile("griddepcontrol.wait;" ::: "memory");
                            waited = true;
                            for (int p = 0; p < pend_n; ++p)
                                load_x(tiles + p * STAGE_BYTES, pend_k[p], &sm->full[p]);
                        }
                        if (sm->failed || !mbar_wait(&sm->empty[s], ph, a.spin_limit)) {
                            sm->failed = 1;
                            ok = false;
                            break;
                        }
                    }
                    uint8_t *st = tiles + s * STAGE_BYTES;
                    const int k = (sg.kb0 + i) * BK;
                    mbar_expect_tx(&sm->full[s], stage_tx);
                    // packed weights: tile (tile row, k block) is 16 KiB of consecutive bytes, rows of 64 elements
                    if (a.packed)
                        tma_load_2d(st, mapW, 0, ((trow >> 7) * a.KB + (sg.kb0 + i)) * BM, &sm->full[s], pol_stream);
                    else
                        tma_load_2d(st, mapW, k, trow, &sm->full[s], pol_stream);
                    if (waited) {
                        load_x(st, k, &sm->full[s]);
                    } else {
                        pend_k[pend_n++] = k;  // n < STAGES here, so stage index == pend index
                    }
                    if (++rs == STAGES) {
                        rs = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!waited && ok) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                for (int p = 0; p < pend_n; ++p)
                    load_x(tiles + p * STAGE_BYTES, pend_k[p], &sm->full[p]);
            }
        }
    } else if (warp == 1) {
        {
            // ---------------- MMA issuer (lane 0 of a convergent warp)
            const uint32_t leader = lane == 0 ? 1u : 0u;
            const uint32_t idesc_n = RT == 1 ? IDESC : idesc(rt_n * UMMA_N);  // N = all token tiles of this launch
            SegmentIter it(a, blockIdx.x);
            Segment sg;
            int st = 0, j = 0;       // ring stage and its phase, advanced per k block
            uint32_t ph = 0;
            bool ok = true;
            while (ok && it.next(sg)) {
                const int b = j & 1;
                if (j >= 2 && (sm->failed || !mbar_wait(&sm->acc_empty[b], ((j >> 1) - 1) & 1, a.spin_limit))) {
                    sm->failed = 1;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");  // the epilogue has drained this accumulator
                const uint32_t tmem_d = tmem_base + (uint32_t)b * ACC_COLS;
                for (int i = 0; i < sg.nkb; ++i) {
                    if (sm->failed || !mbar_wait(&sm->full[st], ph, a.spin_limit)) {
                        sm->failed = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t sa = smem_u32(tiles + st * STAGE_BYTES);
                    // the two activation planes of a token tile sit back to back in the stage: one 128-row K-major operand
                    // and the token tiles of the launch follow one another, so all of them are ONE K-major operand of
                    // rt_n * UMMA_N rows: a single MMA per k step reads the weight tile once for every token tile, and its
                    // accumulator columns rt * UMMA_N .. are where the epilogue looks for tile rt
                    const uint64_t da = umma_desc(sa), db = umma_desc(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t adv = (uint64_t)((k * UMMA_K * 2) >> 4);  // 32 bytes per step inside the swizzled row
                        umma(tmem_d, da + adv, db + adv, idesc_n, (i | k) ? 1u : 0u, leader);
                    }
                    umma_commit(&sm->empty[st], leader);  // frees the stage once these MMAs have read it
                    if (++st == STAGES) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
                umma_commit(&sm->acc_full[b], leader);   // accumulator of this segment complete
                ++j;
            }
        }
    } else {
        // ---------------- epilogue warps 2..5: TMEM lane quadrant = warp % 4
        const int quad = warp & 3;
        SegmentIter it(a, blockIdx.x);
        Segment sg;
        int j = 0;
        while (it.next(sg)) {
            const int b = j & 1;
            const bool ready = !sm->failed && mbar_wait(&sm->acc_full[b], (j >> 1) & 1, a.spin_limit);
            if (!ready) {
                sm->failed = 1;
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int rest = sg.tile - a.seg0_tiles;
            const int seg = rest < 0 ? 0 : 1 + rest / a.seg_tiles;
            const int n = (rest < 0 ? sg.tile : rest % a.seg_tiles) * BM + quad * 32 + lane;  // weight row inside the segment
            const int col0 = seg == 0 ? 0 : a.seg0_cols + (seg - 1) * a.seg_cols;            // its first output column
            float *out = a.P + (size_t)sg.piece * a.plane_stride + (size_t)col0 + n;
            const bool n_ok = n < (seg == 0 ? a.seg0_cols : a.seg_cols);
            // columns t (W * X_hi) and 64 + t (W * X_lo) of the same lane add up to the result for token t; both
            // loads of a half are in flight together, and a full 64-row store runs without per-row tests
#pragma unroll
            for (int rt = 0; rt < RT; ++rt) {
                if (rt >= rt_n)
                    break;
                const int tb = rt * BN;  // first token row of this tile inside the launch
                const bool all_rows = a.row0 <= tb && a.T >= tb + BN;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t v[32], w[32];
                    const uint32_t col = (uint32_t)b * ACC_COLS + (uint32_t)(rt * UMMA_N + half * 32);
                    tmem_ld32_issue(tmem_base + ((uint32_t)(quad * 32) << 16) + col, v);
                    if (PL == 2)
                        tmem_ld32_issue(tmem_base + ((uint32_t)(quad * 32) << 16) + col + BN, w);
                    tmem_ld_wait();
                    if (PL == 1) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            w[i] = 0u;  // +0.0f
                    }
                    if (OT && n_ok && a.out_t) {
                        // transposed result: this thread's 32 tokens are consecutive floats of row (col0 + n)
                        float *o = a.P + (size_t)(col0 + n) * a.ldt + (tb + half * 32);
                        if (all_rows) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                float4 r = a.out_t == 2 ? *reinterpret_cast<const float4 *>(o + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                                r.x += __uint_as_float(v[i]) + __uint_as_float(w[i]);
                                r.y += __uint_as_float(v[i + 1]) + __uint_as_float(w[i + 1]);
                                r.z += __uint_as_float(v[i + 2]) + __uint_as_float(w[i + 2]);
                                r.w += __uint_as_float(v[i + 3]) + __uint_as_float(w[i + 3]);
                                *reinterpret_cast<float4 *>(o + i) = r;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const int t = tb + half * 32 + i;
                                if (t >= a.row0 && t < a.T)
                                    o[i] = (a.out_t == 2 ? o[i] : 0.f) + (__uint_as_float(v[i]) + __uint_as_float(w[i]));
                            }
                        }
                    } else if (n_ok) {
                        float *o = out + (size_t)(tb + half * 32) * a.ldy;  // a warp writes 32 consecutive floats per token row
                        if (all_rows) {
#pragma unroll
                            for (int i = 0; i < 32; ++i, o += a.ldy)
                                *o = __uint_as_float(v[i]) + __uint_as_float(w[i]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i, o += a.ldy) {
                                const int t = tb + half * 32 + i;
                                if (t >= a.row0 && t < a.T)
                                    *o = __uint_as_float(v[i]) + __uint_as_float(w[i]);
                            }
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                mbar_arrive(&sm->acc_empty[b]);
            ++j;
        }
    }

    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (sm->failed) {
        if (threadIdx.x == 0) {
            atomicExch(a.status, MEDUSA_ERR_TIMEOUT);
            // loads already issued still write into this CTA's shared memory: wait (bounded) before exiting
            if (!a.withhold)
                for (int s = 0; s < STAGES; ++s)
                    (void)mbar_wait(&sm->full[s], 0, a.spin_limit);
        }
        __syncthreads();
    }
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * ACC_COLS));
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// rows x K bf16 row-major matrix, box = 64 k-elements x box_rows rows, 128-byte swizzle
bool make_tensor_map(TensorMap *out, const void *base, int rows, int K, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn)
        return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn((CUtensorMap *)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

static_assert(sizeof(TensorMap) == sizeof(CUtensorMap), "TensorMap must mirror CUtensorMap");

bool make_weight_map(TensorMap *out, const void *W, int N, int K) { return make_tensor_map(out, W, N, K, BM); }
bool make_packed_weight_map(TensorMap *out, const void *Wp, int N, int K)
{
    const long long tiles = (N + BM - 1) / BM, KB = (K + BK - 1) / BK;
    if (tiles * KB * BM > 0x7fffffffLL) return false;
    return make_tensor_map(out, Wp, (int)(tiles * KB * BM), BK, BM);
}
size_t packed_weight_elems(int N, int K) { return (size_t)((N + BM - 1) / BM) * ((K + BK - 1) / BK) * BM * BK; }

// Wp[((tile row * KB + k block) * 128 + r) * 64 + c] = W[(tile row * 128 + r) * K + k block * 64 + c], zero outside W:
// one block per (k block, tile row), 16 bytes per thread
__global__ void __launch_bounds__(1024) pack_weight_kernel(const bf16 *__restrict__ W, int N, int K, bf16 *__restrict__ Wp)
{
    const int kb = blockIdx.x, tr = blockIdx.y, KB = gridDim.x;
    const int r = threadIdx.x >> 3, c8 = threadIdx.x & 7;
    const int row = tr * BM + r, col = kb * BK + c8 * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < N && col + 8 <= K) {
        v = *reinterpret_cast<const uint4 *>(W + (size_t)row * K + col);
    } else if (row < N && col < K) {  // a ragged last k block: element by element
        bf16 t[8];
        for (int e = 0; e < 8; ++e)
            t[e] = col + e < K ? W[(size_t)row * K + col + e] : __float2bfloat16_rn(0.f);
        v = *reinterpret_cast<const uint4 *>(t);
    }
    *reinterpret_cast<uint4 *>(Wp + (((size_t)tr * KB + kb) * BM + r) * BK + c8 * 8) = v;
}
void launch_pack_weight(const void *W, int N, int K, void *Wp, cudaStream_t s)
{
    pack_weight_kernel<<<dim3((K + BK - 1) / BK, (N + BM - 1) / BM), 1024, 0, s>>>((const bf16 *)W, N, K, (bf16 *)Wp);
}
bool make_act_map(TensorMap *out, const void *X_planes, int K, int rows) { return make_tensor_map(out, X_planes, 2 * rows, K, BN); }

// CTAs resident per SM and TMA ring depth; MEDUSA_GEMM_CTAS_PER_SM / MEDUSA_GEMM_STAGES override for tuning
static int env_int(const char *name, int dflt, int lo, int hi)
{
    const char *v = tuning_env(name);
    if (!v) return dflt;
    int x = atoi(v);
    return x < lo ? lo : (x > hi ? hi : x);
}
int gemm_tc_ctas_per_sm() { static int v = env_int("MEDUSA_GEMM_CTAS_PER_SM", 2, 1, 4); return v; }
int gemm_tc_stages()
{
    static int v = env_int("MEDUSA_GEMM_STAGES", gemm_tc_ctas_per_sm() == 1 ? 6 : (gemm_tc_ctas_per_sm() == 2 ? 3 : 2), 2, MAX_STAGES);
    return v;
}

// Token tiles per launch: one for up to 64 rows, two for more (the weight stream then serves both tiles); with a
// single activation plane four tiles fit the tensor memory, so up to 256 rows share one weight stream.
int gemm_tc_row_tiles(int T, int planes) { return T > 2 * BN && planes == 1 ? 4 : (T > BN ? 2 : 1); }
// CTAs per SM and ring depth by (token tiles, planes): two CTAs per SM while 2 * RT * PL * 64 columns fit 256
static int cfg_ctas_per_sm(int rt, int pl) { return rt * pl <= 2 ? gemm_tc_ctas_per_sm() : 1; }
static int cfg_stages(int rt, int pl)
{
    if (rt == 1 && pl == 2) return gemm_tc_stages();  // 32 KiB stages, the tuned default
    if (rt * pl <= 2) return rt == 1 ? 4 : 3;         // (1,1): 24 KiB x 4;  (2,1): 32 KiB x 3
    return 4;                                         // (2,2) and (4,1): 48 KiB x 4, one CTA per SM
}

int gemm_tc_num_ctas(int row_tiles, int planes)
{
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
    }
    return sms * cfg_ctas_per_sm(row_tiles, planes);
}

PlaneDesc gemm_tc_plan(int n_seg, int seg_cols, int K, bool whole_tiles, long long plane_stride, int seg0_cols, int row_tiles,
                       int planes)
{
    PlaneDesc pd{};
    if (seg0_cols <= 0) seg0_cols = seg_cols;
    const int tiles = (seg0_cols + BM - 1) / BM + (n_seg - 1) * ((seg_cols + BM - 1) / BM);
    const int KB = (K + BK - 1) / BK;
    const long long total = (long long)tiles * KB;
    int G = gemm_tc_num_ctas(row_tiles, planes);
    if (whole_tiles) {
        if (G > tiles) G = tiles;
        pd.n_max = 1; pd.KB = KB; pd.G = 0; pd.total = total; pd.stride = plane_stride; pd.ctas = G;
        return pd;
    }
    if ((long long)G > total) G = (int)total;
    int n_max = 1;
    for (int t = 0; t < tiles; ++t) {
        int n = gemm_tc_pieces(t, KB, G, total);
        if (n > n_max) n_max = n;
    }
    pd.n_max = n_max; pd.KB = KB; pd.G = G; pd.total = total; pd.stride = plane_stride; pd.ctas = G;
    return pd;
}

typedef void (*GemmKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, GemmTcArgs);
static GemmKernel gemm_kernel(int rt, int pl)
{
    if (pl == 2) return rt == 1 ? gemm_tc_kernel<1, 2> : gemm_tc_kernel<2, 2>;
    return rt == 1 ? gemm_tc_kernel<1, 1> : (rt == 2 ? gemm_tc_kernel<2, 1> : gemm_tc_kernel<4, 1>);
}
// the instantiation whose epilogue can store transposed: four token tiles, one plane
static GemmKernel gemm_kernel_transposing()
{
    return gemm_tc_kernel<4, 1, true>;
}

cudaError_t launch_gemm_tc(const TensorMap *mapX, const TensorMap *const *mapW, int n_seg, int seg_cols, int K,
                           const PlaneDesc &pd, float *P, int ldy, int T, int row0, int32_t *status, cudaStream_t s,
                           int seg0_cols, uint32_t spin_limit, int withhold, int x_row_hi, int x_row_lo, int row_tiles,
                           int planes, bool serialize, int out_t, long long ldt, bool packed)
{
    if (out_t && (pd.G != 0 || row_tiles < 4 || planes != 1))
        return cudaErrorInvalidValue;  // a transposed result needs whole tiles (one plane, every element written once);
                                       // only the four-tile single-plane kernel is built with that epilogue
    if (seg0_cols <= 0) seg0_cols = seg_cols;
    const int rt = row_tiles >= 4 && planes == 1 ? 4 : (row_tiles >= 2 ? 2 : 1), pl = planes == 1 ? 1 : 2;
    const int stages = cfg_stages(rt, pl);
    static bool attr_set[64] = {};
    if (first_use_on_current_device(attr_set)) {
        const int cfgs[5][2] = {{1, 2}, {2, 2}, {1, 1}, {2, 1}, {4, 1}};
        for (auto &cf : cfgs) {
            cudaError_t e = cudaFuncSetAttribute(gemm_kernel(cf[0], cf[1]), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 smem_bytes(cfg_stages(cf[0], cf[1]), cf[0], cf[1]));
            if (e != cudaSuccess)
                return e;
        }
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel_transposing(), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             smem_bytes(cfg_stages(4, 1), 4, 1));
        if (e != cudaSuccess)
            return e;
    }
    GemmTcArgs a;
    a.P = P;
    a.plane_stride = pd.stride;
    a.ldy = ldy;
    a.n_seg = n_seg;
    a.seg_tiles = (seg_cols + BM - 1) / BM;
    a.seg_cols = seg_cols;
    a.seg0_tiles = (seg0_cols + BM - 1) / BM;
    a.seg0_cols = seg0_cols;
    a.KB = pd.KB;
    a.G = pd.ctas;
    a.whole_tiles = pd.G == 0 ? 1 : 0;
    a.T = T;
    a.row0 = row0;
    a.status = status;
    a.stages = stages;
    a.spin_limit = spin_limit ? spin_limit : DEFAULT_SPIN_LIMIT;
    a.withhold = withhold;
    a.x_row_hi = x_row_hi;
    a.x_row_lo = x_row_lo;
    a.out_t = out_t;
    a.ldt = ldt;
    a.packed = packed ? 1 : 0;
    const CUtensorMap *w0 = (const CUtensorMap *)mapW[0];
    const CUtensorMap *w1 = (const CUtensorMap *)mapW[n_seg > 1 ? 1 : 0];
    const CUtensorMap *w2 = (const CUtensorMap *)mapW[n_seg > 2 ? 2 : 0];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pd.ctas);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem_bytes(stages, rt, pl);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = serialize || tuning_env("MEDUSA_NO_PDL") ? 0 : 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, out_t ? gemm_kernel_transposing() : gemm_kernel(rt, pl), *(const CUtensorMap *)mapX, *w0, *w1, *w2, a);
}

}  // namespace medusa

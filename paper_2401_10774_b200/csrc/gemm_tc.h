// Interface of the tcgen05 tensor-core GEMM (gemm_tc.cu) used by the bf16 model, and the description of the
// partial planes a projection leaves behind for the kernel that consumes it.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace medusa {

// opaque 128-byte TMA descriptor (same size and alignment as the driver's CUtensorMap)
struct alignas(64) TensorMap {
    uint64_t opaque[16];
};

// A projection result is the sum of 1..n_max float planes P[p][t][col], `stride` elements apart.
// G == 0: every column has exactly n_max planes.  G > 0 (stream-K): the 128-column tile holding `col` has
// gemm_tc_pieces(tile, KB, G, total) planes; higher planes hold stale data and must not be read.
struct PlaneDesc {
    int n_max;        // 0 = nothing to add
    int KB, G;        // k blocks per tile; number of CTAs the flat (tile, k block) sequence was cut into
    long long total;  // tiles * KB
    long long stride;
    int ctas;         // grid size of the launch
};

// index of the CTA whose range [c*total/G, (c+1)*total/G) contains flat k-block index x
__host__ __device__ inline int gemm_tc_first_cta(long long x, int G, long long total)
{
    const long long num = (x + 1) * G - 1;
    if (num < 0x7fffffffLL)  // every shape in use: plain 32-bit division
        return (int)((unsigned)num / (unsigned)total);
    return (int)(num / total);
}
__host__ __device__ inline int gemm_tc_pieces(int tile, int KB, int G, long long total)
{
    return gemm_tc_first_cta((long long)(tile + 1) * KB - 1, G, total) - gemm_tc_first_cta((long long)tile * KB, G, total) + 1;
}
// planes to add for column `col` of a projection output
__host__ __device__ inline int planes_of_col(const PlaneDesc &pd, int col)
{
    return pd.G == 0 ? pd.n_max : gemm_tc_pieces(col >> 7, pd.KB, pd.G, pd.total);
}

struct GemmTcArgs {
    float *P;                // partial planes: P[piece][t][first column of the segment + n]
    long long plane_stride;  // elements between planes
    int ldy;                 // row stride of a plane
    int n_seg, seg_tiles, seg_cols;  // weight segments, 128-row tiles per segment, rows per segment
    int seg0_tiles, seg0_cols;       // the same for segment 0, which may be wider than the others
    int KB, G;               // 64-wide k blocks per tile, CTAs
    int whole_tiles;         // 1: CTA c owns tiles c, c+G, ... completely (one plane)
    int T, row0;             // token rows [row0, T) are stored
    int32_t *status;         // device status word (set to MEDUSA_ERR_TIMEOUT if a bounded wait expires)
    int stages;              // depth of the TMA ring
    uint32_t spin_limit;     // polls before a bounded wait gives up
    int withhold;            // test hook: CTA 0's producer issues no load at all, so its consumers' waits expire
    int x_row_hi, x_row_lo;  // rows of the activation tensor where this launch's 64 token rows start in the hi / lo plane
    int packed;              // 1: the weight maps describe packed matrices (make_packed_weight_map)
    int out_t;               // 0: P[t][n];  1: P[n * ldt + t] = result (transposed store);  2: P[n * ldt + t] += result
    long long ldt;           // row stride of the transposed output (whole-tile launches only)
};

// W: [N][K] bf16 row-major
bool make_weight_map(TensorMap *out, const void *W, int N, int K);
// Packed weights: the matrix re-laid tile by tile, [ceil(N/128)][ceil(K/64)][128 rows][64 k], zero-padded, so that the
// 16 KiB a CTA requests per k block are consecutive bytes (a row-major matrix hands out 128 separate 128-byte pieces
// K * 2 bytes apart, which the memory system serves less efficiently).  launch_pack_weight writes that layout,
// make_packed_weight_map describes it, launch_gemm_tc(..., packed = true) addresses it.
size_t packed_weight_elems(int N, int K);
void launch_pack_weight(const void *W, int N, int K, void *Wp, cudaStream_t s);
bool make_packed_weight_map(TensorMap *out, const void *Wp, int N, int K);
// X_planes: split activation, [2][rows][K] bf16 (hi plane, then lo plane; rows a multiple of 64)
bool make_act_map(TensorMap *out, const void *X_planes, int K, int rows = 64);
int gemm_tc_num_ctas(int row_tiles = 1, int planes = 2);
// token tiles (64 rows each) one launch covers for a pass over T rows: 1 up to 64 rows, 2 beyond; 4 beyond 128 rows when
// the activations come as a single plane (the accumulators of four tiles then fit the tensor memory)
int gemm_tc_row_tiles(int T, int planes = 2);
int gemm_tc_stages();
int gemm_tc_ctas_per_sm();
// plan of a launch over n_seg weight matrices of seg_cols rows (seg_cols % 128 == 0 unless n_seg == 1); the first
// matrix has seg0_cols rows if that is given (> 0, a multiple of 128)
PlaneDesc gemm_tc_plan(int n_seg, int seg_cols, int K, bool whole_tiles, long long plane_stride, int seg0_cols = 0,
                       int row_tiles = 1, int planes = 2);
// P[piece][t][first column of segment seg + n] = partial sums over k of (X_hi + X_lo)[t][k] * W_seg[n][k], t in [row0, T);
// the launch's token rows t = 0.. are rows x_row_hi + t and x_row_lo + t of the activation tensor: 64 rows per launch
// with row_tiles = 1, 128 with row_tiles = 2, 256 with row_tiles = 4 (single plane only; pd must come from
// gemm_tc_plan with the same row_tiles and planes); planes = 1: only the hi plane is read (P = X_hi * W); a tree of more
// rows than one launch covers is projected launch by launch with P advanced accordingly
cudaError_t launch_gemm_tc(const TensorMap *mapX, const TensorMap *const *mapW, int n_seg, int seg_cols, int K,
                           const PlaneDesc &pd, float *P, int ldy, int T, int row0, int32_t *status, cudaStream_t s,
                           int seg0_cols = 0, uint32_t spin_limit = 0, int withhold = 0, int x_row_hi = 0, int x_row_lo = 64,
                           int row_tiles = 1, int planes = 2, bool serialize = false, int out_t = 0, long long ldt = 0,
                           bool packed = false);
// serialize: launch without programmatic dependent launch.  The kernel requests its streamed ("weight") operand BEFORE it
// waits for the preceding kernel, which is right for constant weights; a launch whose streamed operand was written by
// the preceding kernel (the gradient projections of the heads' training) must be fully serialised behind it.
// out_t = 1 / 2 (plans with whole tiles only): the result is stored / accumulated transposed, P[n * ldt + t] with n the
// streamed operand's row and t the token row counted from the launch's first one (P points at that column); every thread
// of the epilogue then owns 32 consecutive floats of a row.

}  // namespace medusa

// Internal declarations shared by the translation units of libbcq: descriptor checks, the
// index arithmetic of the two memory layouts, and the kernel launchers.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bcq.h"

namespace bcq {

constexpr int kWindow = 512;        // weights along K covered by one lookup-table build
constexpr int kUnitRows = 8;        // rows of one row unit
constexpr int kGroupsPerWindow = 4; // 128-weight groups in a window
constexpr int kLutConsumersMax = 23; // consumer warps per block of the lookup-table kernel (some instantiations have fewer)
constexpr int kLutUnitsPerWarp = 8;  // row units a consumer warp keeps accumulators for
constexpr int kMaxWindowsPerBlock = 32; // windows one block may walk (bounds the planner's search)
constexpr int kMmaWarps = 22;        // consumer warps per block of the small-batch kernel
constexpr int kMmaPairsPerWarp = 4;  // pairs of row units a warp keeps accumulators for
constexpr int kMmaMaxUnitsPerBlock = 2 * kMmaWarps * kMmaPairsPerWarp;
constexpr int kMaxRowBlocks = 4096; // small-batch kernel: arrival counters at the head of its workspace
constexpr size_t kCounterBytes = size_t(kMaxRowBlocks) * sizeof(int);   // small-batch kernel: one counter per row block

// The lookup-table kernel's split-K workspace: one 64-bit word per row and column (sum and arrival count in
// one word, see bcq_lut_kernel.cuh); all zero between launches.
inline size_t lut_workspace_bytes(int N, int cols) { return size_t(cols) * size_t(N) * sizeof(unsigned long long); }
// consumer warps and tiles per copy of the instantiation for (q, scales per group?, columns per launch)
// (sub: scaling units per 128 weights -- 0 = one scale per row, 1, 2 or 4 = groups of 128, 64 or 32)
int lut_consumer_warps(int q, int sub, int cols);
int lut_tiles_per_job(int q, int sub, int cols);
inline int scale_subs(int group) { return group == 0 ? 0 : 128 / group; }

inline int n_groups(const bcq_desc &d) { return d.group == 0 ? 1 : d.K / d.group; }

// ---- where the operands of one layer live (host and device) ---------------------------------
//
// Canonical: packed[i][n][k/8], alpha[i][n][g], z[n][g] in three arrays.
// Tiled: tile (w, u) of `packed` covers window w (512 weights = 64 chunks of 8 = 4 segments of 128)
// of row unit u (8 rows).  Lane l = 8 g + j of a warp owns row 8u + j and segment g of the window:
//   q*512 bytes of planes as [i < q][lane < 32][s < 16].  With groups of 128 (or one scale per row) byte s of a
//   lane in plane i is plane i of chunk 16 g + ((s + 2 j) mod 16): the 8 lanes of a segment walk its 16 chunks
//   skewed by two chunks per row, so that at every step the 32 lanes of a warp look up 32 different chunk
//   columns of the table (32 different shared-memory banks).  With SUB = 2 or 4 scaling units per segment
//   (groups of 64 or 32) a lane walks its segment unit by unit -- steps ph*(16/SUB) .. cover unit
//   (ph + j / (8/SUB)) mod SUB, inside it the chunk pairs rotate by j -- which keeps the 32 columns distinct
//   and a unit's chunks in consecutive steps (tile_step / tile_chunk below are the two directions);
//   grouped scales: followed, in the same tile, by the lanes' scales [lane < 32][ph < SUB][alpha_0 ..
//   alpha_{q-1}, z] (fp16), ph-th entry = the unit the lane walks in phase ph -- the tile is one contiguous
//   piece of memory, fetched by one bulk copy;
//   group 0 (per row): alpha [u][i][r] and z [u][r] stay in their own arrays.
// chunk (0..15 inside the segment) that byte s of lane row j covers, and the inverse
__host__ __device__ inline int tile_chunk(int sub, int j, int s)
{
    if (sub <= 1) return (s + 2 * j) & 15;
    const int cps = 16 / sub, wps = 8 / sub;
    const int ph = s / cps, t = s % cps;
    const int sg = (ph + j / wps) % sub;
    return 2 * (wps * sg + ((t >> 1) + j) % wps) + (t & 1);
}
__host__ __device__ inline int tile_step(int sub, int j, int cc)
{
    if (sub <= 1) return (cc - 2 * j) & 15;
    const int cps = 16 / sub, wps = 8 / sub;
    const int col = cc >> 1, sg = col / wps, cw = col % wps;
    const int ph = (sg - j / wps + sub) % sub, th = (cw - j % wps + wps) % wps;
    return ph * cps + 2 * th + (cc & 1);
}
// phase in which lane row j walks scaling unit sg of its segment
__host__ __device__ inline int tile_phase(int sub, int j, int sg)
{
    if (sub <= 1) return 0;
    return (sg - j / (8 / sub) + sub) % sub;
}
struct View {
    int layout, N, K, q, group;
    unsigned char *packed;
    uint16_t *alpha;
    uint16_t *z;

    __host__ __device__ int G() const { return group == 0 ? 1 : K / group; }
    __host__ __device__ bool interleaved() const { return layout == BCQ_LAYOUT_TILED && group != 0; }
    __host__ __device__ int subs() const { return group == 0 ? 0 : 128 / group; }   // scaling units per segment (tiled: group 32, 64, 128)
    __host__ __device__ size_t tile_bytes() const { return size_t(q) * 512 + (interleaved() ? size_t(subs()) * (q + 1) * 64 : 0); }
    __host__ __device__ size_t tile_base(int w, int u) const { return (size_t(w) * (N / kUnitRows) + u) * tile_bytes(); }

    // the byte holding weights k = 8*kb .. 8*kb+7 of (plane i, row n)
    __host__ __device__ unsigned char *plane_byte(int i, int n, int kb) const
    {
        if (layout == BCQ_LAYOUT_CANONICAL) return packed + (size_t(i) * N + n) * size_t(K / 8) + kb;
        const int w = kb / (kWindow / 8), c = kb % (kWindow / 8);
        const int g = c >> 4, u = n / kUnitRows, j = n % kUnitRows;
        const int s = tile_step(subs(), j, c & 15);   // step at which lane 8g + j reaches chunk c
        const int lane = 8 * g + j;
        return packed + tile_base(w, u) + size_t(i) * 512 + size_t(lane) * 16 + s;
    }
    // distance in bytes from plane_byte(i, n, kb) to plane_byte(i + 1, n, kb)
    __host__ __device__ size_t plane_stride() const
    {
        return layout == BCQ_LAYOUT_CANONICAL ? size_t(N) * size_t(K / 8) : size_t(512);
    }
    __host__ __device__ uint16_t *alpha_elem(int i, int n, int g) const
    {
        if (layout == BCQ_LAYOUT_CANONICAL) return alpha + (size_t(i) * N + n) * G() + g;
        const int u = n / kUnitRows, r = n % kUnitRows;
        if (group == 0) return alpha + (size_t(u) * q + i) * kUnitRows + r;
        const int sub = subs(), per_window = kGroupsPerWindow * sub;
        const int w = g / per_window, gi = (g % per_window) / sub, ph = tile_phase(sub, r, g % sub);
        return reinterpret_cast<uint16_t *>(packed + tile_base(w, u) + size_t(q) * 512) + ((gi * kUnitRows + r) * sub + ph) * (q + 1) + i;
    }
    __host__ __device__ uint16_t *z_elem(int n, int g) const
    {
        if (layout == BCQ_LAYOUT_CANONICAL) return z + size_t(n) * G() + g;
        const int u = n / kUnitRows, r = n % kUnitRows;
        if (group == 0) return z + size_t(u) * kUnitRows + r;
        const int sub = subs(), per_window = kGroupsPerWindow * sub;
        const int w = g / per_window, gi = (g % per_window) / sub, ph = tile_phase(sub, r, g % sub);
        return reinterpret_cast<uint16_t *>(packed + tile_base(w, u) + size_t(q) * 512) + ((gi * kUnitRows + r) * sub + ph) * (q + 1) + q;
    }
};

inline View make_view(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z)
{
    View v;
    v.layout = d.layout, v.N = d.N, v.K = d.K, v.q = d.q, v.group = d.group;
    v.packed = static_cast<unsigned char *>(const_cast<void *>(packed));
    v.alpha = const_cast<uint16_t *>(alpha);
    v.z = const_cast<uint16_t *>(z);
    return v;
}

// ---- launchers (each returns the cudaError_t of its launch) ------------------------------

cudaError_t launch_merge(const bcq_desc &d, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias,
                         int n_bits, const uint8_t *code_of_int /*[256]*/, const double *plane_weight /*[q]*/,
                         uint8_t *codes, uint16_t *alpha, uint16_t *z, cudaStream_t st);
cudaError_t launch_quantize_rtn(const uint16_t *W, int n_bits, double s_factor, const uint8_t *code_of_int /*[256]*/,
                                const double *plane_weight /*[q]*/, uint16_t *S, uint16_t *qbias, uint8_t *w_int,
                                const View &dst, cudaStream_t st, bool pack = true);   // pack = false: S, qbias, w_int only
cudaError_t launch_pack(const uint8_t *codes, const View &dst, cudaStream_t st);
cudaError_t launch_permute_planes(const View &src, const View &dst, cudaStream_t st);
cudaError_t launch_permute_scales(const View &src, const View &dst, cudaStream_t st);

cudaError_t launch_generic(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                           const uint16_t *X, uint16_t *Y, int B, cudaStream_t st);
cudaError_t launch_lut_gemv(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *x, uint16_t *y, void *workspace, cudaStream_t st,
                            int cols = 1, const bcq_epilogue *epilogue = nullptr, bool bf16 = false);
// Several operands that share x, K, q and the scaling unit, one launch: d.N = all their rows, the operands' row
// blocks add up to plan.row_blocks.
constexpr int kLutMaxOperands = 4;
struct LutOperand {
    const void *packed;
    const uint16_t *alpha, *z;
    uint16_t *y;
    int N, row_blocks;
};
cudaError_t launch_lut_multi(const bcq_desc &d, const bcq_plan &plan, const LutOperand *ops, int count, const uint16_t *x,
                             void *workspace, cudaStream_t st);

// the ablation without lookup tables (tiled layout): every weight dequantised to fp16 and multiplied
cudaError_t launch_dequant_gemv(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                                const uint16_t *x, uint16_t *y, cudaStream_t st);

cudaError_t launch_mma_gemm(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *X, uint16_t *Y, int B, void *workspace, cudaStream_t st);

int record_cuda_error(cudaError_t e);   // text for bcq_last_cuda_error(); returns BCQ_ERR_CUDA

// The search of section "Quantize Weight Twice" / "Re-explore Scale Factor": output errors of P candidates for
// `scales` scale factors in one launch (step 1's outputs of the factors side by side: w_int [scales][N][K], S and
// qbias `scale_stride` elements apart; err_rows [scales][P][N] per row, err [scales][P] summed in a fixed order),
// and the first minimum of `count` errors laid out [.][P].
cudaError_t launch_search_errors(const uint16_t *W, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias, size_t scale_stride,
                                 const uint16_t *X, int N, int K, int group, int T, int n_bits, const float *lut_dev /*[P][64]*/, int P,
                                 int scales, float *err_rows, double *err, cudaStream_t st);
cudaError_t launch_search_argmin(const double *err, int count, int P, int *best, cudaStream_t st);
cudaError_t search_status_take(int *status);

cudaError_t lut_status_take(int *status);
cudaError_t mma_status_take(int *status);

}  // namespace bcq

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
constexpr int kLutWarps = 16;       // warps per block of the lookup-table kernel
constexpr int kLutUnitsPerWarp = 4; // row units a warp keeps accumulators for
constexpr int kMaxUnitsPerBlock = kLutWarps * kLutUnitsPerWarp;
constexpr int kMaxWindowsPerBlock = 14; // windows of x a block keeps in shared memory
constexpr int kMaxRowBlocks = 4096; // arrival counters at the head of the workspace
constexpr size_t kCounterBytes = size_t(kMaxRowBlocks) * sizeof(int);

inline int n_groups(const bcq_desc &d) { return d.group == 0 ? 1 : d.K / d.group; }

// ---- layout index arithmetic (host and device) ------------------------------------------

// Byte offset of the byte holding weights k = 8*kb .. 8*kb+7 of (plane i, row n).
__host__ __device__ inline size_t plane_byte_offset(int layout, int N, int K, int q, int i, int n, int kb)
{
    if (layout == BCQ_LAYOUT_CANONICAL) return (size_t(i) * N + n) * size_t(K / 8) + kb;
    const int U = N / kUnitRows;
    const int w = kb / (kWindow / 8), c = kb % (kWindow / 8);
    const int lane = c >> 1, s = c & 1;
    const int u = n / kUnitRows, r = n % kUnitRows;
    const int p = (r * q + i) * 2 + s;
    return ((size_t(w) * U + u) * q + (p >> 4)) * 512 + size_t(lane) * 16 + (p & 15);
}

// Element offset of alpha[i][n][g].
__host__ __device__ inline size_t alpha_elem_offset(int layout, int N, int G, int q, int group, int i, int n, int g)
{
    if (layout == BCQ_LAYOUT_CANONICAL) return (size_t(i) * N + n) * G + g;
    const int U = N / kUnitRows;
    const int u = n / kUnitRows, r = n % kUnitRows;
    if (group == 0) return (size_t(u) * q + i) * kUnitRows + r;
    const int w = g / kGroupsPerWindow, gi = g % kGroupsPerWindow;
    return (((size_t(w) * U + u) * kGroupsPerWindow + gi) * q + i) * kUnitRows + r;
}

// Element offset of z[n][g].
__host__ __device__ inline size_t offset_elem_offset(int layout, int N, int G, int group, int n, int g)
{
    if (layout == BCQ_LAYOUT_CANONICAL) return size_t(n) * G + g;
    const int U = N / kUnitRows;
    const int u = n / kUnitRows, r = n % kUnitRows;
    if (group == 0) return size_t(u) * kUnitRows + r;
    const int w = g / kGroupsPerWindow, gi = g % kGroupsPerWindow;
    return ((size_t(w) * U + u) * kGroupsPerWindow + gi) * kUnitRows + r;
}

// ---- launchers (each returns the cudaError_t of its launch) ------------------------------

cudaError_t launch_merge(const bcq_desc &d, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias,
                         int n_bits, const uint8_t *code_of_int /*[256]*/, const double *plane_weight /*[q]*/,
                         uint8_t *codes, uint16_t *alpha, uint16_t *z, cudaStream_t st);
cudaError_t launch_pack(const bcq_desc &d, const uint8_t *codes, void *packed, cudaStream_t st);
cudaError_t launch_permute_planes(const bcq_desc &src, const void *in, const bcq_desc &dst, void *out, cudaStream_t st);
cudaError_t launch_permute_scales(const bcq_desc &src, const uint16_t *alpha_in, const uint16_t *z_in,
                                  const bcq_desc &dst, uint16_t *alpha_out, uint16_t *z_out, cudaStream_t st);

cudaError_t launch_generic(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                           const uint16_t *X, uint16_t *Y, int B, cudaStream_t st);
cudaError_t launch_lut_gemv(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *x, uint16_t *y, void *workspace, cudaStream_t st);

cudaError_t lut_status_take(int *status);

}  // namespace bcq

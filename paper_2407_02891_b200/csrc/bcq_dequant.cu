// Ablation: the same product without lookup tables.  Every weight is dequantised to fp16,
//     w = sum_i alpha_i b_i + z                                   (Eq. bcw dequantisation + Eq. fuse_step3),
// and multiplied with its activation, as a kernel for linearly quantised weights would do it; the packed
// operand, its tiled layout and the bytes read are those of the lookup-table kernel.  It exists to show on
// this GPU the shape of the paper's speed claim for binary-coded weights (Tab. "The speed up of GPTQT"):
// the time of this kernel against bcq_gemv on equal operands.
//
// One block of 8 warps per row unit; warp w takes the windows w, w + 8, ...; lane 8 g + j owns row j and the
// g-th group of 128 weights of a window, as in the tile layout.  Per pair of weights: q sign flips of
// (alpha_i, alpha_i) and q + 1 half2 additions give the two fp16 weights, two fp32 multiply-adds use them.
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kDequantWarps = 8;

template <int Q, bool GROUPED>
__global__ void __launch_bounds__(32 * kDequantWarps) dequant_gemv_kernel(const unsigned char *__restrict__ tiles,
                                                                          const __half *__restrict__ alpha,
                                                                          const __half *__restrict__ zoff,
                                                                          const __half *__restrict__ x, __half *__restrict__ y,
                                                                          int N, int K)
{
    __shared__ float part[kDequantWarps][kUnitRows];
    constexpr int kTile = Q * 512 + (GROUPED ? Q * 64 + 64 : 0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g4 = lane >> 3, jr = lane & 7;
    const int U = N / kUnitRows, W = K / kWindow, u = blockIdx.x;
    float acc = 0.f;
    uint32_t neg[Q];     // (-alpha_i, -alpha_i) as two fp16
    uint32_t zz = 0u;    // (z, z)
    if constexpr (!GROUPED) {
#pragma unroll
        for (int i = 0; i < Q; ++i) {
            const uint32_t a = __half_as_ushort(alpha[(size_t(u) * Q + i) * kUnitRows + jr]) ^ 0x8000u;
            neg[i] = a | (a << 16);
        }
        const uint32_t zb = __half_as_ushort(zoff[size_t(u) * kUnitRows + jr]);
        zz = zb | (zb << 16);
    }
    for (int w = warp; w < W; w += kDequantWarps) {
        const unsigned char *tile = tiles + (size_t(w) * U + u) * kTile;
        uint32_t wbuf[4 * Q];
#pragma unroll
        for (int i = 0; i < Q; ++i) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(tile + i * 512 + lane * 16));
            wbuf[4 * i + 0] = v.x, wbuf[4 * i + 1] = v.y, wbuf[4 * i + 2] = v.z, wbuf[4 * i + 3] = v.w;
        }
        if constexpr (GROUPED) {
            const uint16_t *sp = reinterpret_cast<const uint16_t *>(tile + Q * 512 + lane * (2 * (Q + 1)));
#pragma unroll
            for (int i = 0; i < Q; ++i) {
                const uint32_t a = uint32_t(__ldg(sp + i)) ^ 0x8000u;
                neg[i] = a | (a << 16);
            }
            const uint32_t zb = __ldg(sp + Q);
            zz = zb | (zb << 16);
        }
        const __half *xw = x + size_t(w) * kWindow + 128 * g4;
#pragma unroll
        for (int s = 0; s < 16; ++s) {
            const int c = (s + 2 * jr) & 15;   // the chunk this lane's byte s covers (see the tile layout)
            const uint4 xr = __ldg(reinterpret_cast<const uint4 *>(xw + 8 * c));
            const uint32_t x2[4] = {xr.x, xr.y, xr.z, xr.w};
            uint32_t b[Q];
#pragma unroll
            for (int i = 0; i < Q; ++i) b[i] = (wbuf[4 * i + (s >> 2)] >> (8 * (s & 3))) & 0xffu;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                __half2 w2 = *reinterpret_cast<const __half2 *>(&zz);
#pragma unroll
                for (int i = 0; i < Q; ++i) {
                    // weight bit 1 = +alpha: flip the sign of -alpha
                    const uint32_t flip = ((b[i] << (15 - 2 * p)) & 0x8000u) | ((b[i] << (30 - 2 * p)) & 0x80000000u);
                    const uint32_t term = neg[i] ^ flip;
                    w2 = __hadd2(w2, *reinterpret_cast<const __half2 *>(&term));
                }
                const float2 wf = __half22float2(w2);
                const float2 xf = __half22float2(*reinterpret_cast<const __half2 *>(&x2[p]));
                acc = fmaf(wf.x, xf.x, acc);
                acc = fmaf(wf.y, xf.y, acc);
            }
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 8);
    acc += __shfl_xor_sync(0xffffffffu, acc, 16);
    if (lane < kUnitRows) part[warp][lane] = acc;
    __syncthreads();
    if (threadIdx.x < kUnitRows) {
        float v = 0.f;
#pragma unroll
        for (int k = 0; k < kDequantWarps; ++k) v += part[k][threadIdx.x];
        y[size_t(u) * kUnitRows + threadIdx.x] = __float2half_rn(v);
    }
}

template <int Q>
static cudaError_t launch_dequant_q(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                                    const uint16_t *x, uint16_t *y, cudaStream_t st)
{
    const dim3 grid(unsigned(d.N / kUnitRows)), block(32 * kDequantWarps);
    auto t = static_cast<const unsigned char *>(packed);
    auto a = reinterpret_cast<const __half *>(alpha), zz = reinterpret_cast<const __half *>(z);
    auto xx = reinterpret_cast<const __half *>(x);
    auto yy = reinterpret_cast<__half *>(y);
    if (d.group != 0)
        dequant_gemv_kernel<Q, true><<<grid, block, 0, st>>>(t, a, zz, xx, yy, d.N, d.K);
    else
        dequant_gemv_kernel<Q, false><<<grid, block, 0, st>>>(t, a, zz, xx, yy, d.N, d.K);
    return cudaGetLastError();
}

cudaError_t launch_dequant_gemv(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                                const uint16_t *x, uint16_t *y, cudaStream_t st)
{
    switch (d.q) {
        case 1: return launch_dequant_q<1>(d, packed, alpha, z, x, y, st);
        case 2: return launch_dequant_q<2>(d, packed, alpha, z, x, y, st);
        case 3: return launch_dequant_q<3>(d, packed, alpha, z, x, y, st);
        case 4: return launch_dequant_q<4>(d, packed, alpha, z, x, y, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace bcq

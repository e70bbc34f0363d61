// The BCQ product  y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )  (Eq. bcw + Eq. fuse_step3),
// generic form: one warp per output row, direct sign arithmetic, any valid shape, either layout,
// batch 1..16.  The slow, always-available path; the batch-1 hot path is in bcq_lut.cu.
#include "bcq_internal.cuh"

namespace bcq {

// =============================================================================================
// generic kernel
// =============================================================================================

template <int BMAX>
__global__ void __launch_bounds__(256) generic_kernel(const uint8_t *__restrict__ packed,
                                                       const __half *__restrict__ alpha,
                                                       const __half *__restrict__ z, const __half *__restrict__ X,
                                                       __half *__restrict__ Y, int N, int K, int q, int group,
                                                       int layout, int B)
{
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const int G = group == 0 ? 1 : K / group;
    const int L = group == 0 ? K : group;
    float acc[BMAX];
#pragma unroll
    for (int b = 0; b < BMAX; ++b) acc[b] = 0.f;

    for (int kb = lane; kb < K / 8; kb += 32) {
        const int g = (kb * 8) / L;
        const float zz = __half2float(z[offset_elem_offset(layout, N, G, group, n, g)]);
        float a[4];
        uint32_t bits[4];
        for (int i = 0; i < q; ++i) {
            a[i] = __half2float(alpha[alpha_elem_offset(layout, N, G, q, group, i, n, g)]);
            bits[i] = packed[plane_byte_offset(layout, N, K, q, i, n, kb)];
        }
#pragma unroll
        for (int b = 0; b < BMAX; ++b) {
            if (b < B) {
                float xs[8], sum_x = 0.f;
                for (int j = 0; j < 8; ++j) {
                    xs[j] = __half2float(X[size_t(b) * K + size_t(kb) * 8 + j]);
                    sum_x += xs[j];
                }
                float part = zz * sum_x;
                for (int i = 0; i < q; ++i) {
                    float s = 0.f;
                    for (int j = 0; j < 8; ++j) s += ((bits[i] >> j) & 1u) ? xs[j] : -xs[j];
                    part = fmaf(a[i], s, part);
                }
                acc[b] += part;
            }
        }
    }
#pragma unroll
    for (int b = 0; b < BMAX; ++b) {
        float v = acc[b];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && b < B) Y[size_t(b) * N + n] = __float2half_rn(v);
    }
}

cudaError_t launch_generic(const bcq_desc &d, const void *packed, const uint16_t *alpha, const uint16_t *z,
                           const uint16_t *X, uint16_t *Y, int B, cudaStream_t st)
{
    const int warps = 8;
    dim3 grid((d.N + warps - 1) / warps), block(32 * warps);
    auto p = static_cast<const uint8_t *>(packed);
    auto a = reinterpret_cast<const __half *>(alpha);
    auto zz = reinterpret_cast<const __half *>(z);
    auto x = reinterpret_cast<const __half *>(X);
    auto y = reinterpret_cast<__half *>(Y);
    if (B == 1)
        generic_kernel<1><<<grid, block, 0, st>>>(p, a, zz, x, y, d.N, d.K, d.q, d.group, d.layout, B);
    else if (B <= 4)
        generic_kernel<4><<<grid, block, 0, st>>>(p, a, zz, x, y, d.N, d.K, d.q, d.group, d.layout, B);
    else
        generic_kernel<16><<<grid, block, 0, st>>>(p, a, zz, x, y, d.N, d.K, d.q, d.group, d.layout, B);
    return cudaGetLastError();
}

}  // namespace bcq

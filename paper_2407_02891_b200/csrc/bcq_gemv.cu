// The BCQ product  y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )  (Eq. bcw + Eq. fuse_step3),
// generic form: one warp per output row, direct sign arithmetic, any valid shape, either layout,
// batch 1..16.  The slow, always-available path; the batch-1 hot path is in bcq_lut.cu.
#include "bcq_internal.cuh"

namespace bcq {

// =============================================================================================
// generic kernel
// =============================================================================================

template <int BMAX>
__global__ void __launch_bounds__(256) generic_kernel(const View v, const __half *__restrict__ X, __half *__restrict__ Y, int B)
{
    const int N = v.N, K = v.K, q = v.q, group = v.group;
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const int L = group == 0 ? K : group;
    float acc[BMAX];
#pragma unroll
    for (int b = 0; b < BMAX; ++b) acc[b] = 0.f;

    for (int kb = lane; kb < K / 8; kb += 32) {
        const int g = (kb * 8) / L;
        const float zz = __half2float(*reinterpret_cast<const __half *>(v.z_elem(n, g)));
        float a[4];
        uint32_t bits[4];
        for (int i = 0; i < q; ++i) {
            a[i] = __half2float(*reinterpret_cast<const __half *>(v.alpha_elem(i, n, g)));
            bits[i] = *v.plane_byte(i, n, kb);
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
    const View v = make_view(d, packed, alpha, z);
    auto x = reinterpret_cast<const __half *>(X);
    auto y = reinterpret_cast<__half *>(Y);
    if (B == 1)
        generic_kernel<1><<<grid, block, 0, st>>>(v, x, y, B);
    else if (B <= 4)
        generic_kernel<4><<<grid, block, 0, st>>>(v, x, y, B);
    else
        generic_kernel<16><<<grid, block, 0, st>>>(v, x, y, B);
    return cudaGetLastError();
}

}  // namespace bcq

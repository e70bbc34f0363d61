// Operand preparation kernels: linear-int -> merged binary code (Eq. round, Eq. fuse_step3),
// code -> bit-plane packing, and the canonical <-> tiled permutations.  All run once per
// layer, offline; they are written for clarity and coalesced access, not for peak speed.
#include "bcq_internal.cuh"

namespace bcq {

// ---- merge ---------------------------------------------------------------------------------

struct MergeTable {
    uint8_t code_of_int[256];  // code of the reachable integer nearest to each step-1 integer
    double plane_weight[4];    // m_j = sum of 2^(i-2) over the step-1 bits i of plane j
    double centre;             // (2^n - 1) / 2
};

__global__ void merge_codes_kernel(const uint8_t *__restrict__ w_int, uint8_t *__restrict__ codes, size_t count,
                                   MergeTable tab)
{
    __shared__ uint8_t lut[256];
    for (int t = threadIdx.x; t < 256; t += blockDim.x) lut[t] = tab.code_of_int[t];
    __syncthreads();
    size_t stride = size_t(gridDim.x) * blockDim.x;
    for (size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x; t < count; t += stride) codes[t] = lut[w_int[t]];
}

// alpha_j = S * m_j and z = S * centre + qbias, each evaluated exactly in fp64 (the products
// and the sum of two fp16-derived values fit 53 bits) and rounded once to fp16.
__global__ void merge_scales_kernel(const __half *__restrict__ S, const __half *__restrict__ qbias, int N, int G, int q,
                                    __half *__restrict__ alpha, __half *__restrict__ z, MergeTable tab)
{
    size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= size_t(N) * G) return;
    double s = double(__half2float(S[t]));
    double b = double(__half2float(qbias[t]));
    for (int j = 0; j < q; ++j) alpha[size_t(j) * N * G + t] = __double2half(s * tab.plane_weight[j]);
    z[t] = __double2half(s * tab.centre + b);
}

cudaError_t launch_merge(const bcq_desc &d, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias, int n_bits,
                         const uint8_t *code_of_int, const double *plane_weight, uint8_t *codes, uint16_t *alpha,
                         uint16_t *z, cudaStream_t st)
{
    MergeTable tab;
    for (int t = 0; t < 256; ++t) tab.code_of_int[t] = code_of_int[t];
    for (int j = 0; j < 4; ++j) tab.plane_weight[j] = j < d.q ? plane_weight[j] : 0.0;
    tab.centre = (double((1u << n_bits) - 1u)) / 2.0;
    size_t count = size_t(d.N) * d.K;
    int blocks = int((count + 1023) / 1024 < 65535 ? (count + 1023) / 1024 : 65535);
    merge_codes_kernel<<<blocks, 256, 0, st>>>(w_int, codes, count, tab);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    size_t units = size_t(d.N) * n_groups(d);
    merge_scales_kernel<<<unsigned((units + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const __half *>(S), reinterpret_cast<const __half *>(qbias), d.N, n_groups(d), d.q,
        reinterpret_cast<__half *>(alpha), reinterpret_cast<__half *>(z), tab);
    return cudaGetLastError();
}

// ---- pack: one thread per (row, 8-weight chunk) ---------------------------------------------

__global__ void pack_kernel(const uint8_t *__restrict__ codes, const View dst)
{
    const int kbytes = dst.K / 8;
    size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= size_t(dst.N) * kbytes) return;
    const int n = int(t / kbytes), kb = int(t % kbytes);
    const uint2 c8 = *reinterpret_cast<const uint2 *>(codes + size_t(n) * dst.K + size_t(kb) * 8);
    const uint32_t lo = c8.x, hi = c8.y;
    for (int i = 0; i < dst.q; ++i) {
        uint32_t byte = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            byte |= ((lo >> (8 * j + i)) & 1u) << j;
            byte |= ((hi >> (8 * j + i)) & 1u) << (4 + j);
        }
        *dst.plane_byte(i, n, kb) = uint8_t(byte);
    }
    // The products start fetching packed operands before they wait for the kernel in front of them: every
    // kernel that writes operands makes its writes visible device-wide before its blocks count as finished.
    __threadfence();
}

cudaError_t launch_pack(const uint8_t *codes, const View &dst, cudaStream_t st)
{
    size_t count = size_t(dst.N) * (dst.K / 8);
    pack_kernel<<<unsigned((count + 255) / 256), 256, 0, st>>>(codes, dst);
    return cudaGetLastError();
}

// ---- permutations between layouts -----------------------------------------------------------

__global__ void permute_planes_kernel(const View src, const View dst)
{
    const int kbytes = src.K / 8;
    size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= size_t(src.q) * src.N * kbytes) return;
    const int kb = int(t % kbytes);
    const int n = int((t / kbytes) % src.N);
    const int i = int(t / (size_t(kbytes) * src.N));
    *dst.plane_byte(i, n, kb) = *src.plane_byte(i, n, kb);
    __threadfence();   // see pack_kernel
}

__global__ void permute_scales_kernel(const View src, const View dst)
{
    const int G = src.G();
    size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= size_t(src.N) * G) return;
    const int n = int(t / G), g = int(t % G);
    for (int i = 0; i < src.q; ++i) *dst.alpha_elem(i, n, g) = *src.alpha_elem(i, n, g);
    *dst.z_elem(n, g) = *src.z_elem(n, g);
    __threadfence();   // see pack_kernel
}

cudaError_t launch_permute_planes(const View &src, const View &dst, cudaStream_t st)
{
    size_t count = size_t(src.q) * src.N * (src.K / 8);
    permute_planes_kernel<<<unsigned((count + 255) / 256), 256, 0, st>>>(src, dst);
    return cudaGetLastError();
}

cudaError_t launch_permute_scales(const View &src, const View &dst, cudaStream_t st)
{
    size_t count = size_t(src.N) * src.G();
    permute_scales_kernel<<<unsigned((count + 255) / 256), 256, 0, st>>>(src, dst);
    return cudaGetLastError();
}

}  // namespace bcq

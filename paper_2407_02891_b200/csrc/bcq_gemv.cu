// The BCQ products  y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )  (Eq. bcw + Eq. fuse_step3).
//
//  * generic_kernel: one warp per output row, direct sign arithmetic, any valid shape, either
//    layout, batch 1..16.  The slow, always-available path.
//  * lut_gemv_kernel: the batch-1 hot path for the tiled layout.  Per 512-wide window of K a
//    block builds, in shared memory, all 2^8 signed sums of every 8-activation chunk; packed
//    weight bytes streamed from HBM with 128-bit loads index those tables directly.
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

// =============================================================================================
// lookup-table GEMV (batch 1, tiled layout)
// =============================================================================================
//
// Block = 16 warps; it owns row units [u0,u1) (8 rows each, at most 64) and windows [w0,w1).
// Warp `wp` owns units u0 + wp + 16 t, t < 4, and keeps 8 fp32 accumulators per unit.
//
// Shared memory: two 64 KB tables (double buffered over windows) + per-warp staging of scales.
//   table word address of (entry e, chunk c) = e*64 + (c&1)*32 + (c>>1): lane l of a warp looks
//   up chunks 2l and 2l+1 only, so every lookup of a warp instruction hits 32 distinct banks
//   whatever the weight bytes are.  Entry stride 256 B lets one byte-permute form the address:
//   byte 1 <- weight byte, bytes 0,2,3 <- (table offset + 4*lane).
//
// Weight bytes go HBM -> registers (no shared-memory staging: the table lookups already use
// most of the shared-memory bandwidth); the next window's bytes for unit t are requested as
// soon as the current ones are consumed.  Scales (alpha, z: 1/8 of the bytes at q=3, g=128) go
// HBM -> shared memory with cp.async, because 8 lanes share each value.

constexpr int kLutThreads = kLutWarps * 32;
constexpr int kTableBytes = 256 * 64 * 4;  // 65536
template <int Q>
struct LutSmem {
    static constexpr int kScaleTile = (Q + 1) * 64;  // bytes of alpha+z of one (window, unit), group 128
    static constexpr int kStageBytes = kLutWarps * kLutUnitsPerWarp * kScaleTile;
    static constexpr int kTotal = 2 * kTableBytes + kStageBytes;
};

struct LutParams {
    const uint8_t *planes;
    const uint8_t *alpha;  // tiled
    const uint8_t *z;      // tiled
    const __half *x;
    __half *y;
    float *partial;  // [k_splits][N] when k_splits > 1
    int *counters;   // [row_blocks]
    int N, K, U, W;
    int row_blocks, k_splits;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint4 ldg_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Build the table of window `w` into `table` (a 64 KB region of shared memory).
// Thread t: quad = t & 15 (slot s = quad >> 3, lanes 4*(quad&7) .. +3), high entry bits = t >> 4.
// It walks the 8 entries that share those 5 high bits in Gray-code order: one FMA per entry.
__device__ __forceinline__ void build_table(unsigned char *table, const __half *__restrict__ xw, int tid)
{
    const int quad = tid & 15;
    const int s = quad >> 3, lq = quad & 7;
    const int hi = tid >> 4;  // entry bits 3..7
    float x[4][8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        // chunk c = 2*(4*lq + k) + s  ->  activations 8c .. 8c+7
        const uint4 raw = *reinterpret_cast<const uint4 *>(xw + 8 * (2 * (4 * lq + k) + s));
        const __half2 *h2 = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(h2[j]);
            x[k][2 * j] = f.x;
            x[k][2 * j + 1] = f.y;
        }
    }
    float cur[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float v = -x[k][0] - x[k][1] - x[k][2];
#pragma unroll
        for (int j = 3; j < 8; ++j) v += ((hi >> (j - 3)) & 1) ? x[k][j] : -x[k][j];
        cur[k] = v;
    }
    float4 *dst = reinterpret_cast<float4 *>(table + s * 128 + lq * 16);
    int lo = 0;  // Gray code of the step
#pragma unroll
    for (int step = 0; step < 8; ++step) {
        if (step > 0) {
            // bit that flips between Gray(step-1) and Gray(step): the lowest set bit of `step`
            const int bit = (step & 1) ? 0 : ((step & 2) ? 1 : 2);
            lo ^= 1 << bit;
            const float sgn = ((lo >> bit) & 1) ? 2.f : -2.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) cur[k] = fmaf(sgn, x[k][bit], cur[k]);
        }
        const int e = hi * 8 + lo;
        dst[e * 16] = make_float4(cur[0], cur[1], cur[2], cur[3]);  // entry stride 256 B = 16 float4
    }
}

template <int Q>
__global__ void __launch_bounds__(kLutThreads, 1) lut_gemv_kernel(const LutParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    using S = LutSmem<Q>;
    constexpr int UMAX = kLutUnitsPerWarp;
    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;

    const int rbi = blockIdx.x % p.row_blocks, ks = blockIdx.x / p.row_blocks;
    const int u0 = int((long long)rbi * p.U / p.row_blocks), u1 = int((long long)(rbi + 1) * p.U / p.row_blocks);
    const int w0 = int((long long)ks * p.W / p.k_splits), w1 = int((long long)(ks + 1) * p.W / p.k_splits);

    unsigned char *stage = smem + 2 * kTableBytes + wp * (UMAX * S::kScaleTile);
    const uint32_t stage_u32 = smem_u32(stage);

    uint32_t wbuf[UMAX][4 * Q];
    float acc[UMAX][8];
#pragma unroll
    for (int t = 0; t < UMAX; ++t)
#pragma unroll
        for (int r = 0; r < 8; ++r) acc[t][r] = 0.f;

    // requests for (window w, unit slot t): weight bytes to registers, scales to staging
    auto request = [&](int w, int t) {
        const int u = u0 + wp + kLutWarps * t;
        if (w < w1 && u < u1) {
            const size_t tile = size_t(w) * p.U + u;
            const uint8_t *src = p.planes + tile * (Q * 512) + lane * 16;
#pragma unroll
            for (int j = 0; j < Q; ++j) {
                const uint4 v = ldg_stream(src + j * 512);
                wbuf[t][4 * j + 0] = v.x;
                wbuf[t][4 * j + 1] = v.y;
                wbuf[t][4 * j + 2] = v.z;
                wbuf[t][4 * j + 3] = v.w;
            }
            if (lane < 4 * Q)
                cp_async_16(stage_u32 + t * S::kScaleTile + lane * 16, p.alpha + tile * (Q * 64) + lane * 16);
            else if (lane < 4 * Q + 4)
                cp_async_16(stage_u32 + t * S::kScaleTile + lane * 16, p.z + tile * 64 + (lane - 4 * Q) * 16);
        }
        cp_async_commit();
    };

#pragma unroll
    for (int t = 0; t < UMAX; ++t) request(w0, t);

    build_table(smem, p.x + size_t(w0) * kWindow, tid);
    __syncthreads();

    for (int w = w0; w < w1; ++w) {
        const int cur = (w - w0) & 1;
        if (w + 1 < w1) build_table(smem + (cur ^ 1) * kTableBytes, p.x + size_t(w + 1) * kWindow, tid);

        const unsigned char *table = smem + cur * kTableBytes;
        const uint32_t lane_off = uint32_t(cur * kTableBytes + lane * 4);
        // sum of this lane's 16 activations: the all-ones entries of its two chunks
        const float xsum = *reinterpret_cast<const float *>(table + 255 * 256 + lane * 4) +
                           *reinterpret_cast<const float *>(table + 255 * 256 + 128 + lane * 4);

#pragma unroll
        for (int t = 0; t < UMAX; ++t) {
            const int u = u0 + wp + kLutWarps * t;
            cp_async_wait<UMAX - 1>();
            __syncwarp();
            if (u < u1) {
                const unsigned char *sc = stage + t * S::kScaleTile + (lane >> 3) * (Q * 16);
                uint4 araw[Q];
#pragma unroll
                for (int i = 0; i < Q; ++i) araw[i] = *reinterpret_cast<const uint4 *>(sc + i * 16);
                const uint4 zraw =
                    *reinterpret_cast<const uint4 *>(stage + t * S::kScaleTile + Q * 64 + (lane >> 3) * 16);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    float a_acc = acc[t][r];
#pragma unroll
                    for (int i = 0; i < Q; ++i) {
                        const int pb = (r * Q + i) * 2;  // byte index of slot 0; slot 1 is pb + 1
                        const uint32_t word = wbuf[t][pb >> 2];
                        const uint32_t o0 = __byte_perm(word, lane_off, 0x7604 | ((pb & 3) << 4));
                        const uint32_t o1 = __byte_perm(word, lane_off, 0x7604 | (((pb + 1) & 3) << 4));
                        const float v = *reinterpret_cast<const float *>(smem + o0) +
                                        *reinterpret_cast<const float *>(smem + o1 + 128);
                        const __half ah = reinterpret_cast<const __half *>(&araw[i])[r];
                        a_acc = fmaf(__half2float(ah), v, a_acc);
                    }
                    const __half zh = reinterpret_cast<const __half *>(&zraw)[r];
                    acc[t][r] = fmaf(__half2float(zh), xsum, a_acc);
                }
            }
            __syncwarp();
            request(w + 1, t);
        }
        __syncthreads();
    }
    cp_async_wait<0>();

    // ---- reduce the 8 row sums of each unit over the 32 lanes ---------------------------------
    float *partial = p.k_splits > 1 ? p.partial + size_t(ks) * p.N : nullptr;
#pragma unroll
    for (int t = 0; t < UMAX; ++t) {
        const int u = u0 + wp + kLutWarps * t;
        if (u < u1) {  // warp-uniform
            float v4[4], v2[2], v1;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool up = lane & 16;
                const float keep = up ? acc[t][j + 4] : acc[t][j];
                const float send = up ? acc[t][j] : acc[t][j + 4];
                v4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const bool up = lane & 8;
                const float keep = up ? v4[j + 2] : v4[j];
                const float send = up ? v4[j] : v4[j + 2];
                v2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
            }
            {
                const bool up = lane & 4;
                const float keep = up ? v2[1] : v2[0];
                const float send = up ? v2[0] : v2[1];
                v1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
            }
            v1 += __shfl_xor_sync(0xffffffffu, v1, 2);
            v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
            if ((lane & 3) == 0) {
                const int r = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
                const int n = u * kUnitRows + r;
                if (partial)
                    partial[n] = v1;
                else
                    p.y[n] = __float2half_rn(v1);
            }
        }
    }

    // ---- split-K: the last block to arrive for this row block adds the partials in fixed order --
    if (p.k_splits > 1) {
        __shared__ int s_last;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int old = atomicAdd(p.counters + rbi, 1);
            s_last = (old == p.k_splits - 1);
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int n = u0 * kUnitRows + tid; n < u1 * kUnitRows; n += kLutThreads) {
                float v = 0.f;
                for (int k = 0; k < p.k_splits; ++k) v += __ldcg(p.partial + size_t(k) * p.N + n);
                p.y[n] = __float2half_rn(v);
            }
            if (tid == 0) p.counters[rbi] = 0;
        }
    }
}

template <int Q>
static cudaError_t launch_lut_q(const LutParams &prm, cudaStream_t st)
{
    // The opt-in to more than 48 KB of dynamic shared memory is per function and per device:
    // done on the first launch on each device, remembered afterwards.
    static bool configured[64] = {};
    constexpr int smem = LutSmem<Q>::kTotal;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(lut_gemv_kernel<Q>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    lut_gemv_kernel<Q><<<prm.row_blocks * prm.k_splits, kLutThreads, smem, st>>>(prm);
    return cudaGetLastError();
}

cudaError_t launch_lut_gemv(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *x, uint16_t *y, void *workspace, cudaStream_t st)
{
    LutParams prm;
    prm.planes = static_cast<const uint8_t *>(packed);
    prm.alpha = reinterpret_cast<const uint8_t *>(alpha);
    prm.z = reinterpret_cast<const uint8_t *>(z);
    prm.x = reinterpret_cast<const __half *>(x);
    prm.y = reinterpret_cast<__half *>(y);
    prm.counters = static_cast<int *>(workspace);
    prm.partial = workspace ? reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + kCounterBytes) : nullptr;
    prm.N = d.N;
    prm.K = d.K;
    prm.U = d.N / kUnitRows;
    prm.W = d.K / kWindow;
    prm.row_blocks = plan.row_blocks;
    prm.k_splits = plan.k_splits;
    switch (d.q) {
        case 1: return launch_lut_q<1>(prm, st);
        case 2: return launch_lut_q<2>(prm, st);
        case 3: return launch_lut_q<3>(prm, st);
        case 4: return launch_lut_q<4>(prm, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace bcq

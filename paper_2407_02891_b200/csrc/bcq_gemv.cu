// The BCQ products  y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )  (Eq. bcw + Eq. fuse_step3).
//
//  * generic_kernel: one warp per output row, direct sign arithmetic, any valid shape, either
//    layout, batch 1..16.  The slow, always-available path.
//  * lut_gemv_kernel: the batch-1 hot path for the tiled layout.  Per 512-wide window of K a
//    block builds, in shared memory, all 2^8 signed sums of every 8-activation chunk; packed
//    weight bytes streamed from HBM with 128-bit loads index those tables directly.
#include <type_traits>

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
// lookup-table GEMV (batch 1, tiled layout, group 128)
// =============================================================================================
//
// Block = 16 warps, one block per SM; it owns row units [u0,u1) (8 rows each, at most 64) and
// windows [w0,w1) (at most kMaxWindowsPerBlock).  Warp `wp` owns units u0 + wp + 16 t, t < 4.
//
// Shared memory (the whole 227 KB opt-in is requested):
//   * two 64 KB fp32 tables, double buffered over windows, placed at shared-window addresses
//     that are multiples of 64 KB.  Word address of (entry e, chunk c) = e*64 + (c&1)*32 + (c>>1):
//     lane l looks up chunks 2l and 2l+1 only, so a warp's lookups always hit 32 distinct banks.
//     Entry stride 256 B + 64 KB alignment let ONE byte-permute produce the complete address:
//     byte 1 <- weight byte, bytes 0,2,3 <- (table address + 4*lane).  A lookup is PRMT + LDS.
//   * the block's slice of x converted to fp32 and permuted for the table build, and per-warp
//     staging of the scales, in whichever of the two leftover regions (before / after the
//     tables) is large enough -- their sizes add up to 99 KB, so one always holds the 49 KB needed.
//
// Weight bytes go HBM -> registers (no shared-memory staging: the lookups already use most of
// the shared-memory bandwidth); the bytes of (window w+1, unit t) are requested as soon as those
// of (w, t) are consumed.  Scales go HBM -> shared memory with cp.async (8 lanes share a value).
// fp32 arithmetic is issued two lanes wide (f32x2) to save issue slots: rows come in pairs.

constexpr int kLutThreads = kLutWarps * 32;
constexpr int kTableBytes = 256 * 64 * 4;  // 65536
constexpr int kLutSmemBytes = 232448;      // 227 KB: the per-block opt-in maximum on sm_100
template <int Q>
struct LutSmem {
    static constexpr int kScaleTile = (Q + 1) * 64;  // bytes of alpha+z of one (window, unit)
    static constexpr int kStageBytes = kLutWarps * kLutUnitsPerWarp * kScaleTile;
    static constexpr int kXBytes = kMaxWindowsPerBlock * kWindow * 4;
    static constexpr int kMiscBytes = 64;
    static constexpr int kSideBytes = kStageBytes + kXBytes + kMiscBytes;
    static_assert(2 * kSideBytes <= kLutSmemBytes - 2 * kTableBytes, "side region must fit before or after the tables");
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

template <int I, int N, class F>
__device__ __forceinline__ void static_for(F &&f)
{
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}

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

// table lookups: the address register already holds the complete shared-window address
template <int OFF>
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(OFF));
    return v;
}

// two fp32 lanes in one 64-bit register
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float2 unpack2(f32x2 v)
{
    float2 r;
    asm("mov.b64 {%0,%1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b)
{
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c)
{
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Index, inside a window's 512 staged activations, of activation j of chunk c = 2*(4*lq + k) + s:
// [s][lq][j][k], so that one 128-bit load gives activation j of the four chunks a builder thread owns.
__device__ __forceinline__ int xs_index(int kk)
{
    const int l = kk >> 4, s = (kk >> 3) & 1, j = kk & 7;
    return (((s * 8 + (l >> 2)) * 8 + j) << 2) + (l & 3);
}

// Build one window's table.  Thread t: quad = t & 15 (slot s = quad >> 3, lanes 4*(quad&7) .. +3),
// entry bits 3..7 = t >> 4.  It walks the 8 entries sharing those bits in Gray-code order: one
// packed FMA per entry and chunk pair, one 128-bit conflict-free store per entry.
__device__ __forceinline__ void build_table(unsigned char *table, const float *xs_w, int tid)
{
    const int quad = tid & 15;
    const int hi = tid >> 4;
    const float4 *xq = reinterpret_cast<const float4 *>(xs_w) + quad * 8;  // xq[j] = activation j of 4 chunks
    f32x2 c01 = pack2(0.f, 0.f), c23 = c01;
#pragma unroll
    for (int j = 3; j < 8; ++j) {
        const float4 v = xq[j];
        const float sg = ((hi >> (j - 3)) & 1) ? 1.f : -1.f;
        const f32x2 s2 = pack2(sg, sg);
        c01 = fma2(s2, pack2(v.x, v.y), c01);
        c23 = fma2(s2, pack2(v.z, v.w), c23);
    }
    f32x2 x01[3], x23[3];
    const f32x2 m1 = pack2(-1.f, -1.f), p2 = pack2(2.f, 2.f), m2 = pack2(-2.f, -2.f);
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        const float4 v = xq[j];
        x01[j] = pack2(v.x, v.y);
        x23[j] = pack2(v.z, v.w);
        c01 = fma2(m1, x01[j], c01);
        c23 = fma2(m1, x23[j], c23);
    }
    unsigned char *dst = table + quad * 16 + hi * (8 * 256);
    static_for<0, 8>([&](auto step_c) {
        constexpr int step = decltype(step_c)::value;
        constexpr int gray = step ^ (step >> 1);
        if constexpr (step > 0) {
            constexpr int bit = (step & 1) ? 0 : ((step & 2) ? 1 : 2);  // lowest set bit of step
            constexpr bool on = (gray >> bit) & 1;
            c01 = fma2(on ? p2 : m2, x01[bit], c01);
            c23 = fma2(on ? p2 : m2, x23[bit], c23);
        }
        const float2 a = unpack2(c01), b = unpack2(c23);
        *reinterpret_cast<float4 *>(dst + gray * 256) = make_float4(a.x, a.y, b.x, b.y);
    });
}

template <int Q>
__global__ void __launch_bounds__(kLutThreads, 1) lut_gemv_kernel(const LutParams p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    using S = LutSmem<Q>;
    constexpr int UMAX = kLutUnitsPerWarp;
    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;

    const int rbi = blockIdx.x % p.row_blocks, ks = blockIdx.x / p.row_blocks;
    const int u0 = int((long long)rbi * p.U / p.row_blocks), u1 = int((long long)(rbi + 1) * p.U / p.row_blocks);
    const int w0 = int((long long)ks * p.W / p.k_splits), w1 = int((long long)(ks + 1) * p.W / p.k_splits);

    // ---- carve shared memory -------------------------------------------------------------------
    const uint32_t base = smem_u32(smem);
    const uint32_t tab0 = (base + 0xFFFFu) & ~0xFFFFu;  // shared-window address of table 0
    unsigned char *tables = smem + (tab0 - base);
    unsigned char *side = (tab0 - base >= uint32_t(S::kSideBytes)) ? smem : tables + 2 * kTableBytes;
    unsigned char *stage = side + wp * (UMAX * S::kScaleTile);
    float *xs = reinterpret_cast<float *>(side + S::kStageBytes);
    int *s_last = reinterpret_cast<int *>(side + S::kStageBytes + S::kXBytes);
    const uint32_t stage_u32 = smem_u32(stage);

    // number of units this warp owns
    int nu = (u1 - u0 - wp + kLutWarps - 1) / kLutWarps;
    nu = nu < 0 ? 0 : nu;

    uint32_t wbuf[UMAX][4 * Q];
    f32x2 acc[UMAX][4];
    float zacc[UMAX];
#pragma unroll
    for (int t = 0; t < UMAX; ++t) {
        zacc[t] = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[t][r] = pack2(0.f, 0.f);
    }

    // request (window w, unit slot T): weight bytes to registers, scales to staging
    auto request = [&](int w, auto T) {
        constexpr int t = decltype(T)::value;
        if (w < w1 && t < nu) {
            const size_t tile = size_t(w) * p.U + (u0 + wp + kLutWarps * t);
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
    static_for<0, UMAX>([&](auto T) { request(w0, T); });

    // ---- this block's slice of x: fp16 -> fp32, permuted for the table build ---------------------
    {
        const __half *xg = p.x + size_t(w0) * kWindow;
        const int count = (w1 - w0) * kWindow;
        for (int e = tid; e < count; e += kLutThreads)
            xs[(e & ~(kWindow - 1)) + xs_index(e & (kWindow - 1))] = __half2float(xg[e]);
    }
    __syncthreads();
    build_table(tables, xs, tid);
    __syncthreads();

    for (int w = w0; w < w1; ++w) {
        const int cur = (w - w0) & 1;
        if (w + 1 < w1) build_table(tables + (cur ^ 1) * kTableBytes, xs + (w + 1 - w0) * kWindow, tid);

        const uint32_t lane_off = tab0 + uint32_t(cur * kTableBytes + lane * 4);
        // sum of this lane's 16 activations (the all-ones entries of its two chunks), then of its group
        float xsum = lds_f32<255 * 256>(lane_off) + lds_f32<255 * 256 + 128>(lane_off);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 4);

        static_for<0, UMAX>([&](auto T) {
            constexpr int t = decltype(T)::value;
            cp_async_wait<UMAX - 1>();
            __syncwarp();
            if (t < nu) {
                const unsigned char *tile = stage + t * S::kScaleTile;
                uint4 araw[Q];
#pragma unroll
                for (int i = 0; i < Q; ++i)
                    araw[i] = *reinterpret_cast<const uint4 *>(tile + (lane >> 3) * (Q * 16) + i * 16);
                // offsets: lane (g, j) adds z[g][row j] * (sum of x over group g)
                const __half zh = *reinterpret_cast<const __half *>(tile + Q * 64 + lane * 2);
                zacc[t] = fmaf(__half2float(zh), xsum, zacc[t]);
                static_for<0, 4>([&](auto PR) {
                    constexpr int pr = decltype(PR)::value;  // rows 2pr and 2pr+1
                    f32x2 a2 = acc[t][pr];
                    static_for<0, Q>([&](auto I) {
                        constexpr int i = decltype(I)::value;
                        constexpr int b0 = ((2 * pr) * Q + i) * 2, b1 = ((2 * pr + 1) * Q + i) * 2;
                        const uint32_t word0 = wbuf[t][b0 >> 2], word1 = wbuf[t][b1 >> 2];
                        const float v00 = lds_f32<0>(__byte_perm(word0, lane_off, 0x7604 | ((b0 & 3) << 4)));
                        const float v01 = lds_f32<128>(__byte_perm(word0, lane_off, 0x7604 | (((b0 + 1) & 3) << 4)));
                        const float v10 = lds_f32<0>(__byte_perm(word1, lane_off, 0x7604 | ((b1 & 3) << 4)));
                        const float v11 = lds_f32<128>(__byte_perm(word1, lane_off, 0x7604 | (((b1 + 1) & 3) << 4)));
                        const f32x2 s2 = add2(pack2(v00, v10), pack2(v01, v11));
                        const uint32_t aw = reinterpret_cast<const uint32_t *>(&araw[i])[pr];
                        const float2 af = __half22float2(*reinterpret_cast<const __half2 *>(&aw));
                        a2 = fma2(pack2(af.x, af.y), s2, a2);
                    });
                    acc[t][pr] = a2;
                });
            }
            __syncwarp();
            request(w + 1, T);
        });
        __syncthreads();
    }
    cp_async_wait<0>();

    // ---- reduce each unit's 8 row sums over the 32 lanes: lane l ends with row l & 7 -------------
    float *partial = p.k_splits > 1 ? p.partial + size_t(ks) * p.N : nullptr;
    static_for<0, UMAX>([&](auto T) {
        constexpr int t = decltype(T)::value;
        if (t < nu) {
            float v4[4], v2[2], v1;
#pragma unroll
            for (int pr = 0; pr < 4; ++pr) {  // lane bit 0 picks the row of the pair
                const float2 a = unpack2(acc[t][pr]);
                const bool odd = lane & 1;
                v4[pr] = (odd ? a.y : a.x) + __shfl_xor_sync(0xffffffffu, odd ? a.x : a.y, 1);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {  // lane bit 1 picks the pair inside a half
                const bool up = lane & 2;
                v2[h] = (up ? v4[2 * h + 1] : v4[2 * h]) + __shfl_xor_sync(0xffffffffu, up ? v4[2 * h] : v4[2 * h + 1], 2);
            }
            {
                const bool up = lane & 4;  // lane bit 2 picks the half
                v1 = (up ? v2[1] : v2[0]) + __shfl_xor_sync(0xffffffffu, up ? v2[0] : v2[1], 4);
            }
            v1 += zacc[t];  // lane (g, j) holds group g's offset term of row j = l & 7
            v1 += __shfl_xor_sync(0xffffffffu, v1, 8);
            v1 += __shfl_xor_sync(0xffffffffu, v1, 16);
            if (lane < 8) {
                const int n = (u0 + wp + kLutWarps * t) * kUnitRows + lane;
                if (partial)
                    partial[n] = v1;
                else
                    p.y[n] = __float2half_rn(v1);
            }
        }
    });

    // ---- split-K: the last block to arrive for this row block adds the partials in fixed order --
    if (p.k_splits > 1) {
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int old = atomicAdd(p.counters + rbi, 1);
            *s_last = (old == p.k_splits - 1);
        }
        __syncthreads();
        if (*s_last) {
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
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(lut_gemv_kernel<Q>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLutSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    lut_gemv_kernel<Q><<<prm.row_blocks * prm.k_splits, kLutThreads, kLutSmemBytes, st>>>(prm);
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

// Small-batch BCQ product (2 <= B <= 16 columns, tiled layout) for sm_100a: every weight tile is
// read from HBM once and serves all columns.
//
//   Y[b] = sum_g ( sum_i alpha_i (B_i X[b])_g + z (sum X[b])_g )          (Eq. bcw + Eq. fuse_step3)
//
// With several columns the product is a (thin) dense contraction, so the sums go through the
// tensor cores: mma.sync m16n8k16, fp16 operands, fp32 accumulators, operands in registers.  A
// weight bit is expanded in registers to the fp16 value +-alpha_i of its (row, group) -- +alpha and
// -alpha differ in the sign bit only, so a shift, an AND and an XOR turn two bits of a plane word
// into one operand register -- and x is the other operand, so the products alpha * x are exact and
// all additions are fp32.  The offset term is one more MMA per tile pair: z times the per-group sums
// of x, which the loader warps compute in fp32 and pass on as an fp16 (high, low) pair.
// (The shared-memory-operand tensor path, tcgen05, would need the expanded weights -- 16 times the
// packed bytes -- written to shared or tensor memory first; with at most 16 columns that costs more
// than the MMAs themselves, so the register-operand form is used.)
//
// Operand roles: A (16 x 16) = 16 weight rows (two row units, i.e. two tiles of the same window)
// x 16 weights; B (16 x 8) = the same 16 weights of 8 columns of X; C (16 x 8) fp32.  Lane
// (m = lane / 4, t = lane % 4) holds A elements of rows m and m + 8 only, which is exactly the
// tile's own distribution: it reads the 16 bytes per plane of tile lane 8 t + m (row m, group t).
// Because the scale is folded into the operand, the 16 weights of one MMA may come from four
// different groups (one per t).  The tile stores a row's chunks rotated by two per row (for the
// batch-1 kernel's bank mapping); the lane undoes that while loading -- word rotation through the
// load address, the odd half-word through one byte-permute -- so that all rows of an MMA see the
// same weights k.  X is staged per 512-wide window by two loader warps, already in operand order
// (one 8-byte shared-memory load per MMA and lane), double buffered.
//
// The block structure is that of the batch-1 kernel: one block per SM owns a range of row units and
// a range of windows; every consumer warp owns a few ring slots (one slot = one tile pair = one
// contiguous piece of global memory) that it refills itself with bulk async copies; deterministic
// split-K through fp32 partials and an arrival counter; all waits bounded.
#include "bcq_async.cuh"
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kMmaLoaderWarps = 2;
constexpr int kMmaThreads = (kMmaLoaderWarps + kMmaWarps) * 32;   // 768
constexpr int kMmaConsumerThreads = kMmaWarps * 32;
constexpr int kMmaSmemBytes = 232448;    // 227 KB: the per-block opt-in maximum
constexpr int kMmaFixedBytes = 2048;     // barriers and flags
constexpr int kMmaMaxSlotsPerWarp = 4;
constexpr int kMmaMaxSlots = kMmaWarps * kMmaMaxSlotsPerWarp;
constexpr int kXGroupBytes = 264;        // 256 B of operand-ordered x of one (column, group) + 8 B: no bank conflicts
constexpr int kXRowBytes = 4 * kXGroupBytes;

static_assert(8 * kMmaMaxSlots + 64 <= kMmaFixedBytes, "barrier area");

__device__ int g_mma_status = 0;  // 0, or the code of the wait that ran out (sticky until taken)

struct MmaParams {
    const uint8_t *tiles;
    const uint16_t *alpha;   // per-row scales only: [u][i][r]
    const uint16_t *z;       // per-row scales only: [u][r]
    const __half *X;         // [B][K]
    __half *Y;               // [B][N]
    float *partial;          // [k_splits][B][N] when k_splits > 1
    int *counters;           // [row_blocks]
    int N, K, U, W, B;
    int row_blocks, k_splits;
};

enum { kMmaWaitFull = 11, kMmaWaitXReady = 12, kMmaWaitXFree = 13, kMmaWaitDrain = 14 };

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Q planes; GROUPED: scales per (row, group of 128) inside the tiles, else per row in arrays;
// WIDE: 9..16 columns (two MMAs per step), else at most 8.
template <int Q, bool GROUPED, bool WIDE>
__global__ void __launch_bounds__(kMmaThreads, 1) mma_gemm_kernel(const MmaParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int T = Q * 512 + (GROUPED ? Q * 64 + 64 : 0);   // bytes of one tile
    constexpr int kSlotBytes = 2 * T;
    constexpr int BR = WIDE ? 16 : 8;                          // staged columns (zero-filled beyond B)
    constexpr int kXBufBytes = BR * kXRowBytes;
    constexpr int PMAX = kMmaPairsPerWarp;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int rbi = blockIdx.x % p.row_blocks, ks = blockIdx.x / p.row_blocks;
    const int u0 = int((long long)rbi * p.U / p.row_blocks), u1 = int((long long)(rbi + 1) * p.U / p.row_blocks);
    const int w0 = int((long long)ks * p.W / p.k_splits), w1 = int((long long)(ks + 1) * p.W / p.k_splits);
    const int V = u1 - u0, P = (V + 1) >> 1;   // row units and unit pairs of this block
    const int nwin = w1 - w0;

    // ---- shared memory: [barriers | x operands (2 buffers) | group sums of x (2 buffers) | ring] ----
    unsigned char *fixed = smem;
    unsigned char *xs = smem + kMmaFixedBytes;
    uint32_t *xsum = reinterpret_cast<uint32_t *>(xs + 2 * kXBufBytes);   // [2][BR][4] fp16 (high, low)
    unsigned char *ring = xs + 2 * kXBufBytes + 2 * BR * 16;
    constexpr int kRingBytes = kMmaSmemBytes - kMmaFixedBytes - 2 * kXBufBytes - 2 * BR * 16;
    constexpr int NS = kRingBytes / kSlotBytes < kMmaMaxSlots ? kRingBytes / kSlotBytes : kMmaMaxSlots;
    constexpr int D = NS / kMmaWarps;   // ring slots per consumer warp
    static_assert(D >= 1, "ring too small");

    const uint32_t bars = smem_u32(fixed);
    const uint32_t bar_full = bars;
    const uint32_t bar_x_ready = bars + 8 * kMmaMaxSlots, bar_x_free = bar_x_ready + 16;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(fixed + 8 * kMmaMaxSlots + 32);
    int *s_last = const_cast<int *>(abort_flag) + 1;

    if (warp == 0) {   // one warp initialises the barriers, a few each
        for (int s = lane; s < kMmaMaxSlots; s += 32) mbar_init(bar_full + 8 * s, 1);
        if (lane < 2) {
            mbar_init(bar_x_ready + 8 * lane, BR / 8);   // lane 0 of every loader warp that stages columns
            mbar_init(bar_x_free + 8 * lane, P < kMmaWarps ? P : kMmaWarps);   // the consumer warps that have jobs
        }
        if (lane == 0) *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch, as in the batch-1 kernel: weights are constants and may be
    // fetched before the previous kernel in the stream has finished; X, partials, counters, Y may not.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- consumer warps: their jobs (window-major, then their pairs), D of them in flight ---------
    const int cw = warp - kMmaLoaderWarps;
    const int mine = (cw >= 0 && P > cw) ? (P - cw + kMmaWarps - 1) / kMmaWarps : 0;   // pairs of this warp per window
    const int total_jobs = mine * nwin;
    int issued = 0, consumed = 0, iw = 0, it = 0;
    auto issue_next = [&](int slot_d) {   // lane 0 of a consumer warp only
        if (issued < total_jobs) {
            const int ua = u0 + 2 * (cw + kMmaWarps * it);
            const size_t tile = size_t(w0 + iw) * p.U + ua;
            const uint32_t bytes = (ua + 1 < u1) ? kSlotBytes : T;   // the last pair of an odd block is one tile
            const int s = cw + kMmaWarps * slot_d;
            const uint32_t full = bar_full + 8 * s;
            mbar_expect_tx(full, bytes);
            bulk_g2s(smem_u32(ring + s * kSlotBytes), p.tiles + tile * T, bytes, full);
            ++issued;
            if (++it == mine) {
                it = 0;
                ++iw;
            }
        }
    };
    if (cw >= 0 && lane == 0)
        for (int d0 = 0; d0 < D; ++d0) issue_next(d0);

    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp < kMmaLoaderWarps) {
        // ---- loaders: thread (column b, group t) stages its 128 activations of every window ----------
        // in the order the consumers' B operands want them, plus their fp32 sum as fp16 (high, low).
        const int b = tid >> 2, t = tid & 3;
        if (b >= BR) return;
        for (int wi = 0; wi < nwin; ++wi) {
            const int buf = wi & 1, use = wi >> 1;
            uint32_t x2[64];   // x2[j] = (x[2j], x[2j+1]) of the group
            if (b < p.B) {
                const uint4 *src = reinterpret_cast<const uint4 *>(p.X + size_t(b) * p.K + size_t(w0 + wi) * kWindow + 128 * t);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const uint4 v = __ldg(src + j);
                    x2[4 * j + 0] = v.x, x2[4 * j + 1] = v.y, x2[4 * j + 2] = v.z, x2[4 * j + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 64; ++j) x2[j] = 0u;
            }
            if (use > 0 && !mbar_wait<true>(bar_x_free + 8 * buf, (use - 1) & 1, abort_flag, kMmaWaitXFree, &g_mma_status)) break;
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&x2[j]));
                sum += f.x;
                sum += f.y;
            }
            const __half hi = __float2half_rn(sum), lo = __float2half_rn(sum - __half2float(hi));
            xsum[(buf * BR + b) * 4 + t] = uint32_t(__half_as_ushort(hi)) | (uint32_t(__half_as_ushort(lo)) << 16);
            // Operand order.  Consumer lane (., t) keeps in register position k the plane word of chunks
            // 4L .. 4L+3 of its group, L = (k + t) mod 4; MMA (k, ii) takes, per plane word, the bit pairs
            // (2ii, 2ii + 16) and (2ii + 1, 2ii + 17): weights 2(ii mod 4) and + 1 of chunks 4L + ii/4 and
            // 4L + 2 + ii/4.
            unsigned char *dst = xs + buf * kXBufBytes + b * kXRowBytes + t * kXGroupBytes;
            static_for<0, 4>([&](auto LL) {
                constexpr int L = decltype(LL)::value;
                const int k = (L - t) & 3;
                static_for<0, 8>([&](auto II) {
                    constexpr int ii = decltype(II)::value;
                    const uint32_t lo2 = x2[4 * (4 * L + (ii >> 2)) + (ii & 3)];
                    const uint32_t hi2 = x2[4 * (4 * L + 2 + (ii >> 2)) + (ii & 3)];
                    uint2 out;
                    out.x = __byte_perm(lo2, hi2, 0x5410);   // even weight of both chunks
                    out.y = __byte_perm(lo2, hi2, 0x7632);   // odd weight of both chunks
                    *reinterpret_cast<uint2 *>(dst + (k * 8 + ii) * 8) = out;
                });
            });
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_x_ready + 8 * buf);
        }
        return;
    }

    // =============================================================================================
    // ---- consumers ---------------------------------------------------------------------------------
    const int ctid = tid - kMmaLoaderWarps * 32;
    const int m = lane >> 2, t = lane & 3;
    const int lam = 8 * t + m;                 // the tile lane of (row m, group t)
    const int rot = (m + 1) >> 1;              // the row's chunks are stored rotated by 2 m bytes
    const uint32_t sel = (m & 1) ? 0x5432u : 0x3210u;
    int woff[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) woff[k] = lam * 16 + 4 * ((k + t - rot) & 3);

    float acc[PMAX][4], acc_hi[WIDE ? PMAX : 1][4];
#pragma unroll
    for (int pp = 0; pp < PMAX; ++pp)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[pp][e] = 0.f;
#pragma unroll
    for (int pp = 0; pp < (WIDE ? PMAX : 1); ++pp)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc_hi[pp][e] = 0.f;
    bool alive = true;
    int d = 0, fill = 0;   // this warp's ring position: slot cw + kMmaWarps * d, fill number

    for (int wi = 0; wi < nwin && alive && mine > 0; ++wi) {   // warps without jobs go straight to the end
        const int buf = wi & 1;
        if (!mbar_wait<true>(bar_x_ready + 8 * buf, (wi >> 1) & 1, abort_flag, kMmaWaitXReady, &g_mma_status)) {
            alive = false;
            break;
        }
        const unsigned char *xb = xs + buf * kXBufBytes + m * kXRowBytes + t * kXGroupBytes;   // column m (and m + 8)
        const uint32_t xs_lo = xsum[(buf * BR + m) * 4 + t];
        const uint32_t xs_hi = WIDE ? xsum[(buf * BR + m + 8) * 4 + t] : 0u;

        static_for<0, PMAX>([&](auto PP) {
            constexpr int pp = decltype(PP)::value;
            if (alive && cw + kMmaWarps * pp < P) {
                const int s = cw + kMmaWarps * d;
                if (!mbar_wait(bar_full + 8 * s, fill & 1, abort_flag, kMmaWaitFull, &g_mma_status)) {
                    alive = false;
                } else {
                    ++consumed;
                    const unsigned char *slot = ring + s * kSlotBytes;
                    [[maybe_unused]] const int ua = u0 + 2 * (cw + kMmaWarps * pp);
                    uint32_t Wd[2][Q][4];   // plane words of (row m, group t) of both tiles, rotation undone
                    uint32_t nb[2][Q];      // (-alpha_i, -alpha_i) as fp16 pairs
                    uint32_t zz[2];         // (z, z)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int i = 0; i < Q; ++i) {
                            const unsigned char *base = slot + h * T + i * 512;
                            uint32_t in[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) in[k] = *reinterpret_cast<const uint32_t *>(base + woff[k]);
#pragma unroll
                            for (int k = 0; k < 4; ++k) Wd[h][i][k] = __byte_perm(in[k], in[(k + 1) & 3], sel);
                        }
                        uint32_t sc[Q + 1];
                        if constexpr (GROUPED) {
                            const uint16_t *sp = reinterpret_cast<const uint16_t *>(slot + h * T + Q * 512) + lam * (Q + 1);
#pragma unroll
                            for (int i = 0; i <= Q; ++i) sc[i] = sp[i];
                        } else {
                            const int u = ua + h;
#pragma unroll
                            for (int i = 0; i < Q; ++i) sc[i] = u < u1 ? __ldg(p.alpha + (size_t(u) * Q + i) * kUnitRows + m) : 0;
                            sc[Q] = u < u1 ? __ldg(p.z + size_t(u) * kUnitRows + m) : 0;
                        }
#pragma unroll
                        for (int i = 0; i < Q; ++i) nb[h][i] = (sc[i] * 0x10001u) ^ 0x80008000u;
                        zz[h] = sc[Q] * 0x10001u;
                    }
                    // The pair is in registers: order those reads before the next copy into the slot
                    // (generic-proxy reads, then an async-proxy write), then refill the slot.
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) issue_next(d);

                    // Independent accumulation chains (an MMA waits for the previous one into the same
                    // registers): one per plane; folded into the pair's accumulators at the end.
                    constexpr int NCH = WIDE ? (Q > 1 ? 2 : 1) : Q;
                    float c[NCH][4], ch[WIDE ? NCH : 1][4];
#pragma unroll
                    for (int j = 0; j < NCH; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) c[j][e] = 0.f;
#pragma unroll
                    for (int j = 0; j < (WIDE ? NCH : 1); ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) ch[j][e] = 0.f;

                    // offset term: rows m, m + 8 times (z, z) at k = 2t, 2t + 1; x sums (high, low) there
                    mma_16816(acc[pp], zz[0], zz[1], 0u, 0u, xs_lo, 0u);
                    if constexpr (WIDE) mma_16816(acc_hi[pp], zz[0], zz[1], 0u, 0u, xs_hi, 0u);

                    static_for<0, 4>([&](auto KK) {
                        constexpr int k = decltype(KK)::value;
                        static_for<0, 8>([&](auto II) {
                            constexpr int ii = decltype(II)::value;
                            constexpr int sh0 = 15 - 2 * ii, sh1 = 14 - 2 * ii;
                            const uint2 xf = *reinterpret_cast<const uint2 *>(xb + (k * 8 + ii) * 8);
                            uint2 xg = make_uint2(0u, 0u);
                            if constexpr (WIDE) xg = *reinterpret_cast<const uint2 *>(xb + 8 * kXRowBytes + (k * 8 + ii) * 8);
#pragma unroll
                            for (int i = 0; i < Q; ++i) {
                                const uint32_t a0 = ((Wd[0][i][k] << sh0) & 0x80008000u) ^ nb[0][i];
                                const uint32_t a1 = ((Wd[1][i][k] << sh0) & 0x80008000u) ^ nb[1][i];
                                const uint32_t a2 = ((Wd[0][i][k] << sh1) & 0x80008000u) ^ nb[0][i];
                                const uint32_t a3 = ((Wd[1][i][k] << sh1) & 0x80008000u) ^ nb[1][i];
                                mma_16816(c[i % NCH], a0, a1, a2, a3, xf.x, xf.y);
                                if constexpr (WIDE) mma_16816(ch[i % NCH], a0, a1, a2, a3, xg.x, xg.y);
                            }
                        });
                    });
#pragma unroll
                    for (int j = 0; j < NCH; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[pp][e] += c[j][e];
                            if constexpr (WIDE) acc_hi[pp][e] += ch[j][e];
                        }
                }
                if (++d == D) {
                    d = 0;
                    ++fill;
                }
            }
        });
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_x_free + 8 * buf);
    }

    // Gave up on a wait: copies this warp started may still be in flight.  See them land (bounded)
    // before the block's shared memory can be handed to another block.
    if (!alive && lane == 0) {
        for (int j = consumed; j < issued; ++j) {
            bool landed = false;
            for (int itr = 0; itr < kSpinLimit && !landed; ++itr)
                landed = mbar_try_wait(bar_full + 8 * (cw + kMmaWarps * (j % D)), uint32_t((j / D) & 1));
            if (!landed) atomicExch(&g_mma_status, int(kMmaWaitDrain));
        }
    }

    // ---- store: lane (m, t) holds rows m of both units for columns 2t, 2t+1 (and 8 + those) -------
    float *partial = p.k_splits > 1 ? p.partial + size_t(ks) * p.B * p.N : nullptr;
    auto put = [&](int b, int n, float v) {
        if (b < p.B) {
            if (partial)
                partial[size_t(b) * p.N + n] = v;
            else
                p.Y[size_t(b) * p.N + n] = __float2half_rn(v);
        }
    };
#pragma unroll
    for (int pp = 0; pp < PMAX; ++pp) {
        if (cw + kMmaWarps * pp < P) {
            const int ua = u0 + 2 * (cw + kMmaWarps * pp);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (ua + h < u1) {
                    const int n = (ua + h) * kUnitRows + m;
                    put(2 * t, n, acc[pp][2 * h]);
                    put(2 * t + 1, n, acc[pp][2 * h + 1]);
                    if constexpr (WIDE) {
                        put(8 + 2 * t, n, acc_hi[pp][2 * h]);
                        put(9 + 2 * t, n, acc_hi[pp][2 * h + 1]);
                    }
                }
            }
        }
    }

    // ---- split-K: the last block to arrive for this row block adds the partials in fixed order --
    if (p.k_splits > 1) {
        __threadfence();
        named_barrier(2, kMmaConsumerThreads);
        if (ctid == 0) {
            const int old = atomicAdd(p.counters + rbi, 1);
            *s_last = (old == p.k_splits - 1);
        }
        named_barrier(2, kMmaConsumerThreads);
        if (*s_last) {
            __threadfence();
            const int R = V * kUnitRows;
            for (int idx = ctid; idx < p.B * R; idx += kMmaConsumerThreads) {
                const int b = idx / R, n = u0 * kUnitRows + idx % R;
                float v = 0.f;
                for (int k0 = 0; k0 < p.k_splits; k0 += 8) {
                    float part[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        part[k] = (k0 + k < p.k_splits) ? __ldcg(p.partial + (size_t(k0 + k) * p.B + b) * p.N + n) : 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) v += part[k];
                }
                p.Y[size_t(b) * p.N + n] = __float2half_rn(v);
            }
            if (ctid == 0) p.counters[rbi] = 0;
        }
    }
}

template <int Q, bool GROUPED, bool WIDE>
static cudaError_t launch_mma_q(const MmaParams &prm, cudaStream_t st)
{
    static bool configured[64] = {};   // the shared-memory opt-in is per function and per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(mma_gemm_kernel<Q, GROUPED, WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMmaSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(prm.row_blocks * prm.k_splits);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = kMmaSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, mma_gemm_kernel<Q, GROUPED, WIDE>, prm);
}

template <int Q>
static cudaError_t launch_mma_sel(const MmaParams &prm, bool grouped, cudaStream_t st)
{
    const bool wide = prm.B > 8;
    if (grouped) return wide ? launch_mma_q<Q, true, true>(prm, st) : launch_mma_q<Q, true, false>(prm, st);
    return wide ? launch_mma_q<Q, false, true>(prm, st) : launch_mma_q<Q, false, false>(prm, st);
}

cudaError_t launch_mma_gemm(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *X, uint16_t *Y, int B, void *workspace, cudaStream_t st)
{
    MmaParams prm;
    prm.tiles = static_cast<const uint8_t *>(packed);
    prm.alpha = alpha;   // used with per-row scales only
    prm.z = z;
    prm.X = reinterpret_cast<const __half *>(X);
    prm.Y = reinterpret_cast<__half *>(Y);
    prm.counters = static_cast<int *>(workspace);
    prm.partial = workspace ? reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + kCounterBytes) : nullptr;
    prm.N = d.N;
    prm.K = d.K;
    prm.U = d.N / kUnitRows;
    prm.W = d.K / kWindow;
    prm.B = B;
    prm.row_blocks = plan.row_blocks;
    prm.k_splits = plan.k_splits;
    const bool grouped = d.group != 0;
    switch (d.q) {
        case 1: return launch_mma_sel<1>(prm, grouped, st);
        case 2: return launch_mma_sel<2>(prm, grouped, st);
        case 3: return launch_mma_sel<3>(prm, grouped, st);
        case 4: return launch_mma_sel<4>(prm, grouped, st);
    }
    return cudaErrorInvalidValue;
}

// Read and clear the device status word (synchronises with the device).
cudaError_t mma_status_take(int *status)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_mma_status, sizeof(int));
    if (e != cudaSuccess) return e;
    if (v != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbol(g_mma_status, &zero, sizeof(int));
    }
    *status = v;
    return e;
}

}  // namespace bcq

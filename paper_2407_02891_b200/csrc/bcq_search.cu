// Output error of the candidates of the GPTQT search (Eq. gptqt step 2; Eq. reexplore) on tcgen05.
//
// For one re-explored scale (W_int, S, qbias of step 1 are given) and a set of BCchoice candidates p:
//
//     err[p][n] = sum_t ( sum_k ( S lut_p[W_int[n][k]] + qbias - W[n][k] ) X[t][k] )^2
//
// lut_p[v] = the integer of BCchoice p nearest to v (Eq. round).  The inner sum is a dense contraction
// dW_p (N x K) times X^T (K x T): here the tensor cores are the right unit.  A block owns 128 rows of W
// and up to four candidates; per 64-wide slice of K its threads form the four dW_p tiles in fp16 (dW_p = S step_p[v] + r:
// step_p[v] = lut_p[v] - v, one shared-memory word per element holds it for all four candidates; r = S v + qbias - W, the
// residual of step 1, fp32 and rounded to fp16 once; one fp16 fused multiply-add per pair of elements and candidate)
// straight into shared memory in the 128-byte-swizzled K-major
// operand layout, and a warp of its own issues tcgen05.mma (M = 128, N = T, K = 16, fp16 x fp16 -> fp32) into
// one accumulator per candidate in tensor memory.  The slices of X (same layout), W and W_int arrive by tensor-map
// copies that one thread starts: thousands of 16-byte loads per slice would hold the forming warps at the load
// queue.  Two operand stages: the 16 forming warps publish a stage on its "full" mbarrier, the issuing warp hands it
// back by tcgen05.commit on its "free" mbarrier, so the tensor cores work on one slice while the next is formed
// (issuing 16 MMAs holds a thread for about a microsecond: a forming thread cannot do it).  At the end every row's
// T outputs are read back with tcgen05.ld, squared and summed.  Several scale factors share a launch (grid z).
//
// All waits are bounded; a wait that runs out sets a device status word (see search_status_take), the
// block still frees its tensor memory and returns.
#include <cuda.h>   // CUtensorMap and its enumerations (types only: the encoder is taken from the runtime)

#include "bcq_async.cuh"
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kSearchThreads = 512;      // 16 warps form the operand tiles (latency-bound with fewer)
constexpr int kSearchBlock = kSearchThreads + 32;   // + the warp that issues the MMAs
constexpr int kSearchRows = 128;        // rows of W per block = M of the MMA
constexpr int kSearchKTile = 64;        // weights along K per stage: 128 bytes of fp16, one swizzle row
constexpr int kSearchMaxCand = 4;       // candidates (accumulators) per block
constexpr int kSearchATile = kSearchRows * kSearchKTile * 2;   // 16 KB
constexpr int kSearchMaxT = 256;
constexpr int kSearchWTile = kSearchRows * kSearchKTile * 2;   // a slice of W: 16 KB
constexpr int kSearchITile = kSearchRows * kSearchKTile;       // a slice of W_int: 8 KB
constexpr int kSearchSpin = 1 << 22;

static __device__ int g_search_status = 0;

struct SearchParams {
    const __half *W;        // [N][K]
    const uint8_t *w_int;   // [N][K]
    const __half *S;        // [N][G] per scale factor, scale_stride elements apart
    const __half *qbias;    // [N][G], likewise
    size_t scale_stride;
    const __half *X;        // [T][K]
    float *err_rows;        // [scale factor][P][N]
    int N, K, G, L;         // L = weights per scaling unit (K when one per row)
    int T, P;               // T: tokens of this launch (a piece of at most 256 of the call's)
    int accumulate;         // add to err_rows instead of writing it (every piece but the first)
    int cand_per_block;     // 1..4, so that cand_per_block * T <= 512 columns of tensor memory
    int tmem_cols;          // power of two >= 32 covering cand_per_block * T
    int lut_size;           // 2^n_bits <= 64
    const float *lut;       // [P][64]: lut[p][v] = the integer of BCchoice p nearest to v
};

__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    // K-major operand, 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart
    uint64_t d = 0;
    d |= uint64_t((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= uint64_t(1) << 16;                        // leading byte offset (unused with a swizzled K-major tile)
    d |= uint64_t(1024 >> 4) << 32;                // stride byte offset: 8 rows further on
    d |= uint64_t(1) << 46;                        // descriptor version of this architecture
    d |= uint64_t(2) << 61;                        // 128-byte swizzle
    return d;
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool search_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int code)
{
    for (int it = 0; it < kSearchSpin; ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        __nanosleep(64);
        if ((it & 255) == 255 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(&g_search_status, code);
    return false;
}

// all forming threads take the same decision (a wait that gives up must not split them at a barrier)
__device__ __forceinline__ bool formers_all(bool ok)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.and.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(ok ? 1u : 0u), "n"(kSearchThreads)
        : "memory");
    return out != 0;
}

// one box of a tiled tensor map into shared memory, completion counted in bytes on an mbarrier (x: the
// innermost coordinate in elements, a multiple of 64 here: 64- or 128-byte aligned)
__device__ __forceinline__ void tma_box_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                 "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// a copy this block has started must have landed before the block's shared memory is given up
__device__ __forceinline__ void search_drain(uint32_t bar, uint32_t parity)
{
    for (int it = 0; it < kSearchSpin; ++it) {
        if (mbar_test_wait(bar, parity)) return;
        __nanosleep(64);
    }
}

// grid (row tiles of 128, groups of cand_per_block candidates, scale factors); dynamic shared memory: 2 stages x
// (cand_per_block x 16 KB of dW tiles | X's slice, T x 128 bytes rounded up to 1 KB | W's slice 16 KB | W_int's 8 KB),
// 1024-byte aligned.
__global__ void __launch_bounds__(kSearchBlock, 1)
    search_error_kernel(const SearchParams p, const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
                        const __grid_constant__ CUtensorMap imap)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // stage 0 free, stage 1 free, all done, stage 0/1 full, X of stage 0/1 landed, W and W_int of stage 0/1 landed
    __shared__ __align__(8) unsigned long long bars[9];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    // per value v of W_int one word: byte c = 128 + lut_c[v] - v, the step from v to the nearest integer of the block's
    // candidate c (between -63 and 63).  One lookup per operand element serves the four candidates.
    __shared__ uint32_t step_s[64];
    __shared__ float part[4][kSearchMaxCand][kSearchRows];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cand0 = blockIdx.y * p.cand_per_block;
    const int ncand = min(p.cand_per_block, p.P - cand0);
    const int T = p.T;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_bytes = uint32_t(p.cand_per_block) * kSearchATile, x_bytes = (uint32_t(T) * 128u + 1023u) & ~1023u;
    const uint32_t stage_bytes = a_bytes + x_bytes + kSearchWTile + kSearchITile;   // dW tiles | X | W | W_int
    const uint32_t bar0 = smem_u32(&bars[0]);
    volatile int *abort_flag = &abort_s;

    for (int v = tid; v < p.lut_size; v += kSearchBlock) {
        uint32_t word = 0x80808080u;   // candidates the block does not have: step 0
        for (int c = 0; c < ncand; ++c) {
            const int step = int(p.lut[size_t(cand0 + c) * 64 + v]) - v;   // the table holds integers
            word = (word & ~(0xffu << (8 * c))) | (uint32_t(128 + step) << (8 * c));
        }
        step_s[v] = word;
    }
    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        mbar_init(bar0 + 16, 1);
        mbar_init(bar0 + 24, 1);
        mbar_init(bar0 + 32, 1);
        for (int i = 5; i < 9; ++i) mbar_init(bar0 + 8 * i, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {   // one warp allocates the accumulators' columns of tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(uint32_t(p.tmem_cols)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    // instruction descriptor: fp32 accumulate, fp16 A and B, both K-major, N = T, M = 128
    const uint32_t idesc = (1u << 4) | (uint32_t(T >> 3) << 17) | (uint32_t(kSearchRows >> 4) << 24);

    const int ktiles = p.K / kSearchKTile;
    bool alive = true;
    if (warp == kSearchThreads / 32) {
        // ---- the issuing warp: per slice, wait until the stage is full, issue the slice's MMAs, hand the stage back ----
        for (int kt = 0; kt < ktiles && alive; ++kt) {
            const int s = kt & 1;
            if (!search_wait(bar0 + 24 + 8 * s, uint32_t((kt >> 1) & 1), abort_flag, 3) ||
                !search_wait(bar0 + 40 + 8 * s, uint32_t((kt >> 1) & 1), abort_flag, 4)) {
                alive = false;
                break;
            }
            if (lane == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t st_base = base + uint32_t(s) * stage_bytes;
                const uint64_t bdesc = smem_desc_sw128(st_base + a_bytes);
                for (int c = 0; c < ncand; ++c) {
                    const uint64_t adesc = smem_desc_sw128(st_base + uint32_t(c) * kSearchATile);
                    const uint32_t d = tmem_base + uint32_t(c * T);
#pragma unroll
                    for (int j = 0; j < kSearchKTile / 16; ++j)   // 16 weights = 32 bytes further along the row
                        umma_f16(d, adesc + uint64_t(2 * j), bdesc + uint64_t(2 * j), idesc, (kt > 0 || j > 0) ? 1u : 0u);
                }
                umma_commit(bar0 + 8 * s);
                if (kt == ktiles - 1) umma_commit(bar0 + 16);
            }
            __syncwarp();
        }
    } else {
        // this thread's part of a dW tile: row r of the block, 16 consecutive weights (2 pieces of 16 bytes)
        const int r = tid >> 2, quart = tid & 3;
        const int row0 = blockIdx.x * kSearchRows;
        const int n = row0 + r;
        const bool row_ok = n < p.N;
        const uint32_t a_row_off = uint32_t(r) * 128u;
        const uint32_t step_u32 = smem_u32(step_s);
        // W's slice lands with the 128-byte swizzle (16-byte piece ^ row & 7: a warp's loads then spread over
        // all banks), W_int's as it is
        const uint32_t w_off0 = a_bytes + x_bytes + uint32_t(r) * 128u + uint32_t(((2 * quart) ^ (r & 7)) << 4);
        const uint32_t w_off1 = a_bytes + x_bytes + uint32_t(r) * 128u + uint32_t(((2 * quart + 1) ^ (r & 7)) << 4);
        const uint32_t i_off = a_bytes + x_bytes + kSearchWTile + uint32_t(r) * 64u + uint32_t(quart << 4);

        // scale and offset of (row, scaling unit): loaded one slice before the unit starts (rows beyond N keep 0)
        const int slices_per_unit = p.L / kSearchKTile;
        const size_t s_at = size_t(blockIdx.z) * p.scale_stride + size_t(row_ok ? n : 0) * p.G;
        const __half *srow = p.S + s_at, *brow = p.qbias + s_at;
        const int irow0 = int(blockIdx.z) * p.N + row0;   // W_int of the scale factors: one matrix of gridDim.z * N rows
        __half s_next = __float2half_rn(0.f), b_next = s_next;
        if (row_ok) s_next = __ldg(srow), b_next = __ldg(brow);
        float Sf = 0.f, qb = 0.f;
        __half Sh = s_next;
        int unit = 0, left = 0;   // slices left in the current scaling unit

        // slices of X, W and W_int travel by tensor-map copies that one thread starts: W and W_int one slice ahead
        // of their use, X as soon as the tensor cores have let go of the stage
        int x_started = -1, w_started = -1;
        if (tid == 0) {
            mbar_expect_tx(bar0 + 56, kSearchWTile + kSearchITile);
            tma_box_2d(base + a_bytes + x_bytes, &wmap, 0, row0, bar0 + 56);
            tma_box_2d(base + a_bytes + x_bytes + kSearchWTile, &imap, 0, irow0, bar0 + 56);
            w_started = 0;
        }

        for (int kt = 0; kt < ktiles && alive; ++kt) {
            const int s = kt & 1;
            const uint32_t st_base = base + uint32_t(s) * stage_bytes;
            // the MMAs that read this stage two slices ago must be complete before it is overwritten, and this slice
            // of W must have landed (every thread takes the same decision: a wait that gives up must not split the
            // block at a barrier)
            bool ok = kt < 2 || search_wait(bar0 + 8 * s, uint32_t(((kt >> 1) - 1) & 1), abort_flag, 1);
            ok = ok && search_wait(bar0 + 56 + 8 * s, uint32_t((kt >> 1) & 1), abort_flag, 5);
            if (!formers_all(ok)) {
                alive = false;
                break;
            }
            if (tid == 0) {
                mbar_expect_tx(bar0 + 40 + 8 * s, uint32_t(T) * 128u);
                tma_box_2d(st_base + a_bytes, &xmap, kt * kSearchKTile, 0, bar0 + 40 + 8 * s);
                x_started = kt;
                if (kt + 1 < ktiles) {   // the other stage's W was last read one slice ago, before that slice's barrier
                    const uint32_t other = base + uint32_t(s ^ 1) * stage_bytes + a_bytes + x_bytes;
                    mbar_expect_tx(bar0 + 56 + 8 * (s ^ 1), kSearchWTile + kSearchITile);
                    tma_box_2d(other, &wmap, (kt + 1) * kSearchKTile, row0, bar0 + 56 + 8 * (s ^ 1));
                    tma_box_2d(other + kSearchWTile, &imap, (kt + 1) * kSearchKTile, irow0, bar0 + 56 + 8 * (s ^ 1));
                    w_started = kt + 1;
                }
            }

            uint4 wcur0, wcur1, icur;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(wcur0.x), "=r"(wcur0.y), "=r"(wcur0.z), "=r"(wcur0.w) : "r"(st_base + w_off0));
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(wcur1.x), "=r"(wcur1.y), "=r"(wcur1.z), "=r"(wcur1.w) : "r"(st_base + w_off1));
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(icur.x), "=r"(icur.y), "=r"(icur.z), "=r"(icur.w) : "r"(st_base + i_off));
            if (left == 0) {
                Sh = s_next, Sf = __half2float(s_next), qb = __half2float(b_next);
                left = slices_per_unit;
                ++unit;
                if (row_ok && unit < p.G) s_next = __ldg(srow + unit), b_next = __ldg(brow + unit);
            }
            --left;

            // dW_p = S lut_p[v] + qbias - W = S (lut_p[v] - v) + r with r = S v + qbias - W, the residual of step 1.
            // r: one fp32 fused multiply-add, rounded to fp16 once for all candidates.  Per candidate the step comes
            // out of the lookup's byte as the fp16 number 1024 + byte (bit pattern 0x6400 | byte), minus 1152; one
            // fp16 fused multiply-add on a pair of weights then is the operand as it is stored (rounded once).
            uint32_t resid[8];     // r of weights (2 j, 2 j + 1), fp16 pairs
            uint32_t at[16];       // shared-memory address of the word of W_int's value
            {
                const uint32_t w8[8] = {wcur0.x, wcur0.y, wcur0.z, wcur0.w, wcur1.x, wcur1.y, wcur1.z, wcur1.w};
                const uint32_t i4[4] = {icur.x, icur.y, icur.z, icur.w};
    #pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w8[j]));
                    const float v0 = float((i4[j >> 1] >> (16 * (j & 1))) & 0xffu);
                    const float v1 = float((i4[j >> 1] >> (16 * (j & 1) + 8)) & 0xffu);
                    const __half2 h = __floats2half2_rn(fmaf(Sf, v0, qb - f.x), fmaf(Sf, v1, qb - f.y));
                    resid[j] = *reinterpret_cast<const uint32_t *>(&h);
                }
    #pragma unroll
                for (int j = 0; j < 16; ++j) at[j] = step_u32 + (((i4[j >> 2] >> (8 * (j & 3))) & 0xffu) << 2);
            }
            const __half2 S2 = __half2half2(Sh);
            const __half2 bias2 = __half2half2(__float2half_rn(-1152.f));
            // (rows beyond N: W reads as zeros and the scale and offset are 0, so dW = 0 whatever W_int holds there --
            // zeros, or the next scale factor's first rows)
    #pragma unroll
            for (int i = 0; i < 2; ++i) {
                uint32_t e[8];   // the words of weights 8 i .. 8 i + 7
    #pragma unroll
                for (int j = 0; j < 8; ++j) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(e[j]) : "r"(at[8 * i + j]));
                uint32_t pair01[4], pair23[4];   // bytes: candidates (0, 1) resp. (2, 3) of weights (2 j, 2 j + 1)
    #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    pair01[j] = __byte_perm(e[2 * j], e[2 * j + 1], 0x5140u);
                    pair23[j] = __byte_perm(e[2 * j], e[2 * j + 1], 0x7362u);
                }
                const int piece = 2 * quart + i;
                const uint32_t dst = st_base + a_row_off + uint32_t((piece ^ (r & 7)) << 4);
                static_for<0, kSearchMaxCand>([&](auto C) {
                    constexpr int c = decltype(C)::value;
                    if (c < ncand) {
                        uint32_t packed[4];
    #pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t raw = __byte_perm(c < 2 ? pair01[j] : pair23[j], 0x64646464u, (c & 1) ? 0x4342u : 0x4140u);
                            const __half2 step = __hadd2(*reinterpret_cast<const __half2 *>(&raw), bias2);
                            const __half2 h = __hfma2(S2, step, *reinterpret_cast<const __half2 *>(&resid[4 * i + j]));
                            packed[j] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + uint32_t(c) * kSearchATile), "r"(packed[0]), "r"(packed[1]), "r"(packed[2]), "r"(packed[3]) : "memory");
                    }
                });
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tiles are read by the tensor cores' proxy
            named_barrier(1, kSearchThreads);                 // every forming thread's part of the stage is written and fenced
            if (tid == 0) mbar_arrive(bar0 + 24 + 8 * s);     // the stage is full
        }
        if (tid == 0 && !alive) {   // giving up: the copies that were started still land in this block's shared memory
            for (int j = x_started; j >= 0 && j > x_started - 2; --j) search_drain(bar0 + 40 + 8 * (j & 1), uint32_t((j >> 1) & 1));
            for (int j = w_started; j >= 0 && j > w_started - 2; --j) search_drain(bar0 + 56 + 8 * (j & 1), uint32_t((j >> 1) & 1));
        }

    }

    // ---- the accumulators are complete: every row's squared outputs ------------------------------------
    alive = __syncthreads_and((alive && search_wait(bar0 + 16, 0u, abort_flag, 2)) ? 1 : 0) != 0;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int quarter = warp & 3, colpart = warp >> 2;   // a warp reads the 32 lanes of its quarter, every fourth piece of 16 columns
    if (alive && warp < kSearchThreads / 32) {
        for (int c = 0; c < ncand; ++c) {
            float sum = 0.f;
            for (int ch = colpart; ch < T / 16; ch += 4) {
                uint32_t v[16];
                const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(c * T + ch * 16);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                      "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float e = __uint_as_float(v[j]);
                    sum = fmaf(e, e, sum);
                }
            }
            part[colpart][c][quarter * 32 + lane] = sum;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (alive && tid < kSearchRows) {
        const int row = blockIdx.x * kSearchRows + tid;
        if (row < p.N)
            for (int c = 0; c < ncand; ++c) {
                float *out = p.err_rows + (size_t(blockIdx.z) * p.P + size_t(cand0 + c)) * p.N + row;
                const float sum = (part[0][c][tid] + part[1][c][tid]) + (part[2][c][tid] + part[3][c][tid]);
                *out = p.accumulate ? *out + sum : sum;   // pieces of tokens run one after the other on the stream
            }
    }
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(p.tmem_cols)) : "memory");
    }
}

// err[c] = sum over rows of err_rows[c][.] in a fixed order (fp64), one block per candidate
__global__ void __launch_bounds__(256) search_sum_kernel(const float *__restrict__ err_rows, int N, double *__restrict__ err)
{
    __shared__ double sh[256];
    const float *src = err_rows + size_t(blockIdx.x) * N;
    double s = 0.0;
    for (int i = threadIdx.x; i < N; i += 256) s += double(src[i]);
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) err[blockIdx.x] = sh[0];
}

// the first candidate, in order, whose error is below all earlier ones
__global__ void search_argmin_kernel(const double *__restrict__ err, int count, int P, int *__restrict__ best)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int at = 0;
    double lowest = err[0];
    for (int i = 1; i < count; ++i)
        if (err[i] < lowest) lowest = err[i], at = i;
    best[0] = at / P;
    best[1] = at % P;
}

int search_cand_per_block(int T)
{
    int c = 512 / T;
    return c > kSearchMaxCand ? kSearchMaxCand : c;
}

// two stages of (dW tiles | X | W | W_int), each part a multiple of 1024 bytes, + room to align the first
size_t search_smem_bytes(int T)
{
    const size_t x_bytes = (size_t(T) * 128 + 1023) / 1024 * 1024;
    return 2 * (size_t(search_cand_per_block(T)) * kSearchATile + x_bytes + kSearchWTile + kSearchITile) + 1024;
}

// Tensor map of a row-major matrix [rows][cols] for boxes of 64 columns x box_rows rows.  The encoder is a
// driver function; the runtime hands out its address, so the library links against the runtime only.
static cudaError_t search_tensor_map(CUtensorMap *map, const void *ptr, bool bytes, uint64_t rows, uint64_t cols, uint32_t box_rows,
                                     bool swizzle)
{
    using Encode = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Encode encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
        const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found);
        if (e != cudaSuccess) return e;
        if (found != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<Encode>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * (bytes ? 1u : 2u)};
    const cuuint32_t box[2] = {uint32_t(kSearchKTile), box_rows};
    const cuuint32_t steps[2] = {1u, 1u};
    const CUresult r = encode(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims,
                              strides, box, steps, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t launch_search_errors(const uint16_t *W, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias, size_t scale_stride,
                                 const uint16_t *X, int N, int K, int group, int T, int n_bits, const float *lut_dev /*[P][64]*/, int P,
                                 int scales, float *err_rows /*[scales][P][N]*/, double *err /*[scales][P]*/, cudaStream_t st)
{
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    SearchParams p = {};
    p.W = reinterpret_cast<const __half *>(W), p.w_int = w_int;
    p.S = reinterpret_cast<const __half *>(S), p.qbias = reinterpret_cast<const __half *>(qbias), p.scale_stride = scale_stride;
    p.X = reinterpret_cast<const __half *>(X), p.err_rows = err_rows;
    p.N = N, p.K = K, p.L = group == 0 ? K : group, p.G = K / p.L, p.P = P;
    p.lut_size = 1 << n_bits;
    p.lut = lut_dev;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        size_t most = 0;
        for (int t = 16; t <= kSearchMaxT; t += 16) most = search_smem_bytes(t) > most ? search_smem_bytes(t) : most;
        e = cudaFuncSetAttribute(search_error_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(most));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    // the slices of W (the block's 128 rows; rows beyond N read as zeros) and W_int (the scale factors' matrices as one
    // of scales * N rows)
    CUtensorMap xmap, wmap, imap;
    if ((e = search_tensor_map(&wmap, W, false, uint64_t(N), uint64_t(K), uint32_t(kSearchRows), true)) != cudaSuccess) return e;
    if ((e = search_tensor_map(&imap, w_int, true, uint64_t(scales) * uint64_t(N), uint64_t(K), uint32_t(kSearchRows), false)) != cudaSuccess) return e;
    const unsigned row_tiles = unsigned((N + kSearchRows - 1) / kSearchRows);
    // the error is a sum over tokens: pieces of at most 256 tokens, one launch each, the later ones adding to err_rows
    // (pieces of about equal size, multiples of 16)
    const int pieces = (T + kSearchMaxT - 1) / kSearchMaxT, piece = ((T + pieces - 1) / pieces + 15) / 16 * 16;
    for (int t0 = 0; t0 < T; t0 += piece) {
        const int Tp = T - t0 < piece ? T - t0 : piece;
        p.X = reinterpret_cast<const __half *>(X) + size_t(t0) * K;
        p.T = Tp, p.accumulate = t0 > 0 ? 1 : 0;
        p.cand_per_block = search_cand_per_block(Tp);
        int cols = 32;
        while (cols < p.cand_per_block * Tp) cols *= 2;
        p.tmem_cols = cols;
        if ((e = search_tensor_map(&xmap, p.X, false, uint64_t(Tp), uint64_t(K), uint32_t(Tp), true)) != cudaSuccess) return e;   // all rows of the piece
        const unsigned groups = unsigned((P + p.cand_per_block - 1) / p.cand_per_block);
        search_error_kernel<<<dim3(row_tiles, groups, unsigned(scales)), kSearchBlock, search_smem_bytes(Tp), st>>>(p, xmap, wmap, imap);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    search_sum_kernel<<<unsigned(P) * unsigned(scales), 256, 0, st>>>(err_rows, N, err);
    return cudaGetLastError();
}

cudaError_t launch_search_argmin(const double *err, int count, int P, int *best, cudaStream_t st)
{
    search_argmin_kernel<<<1, 32, 0, st>>>(err, count, P, best);
    return cudaGetLastError();
}

cudaError_t search_status_take(int *status)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_search_status, sizeof(int));
    if (e != cudaSuccess) return e;
    if (v != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbol(g_search_status, &zero, sizeof(int));
    }
    *status = v;
    return e;
}

}  // namespace bcq

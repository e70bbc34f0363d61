// Lookup-table BCQ GEMV (batch 1, tiled layout, group 128) for sm_100a.
//
//   y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )          (Eq. bcw + Eq. fuse_step3)
//
// Per 512-wide window of K the block builds, in shared memory, all 2^8 signed sums of every
// 8-activation chunk; packed weight bytes index those tables directly.  One block per SM, three
// kinds of warps:
//
//   builders  (warps 0-2)   convert the block's slice of x to fp32 and build the window tables,
//                           one window ahead of the consumers (two 64 KB tables, double buffered);
//   producer  (warp 3)      one thread feeds a ring of shared-memory slots with bulk async copies
//                           (cp.async.bulk, completion on an mbarrier): per (window, row unit) one
//                           slot = one tile = q*512 B of plane bytes + the unit's alphas and offsets;
//   consumers (warps 4-19)  copy a filled slot into registers, hand the slot back, look every
//                           weight byte up in the window table and accumulate in fp32.
//
// Table layout: word address of (entry e, chunk c) = e*64 + (c&1)*32 + (c>>1).  Lane l = 8 g + j
// of a consumer warp handles row j of a unit and the g-th group of 128 weights of the window; it
// walks the group's 16 chunks skewed by 2 j, so at every step the 32 lanes look up 32 different
// chunk columns -- 32 distinct banks whatever the weight bytes are -- and a lane needs only its
// own (row, group) scales.  The tables sit at shared-window addresses that are
// multiples of 64 KB and an entry is 256 B apart from the next, so ONE byte-permute builds the
// complete address (byte 1 <- weight byte, bytes 0,2,3 <- table address + 4*bank): a lookup is
// PRMT + LDS.  The memory before and after the tables (99 KB together) holds x, the barriers and
// the slot ring.
//
// Every wait on an mbarrier is bounded; if one runs out the block sets an abort flag and a
// device status word, stops waiting, drains its own copies and returns (see lut_status_take).
#include <type_traits>

#include "bcq_internal.cuh"

namespace bcq {

constexpr int kBuilderWarps = 3;
constexpr int kBuilderThreads = kBuilderWarps * 32;
constexpr int kProducerWarp = kBuilderWarps;
constexpr int kFirstConsumerWarp = kBuilderWarps + 1;
constexpr int kConsumerThreads = kLutWarps * 32;
constexpr int kLutThreads = (kBuilderWarps + 1 + kLutWarps) * 32;  // 640
constexpr int kTableBytes = 256 * 64 * 4;                          // 65536
constexpr int kLutSmemBytes = 232448;                              // 227 KB: the per-block opt-in maximum
constexpr int kMaxSlots = 48;
constexpr int kMinSlots = kLutWarps;   // one slot per consumer warp at least
constexpr int kXBytes = kMaxWindowsPerBlock * kWindow * 4;
constexpr int kBarrierBytes = 1024;
constexpr int kFixedBytes = kXBytes + kBarrierBytes;
constexpr int kProducerIdleLimit = 1 << 21;   // polling rounds without progress before the producer gives up
constexpr int kSpinLimit = 1 << 20;   // tries per wait (each try blocks for a short, hardware-defined time)

static_assert(2 * kFixedBytes <= kLutSmemBytes - 2 * kTableBytes, "x + barriers must fit before or after the tables");

__device__ int g_lut_status = 0;  // 0, or the code of the wait that ran out (sticky until taken)

#ifdef BCQ_TRACE
// Development aid (not compiled into the product): per-block event times in ns.
__device__ unsigned long long g_trace[1024][16];
__device__ __forceinline__ unsigned long long gtime()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define TRACE(slot) do { if (blockIdx.x < 1024) g_trace[blockIdx.x][slot] = gtime(); } while (0)
#define TRACE_ADD(slot, v) do { if (blockIdx.x < 1024) g_trace[blockIdx.x][slot] += (v); } while (0)
#else
#define TRACE(slot) do { } while (0)
#define TRACE_ADD(slot, v) do { } while (0)
#endif

template <int Q>
struct Slot {
    static constexpr int kPlaneBytes = Q * 512;
    static constexpr int kAlphaBytes = Q * 64;
    static constexpr int kOffsetBytes = 64;
    static constexpr int kBytes = kPlaneBytes + kAlphaBytes + kOffsetBytes;
};

struct LutParams {
    const uint8_t *tiles;  // tiled operand: per (window, unit) planes, alphas, offsets
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

// ---- mbarrier / bulk-copy primitives ------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)   // never blocks
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the block is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int code)
{
    for (int it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;   // sleeps in hardware until the phase completes or a short time-out
        if ((it & 15) == 15 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(&g_lut_status, code);
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// table lookup: the address register already holds the complete shared-window address
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
// [j][quad = 8s + lq][k], so that one 128-bit load gives activation j of the four chunks of a build
// item and the 16 quads a warp reads at once are 256 contiguous bytes (no bank conflicts).
__device__ __forceinline__ int xs_index(int kk)
{
    const int l = kk >> 4, s = (kk >> 3) & 1, j = kk & 7;
    return ((j * 16 + s * 8 + (l >> 2)) << 2) + (l & 3);
}

// Table build.  A thread owns one quad of chunks (slot s = quad >> 3, lanes 4*(quad&7) .. +3): it
// reads the quad's 8 x 4 activations once, then for each of its values of the entry bits 3..7
// (hi = hi0, hi0 + hi_step, ... < 32) walks the 8 entries sharing those bits in Gray-code order:
// one packed FMA per entry and chunk pair, one 128-bit conflict-free store per entry.
__device__ __forceinline__ void build_quad(unsigned char *table, const float *xs_w, int quad, int hi0, int hi_step)
{
    const float4 *xq = reinterpret_cast<const float4 *>(xs_w) + quad;  // xq[16 j] = activation j of the 4 chunks
    f32x2 x01[8], x23[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float4 v = xq[16 * j];
        x01[j] = pack2(v.x, v.y);
        x23[j] = pack2(v.z, v.w);
    }
    const f32x2 m1 = pack2(-1.f, -1.f), p2 = pack2(2.f, 2.f), m2 = pack2(-2.f, -2.f);
    f32x2 low01 = pack2(0.f, 0.f), low23 = low01;   // -(x0 + x1 + x2): entry bits 0..2 clear
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        low01 = fma2(m1, x01[j], low01);
        low23 = fma2(m1, x23[j], low23);
    }
    for (int hi = hi0; hi < 32; hi += hi_step) {
        f32x2 c01 = low01, c23 = low23;
#pragma unroll
        for (int j = 3; j < 8; ++j) {
            const float sg = ((hi >> (j - 3)) & 1) ? 1.f : -1.f;
            const f32x2 s2 = pack2(sg, sg);
            c01 = fma2(s2, x01[j], c01);
            c23 = fma2(s2, x23[j], c23);
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
}

enum { kWaitEmpty = 1, kWaitFull = 2, kWaitTableReady = 3, kWaitTableFree = 4, kWaitDrain = 5, kTooFewSlots = 6 };

template <int Q>
__global__ void __launch_bounds__(kLutThreads, 1) lut_gemv_kernel(const LutParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    using SL = Slot<Q>;
    constexpr int UMAX = kLutUnitsPerWarp;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int rbi = blockIdx.x % p.row_blocks, ks = blockIdx.x / p.row_blocks;
    const int u0 = int((long long)rbi * p.U / p.row_blocks), u1 = int((long long)(rbi + 1) * p.U / p.row_blocks);
    const int w0 = int((long long)ks * p.W / p.k_splits), w1 = int((long long)(ks + 1) * p.W / p.k_splits);
    const int V = u1 - u0;       // row units of this block
    const int nwin = w1 - w0;    // windows of this block

    // ---- carve shared memory: [front | table 0 | table 1 | back] --------------------------------
    const uint32_t base = smem_u32(smem);
    const uint32_t tab0 = (base + 0xFFFFu) & ~0xFFFFu;  // shared-window address of table 0
    const int front = int(tab0 - base), back = kLutSmemBytes - front - 2 * kTableBytes;
    unsigned char *tables = smem + front;
    unsigned char *after = tables + 2 * kTableBytes;
    const bool fixed_in_back = back >= kFixedBytes;
    unsigned char *fixed = fixed_in_back ? after : smem;
    unsigned char *ring_a = fixed_in_back ? smem : smem + kFixedBytes;
    unsigned char *ring_b = fixed_in_back ? after + kFixedBytes : after;
    const int n_a = (fixed_in_back ? front : front - kFixedBytes) / SL::kBytes;
    const int n_b = (fixed_in_back ? back - kFixedBytes : back) / SL::kBytes;
    const int NS = min(n_a + n_b, kMaxSlots);
    const int D = min(NS / kLutWarps, 3);   // ring slots per consumer warp
    auto slot_ptr = [&](int s) -> unsigned char * { return s < n_a ? ring_a + s * SL::kBytes : ring_b + (s - n_a) * SL::kBytes; };

    float *xs = reinterpret_cast<float *>(fixed);
    const uint32_t bars = smem_u32(fixed + kXBytes);
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kMaxSlots;
    const uint32_t bar_tab_ready = bars + 16 * kMaxSlots, bar_tab_free = bar_tab_ready + 16;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(fixed + kXBytes + 16 * kMaxSlots + 32);
    int *s_last = const_cast<int *>(abort_flag) + 1;

    if (tid == 0) {
        TRACE(0);
#ifdef BCQ_TRACE
        g_trace[blockIdx.x % 1024][13] = 0; g_trace[blockIdx.x % 1024][14] = 0;
#endif
        for (int s = 0; s < kMaxSlots; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_tab_ready + 8 * b, kBuilderThreads);
            mbar_init(bar_tab_free + 8 * b, kLutWarps);
        }
        *abort_flag = (NS < kMinSlots) ? 1 : 0;
        if (NS < kMinSlots) atomicExch(&g_lut_status, int(kTooFewSlots));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) TRACE(1);

    // =============================================================================================
    if (warp != kProducerWarp) {
        // ---- start-up, all warps but the producer: x slice fp16 -> fp32 (permuted for the build)
        //      and the first window's table ----------------------------------------------------------
        constexpr int kStartThreads = kLutThreads - 32;
        const int sid = warp < kProducerWarp ? tid : tid - 32;
        static_assert(kMaxWindowsPerBlock * (kWindow / 8) <= kStartThreads, "one 8-activation chunk per thread");
        if (sid < nwin * (kWindow / 8)) {   // one chunk of 8 activations per thread, one 128-bit load
            const uint4 raw = *reinterpret_cast<const uint4 *>(p.x + size_t(w0) * kWindow + size_t(sid) * 8);
            const __half *h = reinterpret_cast<const __half *>(&raw);
            float *dst = xs + (sid >> 6) * kWindow + xs_index((sid & 63) * 8);
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[j * 64] = __half2float(h[j]);   // xs_index advances by 64 per activation
        }
        named_barrier(1, kStartThreads);
        if (sid == 0) TRACE(2);
        if (sid < 512) build_quad(tables, xs, sid & 15, sid >> 4, 32);
        named_barrier(1, kStartThreads);
        if (sid == 0) TRACE(3);
    }

    if (warp < kBuilderWarps) {
        // ---- builders: one table per window, one window ahead of the consumers ----------------------
        mbar_arrive(bar_tab_ready);   // window 0 was built by everybody above
        for (int wi = 1; wi < nwin; ++wi) {
            const int b = wi & 1, use = wi >> 1;
            if (use > 0 && !mbar_wait(bar_tab_free + 8 * b, (use - 1) & 1, abort_flag, kWaitTableFree)) break;
            unsigned char *table = tables + b * kTableBytes;
            build_quad(table, xs + wi * kWindow, tid & 15, tid >> 4, kBuilderThreads / 16);
            mbar_arrive(bar_tab_ready + 8 * b);
        }
        return;
    }

    if (warp == kProducerWarp) {
        // ---- producer: one thread keeps the slot ring full ---------------------------------------
        // Lane c feeds consumer warp c: slots c and c + 16 (+ 32) belong to that warp alone, so a
        // slot's fills are consumed by one warp, in order, and a wait can never be satisfied by
        // an older phase of the barrier.
        if (lane < kLutWarps && !*abort_flag) {
            const int c = lane;
            const int mine = (V - c + kLutWarps - 1) / kLutWarps;  // units of warp c per window
            int remaining = mine * nwin, t_in_win = 0, wi = 0, idle = 0;
            size_t tile = size_t(w0) * p.U + u0 + c;
            int d = 0, k = 0, last_s = -1, last_par = 0, prev_s = -1, prev_par = 0, pprev_s = -1, pprev_par = 0;
            // The 16 lanes stay together in one polling loop and never block on a barrier, so
            // each refills its warp's slot as soon as that slot is handed back.
            while (true) {
                bool issued = false;
                if (remaining > 0) {
                    const int s = c + kLutWarps * d;
                    if (k == 0 || mbar_test_wait(bar_empty + 8 * s, (k - 1) & 1)) {
                        const uint32_t dst = smem_u32(slot_ptr(s)), full = bar_full + 8 * s;
                        mbar_expect_tx(full, SL::kBytes);
                        bulk_g2s(dst, p.tiles + tile * SL::kBytes, SL::kBytes, full);   // planes + alphas + offsets
                        pprev_s = prev_s, pprev_par = prev_par, prev_s = last_s, prev_par = last_par;
                        last_s = s, last_par = k & 1;
                        if (++d == D) {
                            d = 0;
                            ++k;
                        }
                        tile += kLutWarps;
                        if (++t_in_win == mine) {
                            t_in_win = 0;
                            ++wi;
                            tile = size_t(w0 + wi) * p.U + u0 + c;
                        }
                        --remaining;
                        issued = true;
                    }
                }
                if (__ballot_sync(0xFFFFu, remaining > 0) == 0) break;
                if (__any_sync(0xFFFFu, issued)) {
                    idle = 0;
                    continue;
                }
                __nanosleep(100);   // nothing to refill: leave the issue slots to the consumers
                if (++idle > kProducerIdleLimit || *abort_flag) {
                    if (idle > kProducerIdleLimit) {
                        *abort_flag = 1;
                        atomicExch(&g_lut_status, int(kWaitEmpty));
                    }
                    break;
                }
            }
            // See the last fill of each of this lane's (at most 3) slots land, with a bounded wait,
            // before the warp leaves: the block's shared memory must not be handed to another block
            // while copies into it are in flight, also when the consumers gave up.
            if (lane == 0) TRACE(12);
            const int ss[3] = {last_s, prev_s, pprev_s}, pp[3] = {last_par, prev_par, pprev_par};
#pragma unroll
            for (int q3 = 0; q3 < 3; ++q3) {
                if (ss[q3] < 0 || q3 >= D) continue;
                bool landed = false;
                for (int it = 0; it < kSpinLimit && !landed; ++it) landed = mbar_try_wait(bar_full + 8 * ss[q3], uint32_t(pp[q3]));
                if (!landed) atomicExch(&g_lut_status, int(kWaitDrain));
            }
        }
        return;
    }

    // =============================================================================================
    // ---- consumers ---------------------------------------------------------------------------------
    // Lane l = 8 g + j owns row 8u + j of every unit and the g-th group of 128 weights of every
    // window: its 16q bytes of a tile are the group's 16 chunks (skewed by 2 j, see the layout), so
    // it needs only its own q alphas and one offset per tile and keeps ONE accumulator per unit.
    const int cw = warp - kFirstConsumerWarp;   // 0..15
    const int ctid = tid - kFirstConsumerWarp * 32;
    const int g4 = lane >> 3, jr = lane & 7;
    float acc[UMAX];
#pragma unroll
    for (int t = 0; t < UMAX; ++t) acc[t] = 0.f;
    bool alive = !*abort_flag;
    int d = 0, k = 0;   // this warp's ring position: slot cw + 16 d, fill number k

    for (int wi = 0; wi < nwin && alive; ++wi) {
        const int b = wi & 1;
        if (!mbar_wait(bar_tab_ready + 8 * b, (wi >> 1) & 1, abort_flag, kWaitTableReady)) {
            alive = false;
            break;
        }
        if (ctid == 0 && wi == 0) TRACE(4);
        // Table address part of the lookups of step pair h: chunk 16 g + ((2h + 2j) mod 16) and the
        // next one share bank 8 g + ((h + j) mod 8); the odd chunk sits 128 bytes further.
        uint32_t off[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) off[h] = tab0 + uint32_t(b * kTableBytes + 4 * (8 * g4 + ((h + jr) & 7)));
        // sum of x over this lane's group: the all-ones entries of the group's 16 chunks
        float xsum = lds_f32<255 * 256>(off[0]) + lds_f32<255 * 256 + 128>(off[0]);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 4);

        static_for<0, UMAX>([&](auto T) {
            constexpr int t = decltype(T)::value;
            if (alive && cw + kLutWarps * t < V) {
                const int s = cw + kLutWarps * d;
#ifdef BCQ_TRACE
                const unsigned long long tw0 = gtime();
#endif
                const bool got = mbar_wait(bar_full + 8 * s, k & 1, abort_flag, kWaitFull);
#ifdef BCQ_TRACE
                if (ctid == 0) { TRACE_ADD(13, gtime() - tw0); TRACE_ADD(14, 1); if (wi == 0 && t == 0) TRACE(5); }
#endif
                if (!got) {
                    alive = false;
                } else {
                    // slot -> registers, then hand the slot back to the producer
                    const unsigned char *slot = slot_ptr(s);
                    uint32_t wbuf[4 * Q];
#pragma unroll
                    for (int j = 0; j < Q; ++j) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(slot + j * 512 + lane * 16);
                        wbuf[4 * j + 0] = v.x;
                        wbuf[4 * j + 1] = v.y;
                        wbuf[4 * j + 2] = v.z;
                        wbuf[4 * j + 3] = v.w;
                    }
                    __half sc[Q + 1];   // alpha_0 .. alpha_{q-1}, z of (row, group) = this lane
                    const unsigned char *sp = slot + SL::kPlaneBytes + lane * (2 * (Q + 1));
                    if constexpr (Q == 3) {
                        *reinterpret_cast<uint2 *>(sc) = *reinterpret_cast<const uint2 *>(sp);
                    } else if constexpr (Q == 1) {
                        *reinterpret_cast<uint32_t *>(sc) = *reinterpret_cast<const uint32_t *>(sp);
                    } else {
#pragma unroll
                        for (int i = 0; i <= Q; ++i) sc[i] = reinterpret_cast<const __half *>(sp)[i];
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * s);

                    float sum[Q][2];
#pragma unroll
                    for (int i = 0; i < Q; ++i) sum[i][0] = sum[i][1] = 0.f;
                    static_for<0, 16>([&](auto S) {
                        constexpr int st = decltype(S)::value;
                        static_for<0, Q>([&](auto I) {
                            constexpr int i = decltype(I)::value;
                            constexpr int pb = st * Q + i;
                            const uint32_t addr = __byte_perm(wbuf[pb >> 2], off[st >> 1], 0x7604 | ((pb & 3) << 4));
                            sum[i][st & 1] += (st & 1) ? lds_f32<128>(addr) : lds_f32<0>(addr);
                        });
                    });
                    float a = fmaf(__half2float(sc[Q]), xsum, acc[t]);
#pragma unroll
                    for (int i = 0; i < Q; ++i) a = fmaf(__half2float(sc[i]), sum[i][0] + sum[i][1], a);
                    acc[t] = a;
                }
                if (++d == D) {
                    d = 0;
                    ++k;
                }
            }
        });
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tab_free + 8 * b);
        if (ctid == 0 && wi < 4) TRACE(6 + wi);
    }

    // ---- a unit's row j is spread over the 4 lanes 8 g + j: add them up, lanes 0..7 store ---------
    float *partial = p.k_splits > 1 ? p.partial + size_t(ks) * p.N : nullptr;
#pragma unroll
    for (int t = 0; t < UMAX; ++t) {
        float v = acc[t];
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < 8 && cw + kLutWarps * t < V) {
            const int n = (u0 + cw + kLutWarps * t) * kUnitRows + lane;
            if (partial)
                partial[n] = v;
            else
                p.y[n] = __float2half_rn(v);
        }
    }

    if (ctid == 0) TRACE(10);
    // ---- split-K: the last block to arrive for this row block adds the partials in fixed order --
    if (p.k_splits > 1) {
        __threadfence();
        named_barrier(2, kConsumerThreads);
        if (ctid == 0) {
            const int old = atomicAdd(p.counters + rbi, 1);
            *s_last = (old == p.k_splits - 1);
        }
        named_barrier(2, kConsumerThreads);
        if (*s_last) {
            __threadfence();
            // fixed summation order (deterministic); the loads of 8 splits are issued together
            for (int n = u0 * kUnitRows + ctid; n < u1 * kUnitRows; n += kConsumerThreads) {
                float v = 0.f;
                for (int k0 = 0; k0 < p.k_splits; k0 += 8) {
                    float part[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        part[k] = (k0 + k < p.k_splits) ? __ldcg(p.partial + size_t(k0 + k) * p.N + n) : 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) v += part[k];
                }
                p.y[n] = __float2half_rn(v);
            }
            if (ctid == 0) p.counters[rbi] = 0;
        }
    }
    if (ctid == 0) TRACE(11);
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
    prm.tiles = static_cast<const uint8_t *>(packed);
    (void)alpha;
    (void)z;
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

#ifdef BCQ_TRACE
extern "C" int bcq_debug_read_trace(unsigned long long *host, int blocks)
{
    return int(cudaMemcpyFromSymbol(host, g_trace, size_t(blocks) * 16 * sizeof(unsigned long long)));
}
#endif

// Read and clear the device status word (synchronises with the device).
cudaError_t lut_status_take(int *status)
{
    int v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_lut_status, sizeof(int));
    if (e != cudaSuccess) return e;
    if (v != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbol(g_lut_status, &zero, sizeof(int));
    }
    *status = v;
    return e;
}

}  // namespace bcq

// Lookup-table BCQ GEMV for sm_100a: batch 1 (tiled layout, scales per group of 128 or per row), and a
// two-column variant for group 128.
//
//   y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )          (Eq. bcw + Eq. fuse_step3)
//
// Per 512-wide window of K the block builds, in shared memory, all 2^8 signed sums of every
// 8-activation chunk; packed weight bytes index those tables directly.  One block per SM, two
// kinds of warps:
//
//   builders  (warps 0-3)   build the window tables from x, one window ahead of the consumers
//                           (two tables, double buffered);
//   consumers (warps 4-27)  each owns a few shared-memory slots that it keeps filled with bulk
//                           async copies (cp.async.bulk, completion on an mbarrier), one slot =
//                           one tile = q*512 B of plane bytes + the unit's alphas and offsets of
//                           one (window, row unit).  A consumer waits for its next tile, copies
//                           it into registers, immediately re-uses the slot for the tile that
//                           many jobs ahead, then looks every weight byte up in the window table
//                           and accumulates in fp32.  (One warp can start only about 18 bulk
//                           copies per microsecond: the copies have to be issued by many warps.)
//
// Tables.  The sums are computed in fp32 and stored as fp16 (one rounding, relative 2^-11; the
// accumulation of the looked-up values stays fp32).  Halving the tables to 32 KB each is what
// leaves 140 KB of shared memory for tiles in flight -- the stream is otherwise bound by the DRAM
// latency.  Both tables share one 64 KB region at a shared-window address that is a multiple of
// 64 KB: entry e of table b, chunk c at byte  e*256 + b*128 + (c>>1)*4 + (c&1)*2.  Lane l = 8 g + j
// of a consumer warp handles row j of a unit and the g-th group of 128 weights of the window; it
// walks the group's 16 chunks skewed by 2 j, so at every step the 32 lanes address 32 different
// 4-byte columns -- 32 distinct banks whatever the weight bytes are -- and a lane needs only its
// own (row, group) scales.  With the 256-byte entry stride and the 64 KB alignment ONE byte-permute
// builds the complete address (byte 1 <- weight byte, bytes 0,2,3 <- table address + column): a
// lookup is PRMT + LDS.U16 + one mixed-precision add (fp32 += fp16).
//
// Two columns (NB = 2).  A lookup moves 2 bytes per lane, half of what the shared-memory pipe delivers
// per access; with two activation vectors the entry becomes 4 bytes -- the sums of (column 0, column 1)
// for the same chunk and index -- and one lookup feeds two adds.  Entry e (256 B) is then [even chunks:
// 32 words][odd chunks: 32 words]; all lanes of a warp are at chunks of one parity at any step, so they
// still read 32 different words.  Each table buffer fills a 64 KB region of its own.
//
// The kernel is launched with programmatic stream serialisation: it lets its dependents start as soon as
// it runs and waits for its own predecessor only before it touches x, the workspace or y; the packed
// weights are treated as constants that are complete before the launch.
//
// Every wait on an mbarrier is bounded; if one runs out the block sets an abort flag and a
// device status word, stops waiting, drains its own copies and returns (see lut_status_take).
#include "bcq_async.cuh"
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kBuilderWarps = 4;
constexpr int kBuilderThreads = kBuilderWarps * 32;
constexpr int kFirstConsumerWarp = kBuilderWarps;
constexpr int kConsumerThreads = kLutWarps * 32;
constexpr int kLutThreads = (kBuilderWarps + kLutWarps) * 32;      // 896
constexpr int kLutSmemBytes = 232448;                              // 227 KB: the per-block opt-in maximum
constexpr int kMaxSlotsPerWarp = 5;
constexpr int kMaxSlots = kLutWarps * kMaxSlotsPerWarp;
constexpr int kMinSlots = kLutWarps;   // one slot per consumer warp at least
constexpr int kFixedBytes = 2048;      // barriers and flags

static_assert(8 * kMaxSlots + 64 <= kFixedBytes, "barrier area");
static_assert(2 * kFixedBytes <= kLutSmemBytes - 2 * 65536, "barriers must fit before or after the tables");

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

// One tile = one ring slot.  GROUPED (group 128): planes + the tile's alphas and offsets;
// otherwise (one scale per row) the planes only, alphas and offsets live in their own arrays.
template <int Q, bool GROUPED>
struct Slot {
    static constexpr int kPlaneBytes = Q * 512;
    static constexpr int kBytes = kPlaneBytes + (GROUPED ? Q * 64 + 64 : 0);
};

struct LutParams {
    const uint8_t *tiles;  // tiled operand: per (window, unit) planes (+ alphas, offsets when grouped)
    const __half *alpha;   // per-row scales only: [u][i][r]
    const __half *z;       // per-row scales only: [u][r]
    const __half *x;
    __half *y;
    float *partial;  // [k_splits][N] when k_splits > 1
    int *counters;   // [row_blocks]
    int N, K, U, W;
    int row_blocks, k_splits;
};

// table lookup + accumulate: the address register already holds the complete shared-window
// address of an fp16 entry; acc (fp32) += entry, in one mixed-precision add
template <int OFF>
__device__ __forceinline__ void lut_add(float &acc, uint32_t addr)
{
    asm volatile(
        "{\n\t.reg .b16 h;\n\t"
        "ld.shared.b16 h, [%1+%2];\n\t"
        "add.rn.f32.f16 %0, h, %0;\n\t}"
        : "+f"(acc)
        : "r"(addr), "n"(OFF));
}
// the same for two columns at once: the 4-byte entry holds (column 0, column 1) as fp16
template <int OFF>
__device__ __forceinline__ void lut_add2(float &acc0, float &acc1, uint32_t addr)
{
    asm volatile(
        "{\n\t.reg .b16 l, h;\n\t.reg .b32 v;\n\t"
        "ld.shared.b32 v, [%2+%3];\n\t"
        "mov.b32 {l, h}, v;\n\t"
        "add.rn.f32.f16 %0, l, %0;\n\t"
        "add.rn.f32.f16 %1, h, %1;\n\t}"
        : "+f"(acc0), "+f"(acc1)
        : "r"(addr), "n"(OFF));
}
template <int OFF>
__device__ __forceinline__ uint32_t lds_b32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF));
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

// Table build.  A thread owns four consecutive chunks (quad cq: chunks 4cq .. 4cq+3, i.e. 32
// activations read straight from x): it converts them once, then for each of its values of the
// entry bits 3..7 (hi = hi0, hi0 + hi_step, ... < 32) walks the 8 entries sharing those bits in
// Gray-code order: one packed fp32 FMA per entry and chunk pair, the four sums rounded to fp16 and
// stored with one 64-bit store (16 quads = 128 contiguous bytes per entry: no bank conflicts).
// `table` points at entry 0 of the buffer being built.  Loading (load_quad) and building are separate
// so that a builder can have the next window's activations on their way while it waits for the buffer.
__device__ __forceinline__ void load_quad(const __half *xw, int cq, f32x2 (&x01)[8], f32x2 (&x23)[8])
{
    {
        float xf[4][8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(xw + 32 * cq + 8 * k);
            const __half2 *h2 = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __half22float2(h2[j]);
                xf[k][2 * j] = f.x;
                xf[k][2 * j + 1] = f.y;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            x01[j] = pack2(xf[0][j], xf[1][j]);
            x23[j] = pack2(xf[2][j], xf[3][j]);
        }
    }
}
__device__ __forceinline__ void build_quad(unsigned char *table, const f32x2 (&x01)[8], const f32x2 (&x23)[8], int cq, int hi0,
                                           int hi_step)
{
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
        unsigned char *dst = table + cq * 8 + hi * (8 * 256);
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
            const __half2 h01 = __floats2half2_rn(a.x, a.y), h23 = __floats2half2_rn(b.x, b.y);
            uint2 out;
            out.x = *reinterpret_cast<const uint32_t *>(&h01);
            out.y = *reinterpret_cast<const uint32_t *>(&h23);
            *reinterpret_cast<uint2 *>(dst + gray * 256) = out;
        });
    }
}

// Two columns.  Table entry e (256 B) = [even chunks: 32 words][odd chunks: 32 words], a word = the fp16
// sums of (column 0, column 1) for that chunk and entry.  A thread owns the chunk pair cp (chunks 2cp,
// 2cp + 1) of both columns: xa / xb hold activation j of the two chunks for column 0 / column 1.
__device__ __forceinline__ void load_pair(const __half *xw, size_t col_stride, int cp, f32x2 (&xa)[8], f32x2 (&xb)[8])
{
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const __half *src = xw + c * col_stride + 16 * cp;
        const uint4 r0 = *reinterpret_cast<const uint4 *>(src), r1 = *reinterpret_cast<const uint4 *>(src + 8);
        const __half2 *h0 = reinterpret_cast<const __half2 *>(&r0), *h1 = reinterpret_cast<const __half2 *>(&r1);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f0 = __half22float2(h0[j]), f1 = __half22float2(h1[j]);
            if (c == 0) {
                xa[2 * j] = pack2(f0.x, f1.x);
                xa[2 * j + 1] = pack2(f0.y, f1.y);
            } else {
                xb[2 * j] = pack2(f0.x, f1.x);
                xb[2 * j + 1] = pack2(f0.y, f1.y);
            }
        }
    }
}
__device__ __forceinline__ void build_pair(unsigned char *table, const f32x2 (&xa)[8], const f32x2 (&xb)[8], int cp, int hi0,
                                           int hi_step)
{
    const f32x2 m1 = pack2(-1.f, -1.f), p2 = pack2(2.f, 2.f), m2 = pack2(-2.f, -2.f);
    f32x2 lowa = pack2(0.f, 0.f), lowb = lowa;
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        lowa = fma2(m1, xa[j], lowa);
        lowb = fma2(m1, xb[j], lowb);
    }
    for (int hi = hi0; hi < 32; hi += hi_step) {
        f32x2 ca = lowa, cb = lowb;
#pragma unroll
        for (int j = 3; j < 8; ++j) {
            const float sg = ((hi >> (j - 3)) & 1) ? 1.f : -1.f;
            const f32x2 s2 = pack2(sg, sg);
            ca = fma2(s2, xa[j], ca);
            cb = fma2(s2, xb[j], cb);
        }
        unsigned char *dst = table + cp * 4 + hi * (8 * 256);
        static_for<0, 8>([&](auto step_c) {
            constexpr int step = decltype(step_c)::value;
            constexpr int gray = step ^ (step >> 1);
            if constexpr (step > 0) {
                constexpr int bit = (step & 1) ? 0 : ((step & 2) ? 1 : 2);
                constexpr bool on = (gray >> bit) & 1;
                ca = fma2(on ? p2 : m2, xa[bit], ca);
                cb = fma2(on ? p2 : m2, xb[bit], cb);
            }
            const float2 a = unpack2(ca), b = unpack2(cb);   // a: column 0 of chunks 2cp, 2cp+1; b: column 1
            const __half2 even = __floats2half2_rn(a.x, b.x), odd = __floats2half2_rn(a.y, b.y);
            *reinterpret_cast<uint32_t *>(dst + gray * 256) = *reinterpret_cast<const uint32_t *>(&even);
            *reinterpret_cast<uint32_t *>(dst + gray * 256 + 128) = *reinterpret_cast<const uint32_t *>(&odd);
        });
    }
}

enum { kWaitEmpty = 1, kWaitFull = 2, kWaitTableReady = 3, kWaitTableFree = 4, kWaitDrain = 5, kTooFewSlots = 6 };

// NB columns per launch: 1, or 2 (grouped scales only) with tables that hold both columns' sums side by
// side, so that one 4-byte lookup serves two products; each of the two table buffers then fills a
// 64 KB region of its own.
template <int Q, bool GROUPED, int NB>
__global__ void __launch_bounds__(kLutThreads, 1) lut_gemv_kernel(const LutParams p)
{
    static_assert(NB == 1 || (NB == 2 && GROUPED), "two columns need the scales inside the tiles");
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kTablesBytes = NB * 65536;
    using SL = Slot<Q, GROUPED>;
    constexpr int NACC = GROUPED ? 1 : Q;   // accumulators per unit and lane: the row's sum, or one per plane
    constexpr int UMAX = kLutUnitsPerWarp;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int rbi = blockIdx.x % p.row_blocks, ks = blockIdx.x / p.row_blocks;
    const int u0 = int((long long)rbi * p.U / p.row_blocks), u1 = int((long long)(rbi + 1) * p.U / p.row_blocks);
    const int w0 = int((long long)ks * p.W / p.k_splits), w1 = int((long long)(ks + 1) * p.W / p.k_splits);
    const int V = u1 - u0;       // row units of this block
    const int nwin = w1 - w0;    // windows of this block

    // ---- carve shared memory: [front | tables (64 KB, 64 KB aligned) | back] ----------------------
    const uint32_t base = smem_u32(smem);
    const uint32_t tab0 = (base + 0xFFFFu) & ~0xFFFFu;  // shared-window address of the tables
    const int front = int(tab0 - base), back = kLutSmemBytes - front - kTablesBytes;
    unsigned char *tables = smem + front;
    unsigned char *after = tables + kTablesBytes;
    const bool fixed_in_back = back >= kFixedBytes;
    unsigned char *fixed = fixed_in_back ? after : smem;
    unsigned char *ring_a = fixed_in_back ? smem : smem + kFixedBytes;
    unsigned char *ring_b = fixed_in_back ? after + kFixedBytes : after;
    const int n_a = (fixed_in_back ? front : front - kFixedBytes) / SL::kBytes;
    const int n_b = (fixed_in_back ? back - kFixedBytes : back) / SL::kBytes;
    const int NS = min(n_a + n_b, kMaxSlots);
    const int D = min(NS / kLutWarps, kMaxSlotsPerWarp);   // ring slots per consumer warp
    unsigned char *const ring_b0 = ring_b - n_a * SL::kBytes;   // so that slot s of either piece is at piece + s * kBytes
    auto slot_ptr = [&](int s) -> unsigned char * { return (s < n_a ? ring_a : ring_b0) + s * SL::kBytes; };

    const uint32_t bars = smem_u32(fixed);
    const uint32_t bar_full = bars;
    const uint32_t bar_tab_ready = bars + 8 * kMaxSlots, bar_tab_free = bar_tab_ready + 16;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(fixed + 8 * kMaxSlots + 32);
    int *s_last = const_cast<int *>(abort_flag) + 1;

    if (tid == 0) TRACE(0);
#ifdef BCQ_TRACE
    if (tid == 0) { g_trace[blockIdx.x % 1024][13] = 0; g_trace[blockIdx.x % 1024][14] = 0; g_trace[blockIdx.x % 1024][15] = 0; }
#endif
    if (warp == 0) {   // one warp initialises the barriers, a few each
        for (int s = lane; s < kMaxSlots; s += 32) mbar_init(bar_full + 8 * s, 1);
        if (lane < 2) {
            mbar_init(bar_tab_ready + 8 * lane, kBuilderThreads);
            mbar_init(bar_tab_free + 8 * lane, kLutWarps);
        }
        if (lane == 0) {
            *abort_flag = (NS < kMinSlots) ? 1 : 0;
            if (NS < kMinSlots) atomicExch(&g_lut_status, int(kTooFewSlots));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) TRACE(1);
    // Programmatic dependent launch: the next kernel in the stream may start taking SMs as soon as
    // this kernel's blocks leave them (it still waits, below, for its predecessor to finish before
    // it reads x or writes anything).  Without the launch attribute both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // =============================================================================================
    const __half *xblk = p.x + size_t(w0) * kWindow;   // this block's slice of x
    // ---- consumer warps: job bookkeeping, and the first D tiles of each warp on their way -----------
    // A warp's jobs, in the order it consumes them: windows outermost, its units innermost.  Lane 0
    // keeps D of them in flight; the issue cursor (iw, it) runs D jobs ahead of the consumption.
    const int cw = warp - kFirstConsumerWarp;   // 0 .. kLutWarps-1 for consumers, negative for builders
    const int mine = (cw >= 0 && V > cw) ? (V - cw + kLutWarps - 1) / kLutWarps : 0;   // units of this warp per window
    const int total_jobs = mine * nwin;
    int issued = 0, consumed = 0, it = 0;
    // the next tile to fetch: this warp's units of a window are kLutWarps tiles apart, then on to the next window
    const uint8_t *src = p.tiles + (size_t(w0) * p.U + u0 + (cw < 0 ? 0 : cw)) * SL::kBytes;
    const long long unit_step = (long long)kLutWarps * SL::kBytes;
    const long long window_step = ((long long)p.U - (long long)kLutWarps * mine) * SL::kBytes;
    auto issue_next = [&](int slot_d) {   // lane 0 of a consumer warp only
        if (issued < total_jobs) {
            const int s = cw + kLutWarps * slot_d;
            const uint32_t full = bar_full + 8 * s;
            mbar_expect_tx(full, SL::kBytes);
            bulk_g2s(smem_u32(slot_ptr(s)), src, SL::kBytes, full);   // planes + alphas + offsets
            ++issued;
            src += unit_step;
            if (++it == mine) {
                it = 0;
                src += window_step;
            }
        }
    };
    if (cw >= 0 && lane == 0 && !*abort_flag)
        for (int q5 = 0; q5 < D; ++q5) issue_next(q5);

    // The weights above are constants; everything from here on (x, partial sums, counters, y) may
    // depend on the previous kernel in the stream: wait for it to be complete and visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) TRACE(12);

    // ---- start-up: everybody builds the first window's table -------------------------------------
    if (tid < 512) {
        if constexpr (NB == 1) {
            f32x2 x01[8], x23[8];
            load_quad(xblk, tid & 15, x01, x23);
            build_quad(tables, x01, x23, tid & 15, tid >> 4, 32);
        } else {
            f32x2 xa[8], xb[8];
            load_pair(xblk, size_t(p.K), tid & 31, xa, xb);
            build_pair(tables, xa, xb, tid & 31, tid >> 5, 16);
        }
    }
    __syncthreads();
    if (tid == 0) TRACE(3);

    if (warp < kBuilderWarps) {
        // ---- builders: one table per window, one window ahead of the consumers ----------------------
        // Window 0 was built by everybody above (published by __syncthreads); the builders' fills of
        // buffer 0 are windows 2, 4, ... and of buffer 1 windows 1, 3, ...
        for (int wi = 1; wi < nwin; ++wi) {
            const int b = wi & 1, use = wi >> 1;
            f32x2 x01[8], x23[8];   // one column: a chunk quad; two columns: a chunk pair of each
            if constexpr (NB == 1)
                load_quad(xblk + wi * kWindow, tid & 15, x01, x23);   // in flight while waiting for the buffer
            else
                load_pair(xblk + wi * kWindow, size_t(p.K), tid & 31, x01, x23);
            if (use > 0 && !mbar_wait<true>(bar_tab_free + 8 * b, (use - 1) & 1, abort_flag, kWaitTableFree, &g_lut_status)) break;   // a long wait: nap longer
            if constexpr (NB == 1)
                build_quad(tables + b * 128, x01, x23, tid & 15, tid >> 4, kBuilderThreads / 16);
            else
                build_pair(tables + b * 65536, x01, x23, tid & 31, tid >> 5, kBuilderThreads / 32);
            mbar_arrive(bar_tab_ready + 8 * b);
        }
        return;
    }

    // =============================================================================================
    // ---- consumers ---------------------------------------------------------------------------------
    // Lane l = 8 g + j owns row 8u + j of every unit and the g-th group of 128 weights of every
    // window: its 16q bytes of a tile are the group's 16 chunks (skewed by 2 j, see the layout), so
    // it needs only its own q alphas and one offset per tile and keeps ONE accumulator per unit.
    const int ctid = tid - kFirstConsumerWarp * 32;
    const int g4 = lane >> 3, jr = lane & 7;
    float acc[UMAX][NACC], acc1[NB == 2 ? UMAX : 1];   // acc1: the second column
    float xacc = 0.f;   // per-row scales: sum of x over this lane's groups of all windows
#pragma unroll
    for (int t = 0; t < UMAX; ++t)
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[t][i] = 0.f;
#pragma unroll
    for (int t = 0; t < (NB == 2 ? UMAX : 1); ++t) acc1[t] = 0.f;
    bool alive = !*abort_flag;
    int d = 0, k = 0;   // this warp's ring position: slot cw + kLutWarps * d, fill number k


    for (int wi = 0; wi < nwin && alive; ++wi) {
        const int b = wi & 1;
#ifdef BCQ_TRACE
        const unsigned long long tt0 = gtime();
#endif
        if (wi > 0 && !mbar_wait(bar_tab_ready + 8 * b, ((wi >> 1) - (b == 0 ? 1 : 0)) & 1, abort_flag, kWaitTableReady, &g_lut_status)) {
            alive = false;
            break;
        }
#ifdef BCQ_TRACE
        if (ctid == 0 && wi == 0) TRACE(2);   // before the accumulating trace slots: those read global memory
        if (ctid == 0) TRACE_ADD(15, gtime() - tt0);
#endif
        if (ctid == 0 && wi == 0) TRACE(4);
        // Table address part of the lookups of step pair h: chunk 16 g + ((2h + 2j) mod 16) and the
        // next one share the 4-byte column 8 g + ((h + j) mod 8); the odd chunk is its upper half.
        uint32_t off[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) off[h] = tab0 + uint32_t(b * (NB == 1 ? 128 : 65536) + 4 * (8 * g4 + ((h + jr) & 7)));
        // sum of x over this lane's group: the all-ones entries of the group's 16 chunks (two per lane)
        float xsum, xsum1 = 0.f;
        if constexpr (NB == 1) {
            const uint32_t ones = lds_b32<255 * 256>(off[0]);
            const float2 ones_f = __half22float2(*reinterpret_cast<const __half2 *>(&ones));
            xsum = ones_f.x + ones_f.y;
        } else {
            const uint32_t even = lds_b32<255 * 256>(off[0]), odd = lds_b32<255 * 256 + 128>(off[0]);
            const float2 e = __half22float2(*reinterpret_cast<const __half2 *>(&even));
            const float2 o = __half22float2(*reinterpret_cast<const __half2 *>(&odd));
            xsum = e.x + o.x;
            xsum1 = e.y + o.y;
            xsum1 += __shfl_xor_sync(0xffffffffu, xsum1, 1);
            xsum1 += __shfl_xor_sync(0xffffffffu, xsum1, 2);
            xsum1 += __shfl_xor_sync(0xffffffffu, xsum1, 4);
        }
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 4);
        xacc += xsum;

        static_for<0, UMAX>([&](auto T) {
            constexpr int t = decltype(T)::value;
            if (alive && cw + kLutWarps * t < V) {
                const int s = cw + kLutWarps * d;
#ifdef BCQ_TRACE
                const unsigned long long tw0 = gtime();
#endif
                const bool got = mbar_wait(bar_full + 8 * s, k & 1, abort_flag, kWaitFull, &g_lut_status);
#ifdef BCQ_TRACE
                if (ctid == 0) { TRACE_ADD(13, gtime() - tw0); TRACE_ADD(14, 1); if (wi == 0 && t == 0) TRACE(5); }
#endif
                if (!got) {
                    alive = false;
                } else {
                    ++consumed;
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
                    [[maybe_unused]] __half sc[Q + 1];   // alpha_0 .. alpha_{q-1}, z of (row, group) = this lane
                    if constexpr (GROUPED) {
                        const unsigned char *sp = slot + SL::kPlaneBytes + lane * (2 * (Q + 1));
                        if constexpr (Q == 3) {
                            *reinterpret_cast<uint2 *>(sc) = *reinterpret_cast<const uint2 *>(sp);
                        } else if constexpr (Q == 1) {
                            *reinterpret_cast<uint32_t *>(sc) = *reinterpret_cast<const uint32_t *>(sp);
                        } else {
#pragma unroll
                            for (int i = 0; i <= Q; ++i) sc[i] = reinterpret_cast<const __half *>(sp)[i];
                        }
                    }
                    // The tile is in registers: order those reads before the next copy into the slot
                    // (generic-proxy reads, then an async-proxy write), then refill the slot.
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) issue_next(d);

                    float sum[Q][2], sum1[NB == 2 ? Q : 1][2];
#pragma unroll
                    for (int i = 0; i < Q; ++i) sum[i][0] = sum[i][1] = 0.f;
#pragma unroll
                    for (int i = 0; i < (NB == 2 ? Q : 1); ++i) sum1[i][0] = sum1[i][1] = 0.f;
                    static_for<0, 16>([&](auto S) {
                        constexpr int st = decltype(S)::value;
                        static_for<0, Q>([&](auto I) {
                            constexpr int i = decltype(I)::value;
                            constexpr int pb = i * 16 + st;
                            const uint32_t addr = __byte_perm(wbuf[pb >> 2], off[st >> 1], 0x7604 | ((pb & 3) << 4));
                            if constexpr (NB == 1)
                                lut_add<(st & 1) * 2>(sum[i][st & 1], addr);
                            else
                                lut_add2<(st & 1) * 128>(sum[i][st & 1], sum1[i][st & 1], addr);
                        });
                    });
                    if constexpr (GROUPED) {
                        float a = fmaf(__half2float(sc[Q]), xsum, acc[t][0]);
#pragma unroll
                        for (int i = 0; i < Q; ++i) a = fmaf(__half2float(sc[i]), sum[i][0] + sum[i][1], a);
                        acc[t][0] = a;
                        if constexpr (NB == 2) {
                            float a1 = fmaf(__half2float(sc[Q]), xsum1, acc1[t]);
#pragma unroll
                            for (int i = 0; i < Q; ++i) a1 = fmaf(__half2float(sc[i]), sum1[i][0] + sum1[i][1], a1);
                            acc1[t] = a1;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < Q; ++i) acc[t][i % NACC] += sum[i][0] + sum[i][1];
                    }
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

    // Gave up on a wait: copies this warp started may still be in flight.  See them land (bounded)
    // before the block's shared memory can be handed to another block.
    if (!alive && lane == 0) {
        for (int m = consumed; m < issued; ++m) {
            bool landed = false;
            for (int itr = 0; itr < kSpinLimit && !landed; ++itr)
                landed = mbar_try_wait(bar_full + 8 * (cw + kLutWarps * (m % D)), uint32_t((m / D) & 1));
            if (!landed) atomicExch(&g_lut_status, int(kWaitDrain));
        }
    }

    // ---- a unit's row j is spread over the 4 lanes 8 g + j: add them up, lanes 0..7 store ---------
    // (two columns: y and the partials of column 1 follow those of column 0, N elements further on)
    float *partial = p.k_splits > 1 ? p.partial + size_t(ks) * NB * p.N : nullptr;
#pragma unroll
    for (int t = 0; t < UMAX; ++t) {
        float v = acc[t][0];
        if constexpr (!GROUPED) {
            // one scale per row: apply the row's alphas and offset to the sums over this block's K range
            const int u = u0 + cw + kLutWarps * t;
            v = 0.f;
            if (u < u1) {
#pragma unroll
                for (int i = 0; i < Q; ++i) v = fmaf(__half2float(p.alpha[(size_t(u) * Q + i) * kUnitRows + jr]), acc[t][i % NACC], v);
                v = fmaf(__half2float(p.z[size_t(u) * kUnitRows + jr]), xacc, v);
            }
        }
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        float v1 = 0.f;
        if constexpr (NB == 2) {
            v1 = acc1[t];
            v1 += __shfl_xor_sync(0xffffffffu, v1, 8);
            v1 += __shfl_xor_sync(0xffffffffu, v1, 16);
        }
        if (lane < 8 && cw + kLutWarps * t < V) {
            const int n = (u0 + cw + kLutWarps * t) * kUnitRows + lane;
            if (partial)
                partial[n] = v;
            else
                p.y[n] = __float2half_rn(v);
            if constexpr (NB == 2) {
                if (partial)
                    partial[size_t(p.N) + n] = v1;
                else
                    p.y[size_t(p.N) + n] = __float2half_rn(v1);
            }
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
            const int R = V * kUnitRows;
            for (int idx = ctid; idx < NB * R; idx += kConsumerThreads) {
                const int col = idx >= R ? 1 : 0;
                const size_t at = size_t(col) * p.N + size_t(u0) * kUnitRows + (idx - col * R);
                float v = 0.f;
                for (int k0 = 0; k0 < p.k_splits; k0 += 8) {
                    float part[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        part[k] = (k0 + k < p.k_splits) ? __ldcg(p.partial + size_t(k0 + k) * NB * p.N + at) : 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) v += part[k];
                }
                p.y[at] = __float2half_rn(v);
            }
            if (ctid == 0) p.counters[rbi] = 0;
        }
    }
    if (ctid == 0) TRACE(11);
}

template <int Q, bool GROUPED, int NB>
static cudaError_t launch_lut_q(const LutParams &prm, cudaStream_t st)
{
    // The opt-in to more than 48 KB of dynamic shared memory is per function and per device:
    // done on the first launch on each device, remembered afterwards.
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(lut_gemv_kernel<Q, GROUPED, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLutSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(prm.row_blocks * prm.k_splits);
    cfg.blockDim = dim3(kLutThreads);
    cfg.dynamicSmemBytes = kLutSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, GROUPED, NB>, prm);
}

// cols = 1: y = W x.  cols = 2 (grouped scales only): x and y hold two columns, K and N elements apart.
cudaError_t launch_lut_gemv(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *x, uint16_t *y, void *workspace, cudaStream_t st, int cols)
{
    LutParams prm;
    prm.tiles = static_cast<const uint8_t *>(packed);
    prm.alpha = reinterpret_cast<const __half *>(alpha);   // used with per-row scales only
    prm.z = reinterpret_cast<const __half *>(z);
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
    const bool grouped = d.group != 0;
    if (cols == 2) {
        if (!grouped) return cudaErrorInvalidValue;
        switch (d.q) {
            case 1: return launch_lut_q<1, true, 2>(prm, st);
            case 2: return launch_lut_q<2, true, 2>(prm, st);
            case 3: return launch_lut_q<3, true, 2>(prm, st);
            case 4: return launch_lut_q<4, true, 2>(prm, st);
        }
        return cudaErrorInvalidValue;
    }
    switch (d.q) {
        case 1: return grouped ? launch_lut_q<1, true, 1>(prm, st) : launch_lut_q<1, false, 1>(prm, st);
        case 2: return grouped ? launch_lut_q<2, true, 1>(prm, st) : launch_lut_q<2, false, 1>(prm, st);
        case 3: return grouped ? launch_lut_q<3, true, 1>(prm, st) : launch_lut_q<3, false, 1>(prm, st);
        case 4: return grouped ? launch_lut_q<4, true, 1>(prm, st) : launch_lut_q<4, false, 1>(prm, st);
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

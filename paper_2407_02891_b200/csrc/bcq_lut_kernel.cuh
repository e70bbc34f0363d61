// Lookup-table BCQ GEMV for sm_100a: batch 1 (tiled layout, scales per group of 128 or per row), and a
// two-column variant for group 128.
//
//   y = sum_g ( sum_i alpha_i (B_i x)_g + z (sum x)_g )          (Eq. bcw + Eq. fuse_step3)
//
// Per 512-wide window of K the block builds, in shared memory, all 2^8 signed sums of every
// 8-activation chunk; packed weight bytes index those tables directly.  One block per SM, three
// kinds of warps:
//
//   producers (1 or 2 warps) lane c keeps the private ring of consumer warp c filled with bulk async
//                            copies (cp.async.bulk, completion on the slot's mbarrier).  A slot holds one
//                            job = kJ consecutive tiles of one window (one contiguous piece of memory), a
//                            ring kD slots.  The packed weights are constants, so the first slot of every
//                            ring is requested before the kernel waits for its predecessor in the stream;
//                            the rest follows once the first table stands (requests queued earlier
//                            would delay the activations on their way to the block).
//   builders  (3 warps)      build the window tables from x, one window ahead of the consumers
//                            (two tables, double buffered);
//   consumers (kCons warps)  wait for a slot, copy its tiles to registers (handing the slot back after the
//                            last one), look every weight byte up in the window table and accumulate in
//                            fp32.  One tile = q*512 B of plane bytes + the unit's alphas and offsets of one
//                            (window, row unit).
//
// The lookup itself is bound by the shared-memory pipe: one 32-lane lookup is one wavefront, a tile of
// q = 3 planes costs 48 of them plus 14 to bring the tile to registers and 14 for the copy engine to
// write it; per-tile bookkeeping is kept off the consumers for that reason.
//
// Tables.  The sums are computed in fp32 and stored as fp16 (one rounding, relative 2^-11; the
// accumulation of the looked-up values stays fp32).  Both tables share one 64 KB region at a shared-window
// address that is a multiple of 64 KB: entry e of table b, chunk c at byte  e*256 + b*128 + (c>>1)*4 +
// (c&1)*2.  Lane l = 8 g + j of a consumer warp handles row j of a unit and the g-th group of 128 weights
// of the window; it walks the group's 16 chunks skewed by 2 j, so at every step the 32 lanes address 32
// different 4-byte columns -- 32 distinct banks whatever the weight bytes are -- and a lane needs only
// its own (row, group) scales.  With the 256-byte entry stride and the 64 KB alignment ONE byte-permute
// builds the complete address (byte 1 <- weight byte, bytes 0,2,3 <- table address + column): a
// lookup is PRMT + LDS.U16 + one mixed-precision add (fp32 += fp16).
//
// Two columns (NB = 2).  A lookup moves 2 bytes per lane, half of what the shared-memory pipe delivers
// per access; with two activation vectors the entry becomes 4 bytes -- the sums of (column 0, column 1)
// for the same chunk and index -- and one lookup feeds two adds.  Entry e (256 B) is then [even chunks:
// 32 words][odd chunks: 32 words]; all lanes of a warp are at chunks of one parity at any step, so they
// still read 32 different words.  Each table buffer fills a 64 KB region of its own.
//
// Split K.  Every row of the launch owns one 64-bit word of the workspace.  A K split adds its partial row
// sum to that word as a biased fixed-point number, together with an arrival count in the word's top bits,
// with ONE atomic add per row; the add returns the word as it was, so the split that finds k_splits - 1
// earlier arrivals knows the complete sum (what it got back + what it added), rounds it to fp16, stores y
// and puts the word back to zero.  Integer addition is associative: the result does not depend on the order
// of arrival, there is no fence, no second round trip to read partial rows, and no waiting on other blocks.
//
// The kernel is launched with programmatic stream serialisation: it lets its dependents start as soon as
// it runs and waits for its own predecessor only before it touches x, the workspace or y; the packed
// weights are treated as constants that are complete before the launch.
//
// Every wait is bounded; if one runs out the block sets an abort flag and a device status word, stops
// waiting, sees its own copies land and returns (see lut_status_take).
#pragma once
#include "bcq_async.cuh"
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kLutThreads = 896;                  // 28 warps at 72 registers fill the register file
constexpr int kLutSmemBytes = 232448;             // 227 KB: the per-block opt-in maximum
constexpr int kFixedBytes = 2048;                 // barriers and flags
constexpr int kBuilderWarps = 3;
constexpr int kBuilderThreads = kBuilderWarps * 32;
constexpr int kUnitsPerWarp = kLutUnitsPerWarp;   // row units a consumer warp keeps accumulators for
constexpr int kEarlyJobs = 1;                     // jobs per ring requested before the first table stands
constexpr int kTestSpinLimit = 1 << 12;           // polls per wait when a test shortens the limit

static __device__ int g_lut_status = 0;  // 0, or the code of the wait that ran out (sticky until taken); one per translation unit

// Geometry of one instantiation: tile bytes, tiles per job (kJ), slots per ring (kD), consumer warps.
// The rings are cut from the two pieces of shared memory before and after the 64 KB-aligned tables; the
// sizes below assume the usual 1 KB offset of a block's shared window (the kernel checks what it finds).
// SUB: scaling units per 128 weights: 0 = one scale per row (no scales in the tiles), 1, 2, 4 = groups of 128, 64, 32.
template <int Q, int SUB, int NB>
struct LutCfg {
    static constexpr int kTile = Q * 512 + SUB * (Q + 1) * 64;
    static constexpr int kTables = NB * 65536;
    static constexpr int kFront = 65536 - 1024;
    static constexpr int kBack = kLutSmemBytes - kFront - kTables - kFixedBytes;
    static constexpr int rings(int j, int d) { return kFront / (j * d * kTile) + kBack / (j * d * kTile); }
    // preference: two tiles per copy with three slots (small tiles: a warp is through a job before the copy for the
    // slot after the next has crossed HBM), else with two slots; then one tile per copy with three or two slots
    static constexpr int kChoice =
        rings(2, 3) >= kLutConsumersMax ? 0 : (rings(2, 2) >= kLutConsumersMax ? 1 : (rings(1, 3) >= kLutConsumersMax ? 2 : 3));
    static constexpr int kJ = kChoice <= 1 ? 2 : 1;
    static constexpr int kD = (kChoice == 0 || kChoice == 2) ? 3 : 2;
    static constexpr int kCons = rings(kJ, kD) < kLutConsumersMax ? rings(kJ, kD) : kLutConsumersMax;
    // one warp starts about 18 copies per microsecond: enough for jobs of two 1792-byte tiles, not for smaller ones
    static constexpr int kProducers = (kJ == 1 || Q <= 2) ? 2 : 1;
    static constexpr int kFirstCons = kProducers + kBuilderWarps;
    static constexpr int kWorking = kBuilderWarps + kCons;   // warps that take part after the producers split off
    static constexpr int kJobsPerWarp = kUnitsPerWarp / kJ;
    static constexpr int kRingBytes = kJ * kD * kTile;
    static_assert(kCons >= 16 && kFirstCons + kCons <= kLutThreads / 32, "warp budget");
    static_assert(16 * kCons * kD + 64 <= kFixedBytes, "barrier area");
};

// Kernel parameters.  A launch with one operand takes the compact form: the size of the parameter block is
// paid at every launch (176 bytes more cost a quarter of a microsecond), so the arrays that describe several
// operands travel only with the launches that need them.
struct LutOne {
    const uint8_t *tiles;  // tiled operand: per (window, unit) planes (+ alphas, offsets when grouped)
    const __half *alpha;   // per-row scales only: [u][i][r]
    const __half *z;       // per-row scales only: [u][r]
    const __half *x;
    __half *y;
    unsigned long long *accum;  // [cols][N] split-K words (see splitk_encode), all zero between launches; k_splits > 1 only
    int N, K;        // N: rows of all operands together
    int row_blocks, k_splits;   // the grid: blockIdx.x = row block, blockIdx.y = K split
    // Even partitions, prepared by the host so that no block spends its first microsecond dividing: part r of a
    // range cut into n parts starts at r * base + min(r, rem) and has base + (r < rem) items.
    int u_base, u_rem;   // row units over row blocks (one operand)
    int w_base, w_rem;   // windows over K splits
    int test_flags;  // BCQ_PLAN_TEST_* (read by the test instantiations only)
    // what follows the product (one operand, one column): y = act(W x + bias) + residual, in fp32, rounded once
    const __half *bias;      // [N] or null
    const __half *residual;  // [N] or null
    int activation;          // BCQ_ACT_*
    int bf16;                // x, y, bias and residual are bfloat16 instead of fp16 (one operand, one column)
};
// Up to kLutMaxOperands matrices that share x, K, q and the scaling unit are multiplied in one launch: every
// row block belongs to exactly one operand (row blocks rb_first[o] .. rb_first[o + 1] - 1 split operand o's
// row units evenly), so a block works on one operand exactly as it would in a launch of its own.
struct LutMany {
    LutOne one;      // x, split-K words, sizes and decomposition; its tiles / alpha / z / y are not used
    const uint8_t *tiles[kLutMaxOperands];
    const __half *alpha[kLutMaxOperands];
    const __half *z[kLutMaxOperands];
    __half *y[kLutMaxOperands];
    int U[kLutMaxOperands];       // row units of each operand
    int u_base[kLutMaxOperands], u_rem[kLutMaxOperands];   // its row units over its row blocks
    int row0[kLutMaxOperands];    // first row of each operand among all rows of the launch
    int rb_first[kLutMaxOperands + 1];
    int count;
};
template <bool MULTI> struct LutParamsOf { typedef LutOne type; };
template <> struct LutParamsOf<true> { typedef LutMany type; };

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
// the first lookup of a sum: acc = entry
template <int OFF>
__device__ __forceinline__ float lut_first(uint32_t addr)
{
    float f;
    asm volatile(
        "{\n\t.reg .b16 h;\n\t"
        "ld.shared.b16 h, [%1+%2];\n\t"
        "cvt.f32.f16 %0, h;\n\t}"
        : "=f"(f)
        : "r"(addr), "n"(OFF));
    return f;
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
__device__ __forceinline__ void lut_first2(float &acc0, float &acc1, uint32_t addr)
{
    asm volatile(
        "{\n\t.reg .b16 l, h;\n\t.reg .b32 v;\n\t"
        "ld.shared.b32 v, [%2+%3];\n\t"
        "mov.b32 {l, h}, v;\n\t"
        "cvt.f32.f16 %0, l;\n\t"
        "cvt.f32.f16 %1, h;\n\t}"
        : "=f"(acc0), "=f"(acc1)
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
// two 16-bit activations -> fp32 (exact): fp16, or bfloat16 (the upper half of an fp32)
__device__ __forceinline__ float2 act_pair_to_f32(uint32_t raw, bool bf16)
{
    if (bf16) return make_float2(__uint_as_float(raw << 16), __uint_as_float(raw & 0xffff0000u));
    return __half22float2(*reinterpret_cast<const __half2 *>(&raw));
}
__device__ __forceinline__ void load_quad(const __half *xw, int cq, f32x2 (&x01)[8], f32x2 (&x23)[8], bool bf16 = false)
{
    float xf[4][8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(xw + 32 * cq + 8 * k);
        const uint32_t r4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = act_pair_to_f32(r4[j], bf16);
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

// ---- split-K words -------------------------------------------------------------------------------
// bits 63..57: arrivals; bits 56..50: arrivals whose partial sum was NaN; bits 49..0: sum over the arrivals of
// (partial sum in units of 2^-26, clamped to +-(2^17 - 1)) + 2^43.  Every term of the low field is below 2^44,
// so 64 arrivals stay below 2^50 and no field carries into the next.  fp32 partial sums of magnitude 2^-2
// and more are represented exactly; the rest is rounded to a multiple of 2^-26, a quarter of the smallest
// step of the fp16 result.  Partial sums beyond +-131071 (twice the fp16 range) saturate; an infinite one
// saturates too and makes the result infinite unless the other splits cancel it.
constexpr int kSplitFracBits = 26;
constexpr long long kSplitBias = 1ll << 43;
__device__ __forceinline__ unsigned long long splitk_encode(float v)
{
    if (v != v) return (1ull << 57) + (1ull << 50) + (unsigned long long)kSplitBias;
    v = fminf(fmaxf(v, -131071.f), 131071.f);
    const long long f = __float2ll_rn(v * float(1 << kSplitFracBits));   // exact product, |f| < 2^43
    return (1ull << 57) + (unsigned long long)(f + kSplitBias);
}
__device__ __forceinline__ int splitk_arrivals(unsigned long long w) { return int(w >> 57); }
// the fp16 result from a complete word: one rounding of the exact fixed-point sum
__device__ __forceinline__ __half splitk_decode(unsigned long long w, int k_splits)
{
    if ((w >> 50) & 127) return __ushort_as_half((unsigned short)0x7fffu);   // a NaN partial sum
    const long long s = (long long)(w & ((1ull << 50) - 1)) - (long long)k_splits * kSplitBias;
    return __double2half(double(s) * (1.0 / double(1 << kSplitFracBits)));
}
// the same sum as fp32 (for what follows the product)
__device__ __forceinline__ float splitk_decode_f32(unsigned long long w, int k_splits)
{
    if ((w >> 50) & 127) return __int_as_float(0x7fffffff);
    const long long s = (long long)(w & ((1ull << 50) - 1)) - (long long)k_splits * kSplitBias;
    return float(double(s) * (1.0 / double(1 << kSplitFracBits)));
}

// y = act(v + bias) + residual for row n
__device__ __forceinline__ float lut_ld16(const __half *a, size_t n, bool bf16)
{
    const unsigned short raw = __half_as_ushort(a[n]);
    return bf16 ? __uint_as_float(uint32_t(raw) << 16) : __half2float(__ushort_as_half(raw));
}
__device__ __forceinline__ __half lut_finish(float v, const LutOne &p, size_t n)
{
    const bool bf16 = p.bf16 != 0;
    if (p.bias) v += lut_ld16(p.bias, n, bf16);
    switch (p.activation) {
        case BCQ_ACT_RELU: v = fmaxf(v, 0.f); break;
        case BCQ_ACT_GELU: v = 0.5f * v * (1.f + erff(v * 0.70710678118654752f)); break;
        case BCQ_ACT_SILU: v = v / (1.f + expf(-v)); break;
        default: break;
    }
    if (p.residual) v += lut_ld16(p.residual, n, bf16);
    if (bf16) {   // round to nearest even on the upper 16 bits; NaN stays NaN
        const uint32_t u = __float_as_uint(v);
        const uint32_t r = (v != v) ? 0x7fc0u : ((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
        return __ushort_as_half((unsigned short)r);
    }
    return __float2half_rn(v);
}

__host__ __device__ inline const LutOne &lut_one(const LutOne &p) { return p; }
__host__ __device__ inline const LutOne &lut_one(const LutMany &p) { return p.one; }

enum { kWaitEmpty = 1, kWaitFull = 2, kWaitTableReady = 3, kWaitTableFree = 4, kWaitDrain = 5, kTooFewRings = 6, kWaitStart = 7 };

// A bounded wait whose limit a test can shorten (see BCQ_PLAN_TEST_SHORT_WAITS).
template <bool LONG = false>
__device__ __forceinline__ bool lut_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int code, int limit)
{
    for (int it = 0; it < limit; ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        if (LONG && it >= 8)
            __nanosleep(256);
        else
            __nanosleep(32);
        if ((it & 255) == 255 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(&g_lut_status, code);
    return false;
}

// NB columns per launch: 1, or 2 (grouped scales only) with tables that hold both columns' sums side by
// side, so that one 4-byte lookup serves two products; each of the two table buffers then fills a
// 64 KB region of its own.
// MULTI: several operands (batch 1); TEST: the instantiation the library's tests use to see a wait run out
// (short limits, and the builders keep a finished table to themselves when the plan asks for it).
template <int Q, int SUB, int NB, bool MULTI, bool TEST>
__global__ void __launch_bounds__(kLutThreads, 1) lut_gemv_kernel(const typename LutParamsOf<MULTI>::type pm)
{
    constexpr bool GROUPED = SUB > 0;
    constexpr int kPhase = SUB > 1 ? 16 / SUB : 16;   // steps (chunks) a lane spends in one scaling unit of its segment
    constexpr int kWordsPerUnit = SUB > 1 ? 8 / SUB : 8;
    static_assert(SUB == 0 || SUB == 1 || SUB == 2 || SUB == 4, "scaling units per 128 weights");
    static_assert(NB == 1 || (NB == 2 && SUB == 1), "two columns: groups of 128 only");
    static_assert(!MULTI || NB == 1, "several operands: batch 1");
    const LutOne &p = lut_one(pm);
    using C = LutCfg<Q, SUB, NB>;
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kTile = C::kTile, kJ = C::kJ, kD = C::kD, kCons = C::kCons;
    constexpr int kSlotBytes = kJ * kTile;
    constexpr int NACC = GROUPED ? 1 : Q;   // accumulators per unit and lane: the row's sum, or one per plane
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int rbi = blockIdx.x, ks = blockIdx.y;
    int op = 0, rbl = rbi, U = p.N / kUnitRows, row0 = 0, u_base = p.u_base, u_rem = p.u_rem;
    const uint8_t *tiles = p.tiles;
    const __half *alpha = p.alpha, *zoff = p.z;
    __half *y = p.y;
    if constexpr (MULTI) {   // the operand this row block belongs to
        while (op + 1 < pm.count && rbi >= pm.rb_first[op + 1]) ++op;
        rbl = rbi - pm.rb_first[op];
        U = pm.U[op], row0 = pm.row0[op], u_base = pm.u_base[op], u_rem = pm.u_rem[op];
        tiles = pm.tiles[op], alpha = pm.alpha[op], zoff = pm.z[op], y = pm.y[op];
    }
    const int u0 = rbl * u_base + min(rbl, u_rem);
    const int w0 = ks * p.w_base + min(ks, p.w_rem);
    const int V = u_base + (rbl < u_rem ? 1 : 0);        // row units of this block
    const int nwin = p.w_base + (ks < p.w_rem ? 1 : 0);  // windows of this block
    const int njobs = (V + kJ - 1) / kJ;         // jobs per window
    constexpr int spin_limit = TEST ? kTestSpinLimit : kSpinLimit;

    // ---- carve shared memory: [front | tables (64 KB each, 64 KB aligned) | barriers | back] --------------
    const uint32_t base = smem_u32(smem);
    const uint32_t tab0 = (base + 0xFFFFu) & ~0xFFFFu;  // shared-window address of the tables
    const int front = int(tab0 - base), back = kLutSmemBytes - front - C::kTables;
    unsigned char *tables = smem + front;
    unsigned char *after = tables + C::kTables;
    const bool fixed_in_back = back >= kFixedBytes;
    unsigned char *fixed = fixed_in_back ? after : smem;
    unsigned char *ring_a = fixed_in_back ? smem : smem + kFixedBytes;
    unsigned char *ring_b = fixed_in_back ? after + kFixedBytes : after;
    const int rings_a = (fixed_in_back ? front : front - kFixedBytes) / C::kRingBytes;
    const int rings_b = (fixed_in_back ? back - kFixedBytes : back) / C::kRingBytes;
    auto ring_ptr = [&](int c) -> unsigned char * {
        return c < rings_a ? ring_a + c * C::kRingBytes : ring_b + (c - rings_a) * C::kRingBytes;
    };

    const uint32_t bars = smem_u32(fixed);
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kCons * kD;     // [consumer][slot]
    const uint32_t bar_tab_ready = bars + 16 * kCons * kD, bar_tab_free = bar_tab_ready + 16;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(fixed + 16 * kCons * kD + 32);
    volatile int *started = abort_flag + 1;

    if (warp == 0) {   // one warp initialises the barriers, a few each
        for (int s = lane; s < kCons * kD; s += 32) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        if (lane < 2) {
            mbar_init(bar_tab_ready + 8 * lane, kBuilderThreads);
            mbar_init(bar_tab_free + 8 * lane, kCons);
        }
        if (lane == 0) {
            // every consumer warp needs its ring, and the block's row units must fit the consumers
            const bool bad = rings_a + rings_b < kCons || njobs > kCons * C::kJobsPerWarp;
            *abort_flag = bad ? 1 : 0;
            *started = 0;
            if (bad) atomicExch(&g_lut_status, int(kTooFewRings));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch: the next kernel in the stream may start taking SMs as soon as
    // this kernel's blocks leave them (it still waits, below, for its predecessor to finish before
    // it reads x or writes anything).  Without the launch attribute both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // Work of consumer c: jobs jb = c, c + kCons, ... of every window, in that order; its m-th job uses slot
    // m % kD of its ring in fill number m / kD.
    // =============================================================================================
    // ---- producers: lane -> consumer c; keeps that consumer's ring filled ---------------------------
    if (warp < C::kProducers) {
        const int c = lane * C::kProducers + warp;
        const int mine = (c < kCons && njobs > c) ? (njobs - c + kCons - 1) / kCons : 0;   // jobs per window
        if (mine > 0 && !*abort_flag) {
            const uint32_t ring = smem_u32(ring_ptr(c));
            const uint32_t full0 = bar_full + 8 * kD * c, empty0 = bar_empty + 8 * kD * c;
            int slot = 0, fill = 0, issued = 0;
            const uint8_t *src_w = tiles + (size_t(w0) * U + u0) * kTile;
            bool ok = true;
            for (int wi = 0; wi < nwin && ok; ++wi) {
                for (int jb = c; jb < njobs; jb += kCons) {
                    if (issued == kEarlyJobs) {
                        // The rest of the ring waits until the first table stands.  First wait, like the other
                        // warps, for the previous kernel (however long it runs); the flag follows shortly.
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        int itr = 0;
                        while (!*started && !*abort_flag && itr < spin_limit) {
                            __nanosleep(64);
                            ++itr;
                        }
                        if (!*started) {
                            if (!*abort_flag) {
                                *abort_flag = 1;
                                atomicExch(&g_lut_status, int(kWaitStart));
                            }
                            ok = false;
                            break;
                        }
                    }
                    if (fill > 0 && !lut_wait(empty0 + 8 * slot, (fill - 1) & 1, abort_flag, kWaitEmpty, spin_limit)) {
                        ok = false;
                        break;
                    }
                    const int nt = min(kJ, V - kJ * jb);
                    mbar_expect_tx(full0 + 8 * slot, nt * kTile);
                    bulk_g2s(ring + slot * kSlotBytes, src_w + size_t(kJ * jb) * kTile, nt * kTile, full0 + 8 * slot);
                    ++issued;
                    if (++slot == kD) {
                        slot = 0;
                        ++fill;
                    }
                }
                src_w += size_t(U) * kTile;
            }
            // See the lane's last copies land before the block's shared memory can be handed to another
            // block (they have landed long ago unless the block is giving up).
            for (int m = max(0, issued - kD); m < issued; ++m) {
                bool landed = false;
                for (int itr = 0; itr < kSpinLimit && !landed; ++itr) {
                    landed = mbar_test_wait(full0 + 8 * (m % kD), uint32_t((m / kD) & 1));
                    if (!landed) __nanosleep(256);
                }
                if (!landed) atomicExch(&g_lut_status, int(kWaitDrain));
            }
        }
        return;
    }
    if (warp >= C::kFirstCons + kCons) return;   // warps this instantiation has no use for

    // =============================================================================================
    // The weights above are constants; everything from here on (x, partial sums, counters, y) may
    // depend on the previous kernel in the stream: wait for it to be complete and visible.
    const __half *xblk = p.x + size_t(w0) * kWindow;   // this block's slice of x
    bool in_bf16 = false;
    if constexpr (NB == 1 && !MULTI) in_bf16 = p.bf16 != 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- start-up: builders and consumers build the first window's table together -----------------
    const int bt = tid - C::kProducers * 32;   // 0 .. kWorking*32-1
    if (bt < 512) {
        if constexpr (NB == 1) {
            f32x2 x01[8], x23[8];
            load_quad(xblk, bt & 15, x01, x23, in_bf16);
            build_quad(tables, x01, x23, bt & 15, bt >> 4, 32);
        } else {
            f32x2 xa[8], xb[8];
            load_pair(xblk, size_t(p.K), bt & 31, xa, xb);
            build_pair(tables, xa, xb, bt & 31, bt >> 5, 16);
        }
    }
    named_barrier(1, C::kWorking * 32);
    if (bt == 0) *started = 1;

    if (warp < C::kFirstCons) {
        // ---- builders: one table per window, one window ahead of the consumers ----------------------
        // Window 0 was built above; the builders' fills of buffer 0 are windows 2, 4, ... and of
        // buffer 1 windows 1, 3, ...
        const bool withhold = TEST && (p.test_flags & BCQ_PLAN_TEST_WITHHOLD_TABLE) != 0;
        for (int wi = 1; wi < nwin; ++wi) {
            const int b = wi & 1, use = wi >> 1;
            f32x2 x01[8], x23[8];   // one column: a chunk quad; two columns: a chunk pair of each
            if constexpr (NB == 1)
                load_quad(xblk + wi * kWindow, bt & 15, x01, x23, in_bf16);   // in flight while waiting for the buffer
            else
                load_pair(xblk + wi * kWindow, size_t(p.K), bt & 31, x01, x23);
            if (use > 0 && !lut_wait<true>(bar_tab_free + 8 * b, (use - 1) & 1, abort_flag, kWaitTableFree, spin_limit)) break;
            if constexpr (NB == 1)
                build_quad(tables + b * 128, x01, x23, bt & 15, bt >> 4, kBuilderThreads / 16);
            else
                build_pair(tables + b * 65536, x01, x23, bt & 31, bt >> 5, kBuilderThreads / 32);
            if (!withhold) mbar_arrive(bar_tab_ready + 8 * b);   // (a test withholds it to see the consumers give up)
        }
        return;
    }

    // =============================================================================================
    // ---- consumers ---------------------------------------------------------------------------------
    // Lane l = 8 g + j owns row 8u + j of every unit and the g-th group of 128 weights of every
    // window: its 16q bytes of a tile are the group's 16 chunks (skewed by 2 j, see the layout), so
    // it needs only its own q alphas and one offset per tile and keeps ONE accumulator per unit.
    const int cw = warp - C::kFirstCons;
    const int g4 = lane >> 3, jr = lane & 7;
    float acc[kUnitsPerWarp][NACC], acc1[NB == 2 ? kUnitsPerWarp : 1];   // acc1: the second column
    float xacc = 0.f;   // per-row scales: sum of x over this lane's groups of all windows
#pragma unroll
    for (int t = 0; t < kUnitsPerWarp; ++t)
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[t][i] = 0.f;
#pragma unroll
    for (int t = 0; t < (NB == 2 ? kUnitsPerWarp : 1); ++t) acc1[t] = 0.f;
    if constexpr (!GROUPED) {
        // One scale per row: the rows' alphas and offsets are needed once, after the last window.  Ask for their
        // lines now (constants, like the weights), so that the block's last step does not wait for them.
        if (lane < 2 * kUnitsPerWarp) {
            const int a = lane & (kUnitsPerWarp - 1);
            const int ul = kJ * (cw + kCons * (a / kJ)) + a % kJ;
            if (ul < V) {
                const __half *line = lane < kUnitsPerWarp ? alpha + size_t(u0 + ul) * Q * kUnitRows : zoff + size_t(u0 + ul) * kUnitRows;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
            }
        }
    }
    bool alive = !*abort_flag;
    const unsigned char *ring = ring_ptr(cw);
    const uint32_t full0 = bar_full + 8 * kD * cw, empty0 = bar_empty + 8 * kD * cw;
    int slot = 0, fill = 0;

    for (int wi = 0; wi < nwin && alive; ++wi) {
        const int b = wi & 1;
        if (wi > 0 && !lut_wait(bar_tab_ready + 8 * b, ((wi >> 1) - (b == 0 ? 1 : 0)) & 1, abort_flag, kWaitTableReady, spin_limit)) {
            alive = false;
            break;
        }
        // Table address part of the lookups of step pair h: chunk 16 g + ((2h + 2j) mod 16) and the
        // next one share the 4-byte column 8 g + ((h + j) mod 8); the odd chunk is its upper half.
        uint32_t off[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) {
            int col = (h + jr) & 7;
            if constexpr (SUB > 1) {   // unit by unit: see tile_chunk() for the walk
                const int ph = (2 * h) / kPhase, th = ((2 * h) % kPhase) >> 1;
                col = kWordsPerUnit * ((ph + jr / kWordsPerUnit) % SUB) + (th + jr) % kWordsPerUnit;
            }
            off[h] = tab0 + uint32_t(b * (NB == 1 ? 128 : 65536) + 4 * (8 * g4 + col));
        }
        // sum of x over this lane's group: the all-ones entries of the group's 16 chunks (two per lane)
        float xsum, xsum1 = 0.f;
        [[maybe_unused]] float xs[SUB > 1 ? SUB : 1];   // SUB > 1: sum of x over the unit of every phase
        if constexpr (SUB > 1) {
#pragma unroll
            for (int ph = 0; ph < SUB; ++ph) {
                const int sg = (ph + jr / kWordsPerUnit) % SUB;
                float acc_x = 0.f;
#pragma unroll
                for (int k = 0; k < kWordsPerUnit; ++k) {
                    const uint32_t ones = lds_b32<255 * 256>(tab0 + uint32_t(b * 128 + 4 * (8 * g4 + kWordsPerUnit * sg + k)));
                    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&ones));
                    acc_x += f.x + f.y;
                }
                xs[ph] = acc_x;
            }
            xsum = 0.f;
        } else if constexpr (NB == 1) {
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
        if constexpr (SUB <= 1) {
            xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
            xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
            xsum += __shfl_xor_sync(0xffffffffu, xsum, 4);
        }
        xacc += xsum;

        static_for<0, C::kJobsPerWarp>([&](auto T) {
            constexpr int t = decltype(T)::value;
            const int jb = cw + kCons * t;
            if (alive && jb < njobs) {
                if (!lut_wait(full0 + 8 * slot, fill & 1, abort_flag, kWaitFull, spin_limit)) {
                    alive = false;
                } else {
                    const unsigned char *sl = ring + slot * kSlotBytes;
                    const int nt = min(kJ, V - kJ * jb);   // the last job of a window may be short
                    static_for<0, kJ>([&](auto TT) {
                        constexpr int tt = decltype(TT)::value;
                        constexpr int a = t * kJ + tt;     // accumulator slot of this unit
                        if (tt < nt) {
                            const unsigned char *tile = sl + tt * kTile;
                            uint32_t wbuf[4 * Q];
#pragma unroll
                            for (int j = 0; j < Q; ++j) {
                                const uint4 v = *reinterpret_cast<const uint4 *>(tile + j * 512 + lane * 16);
                                wbuf[4 * j + 0] = v.x;
                                wbuf[4 * j + 1] = v.y;
                                wbuf[4 * j + 2] = v.z;
                                wbuf[4 * j + 3] = v.w;
                            }
                            // alpha_0 .. alpha_{q-1}, z of (row, group) = this lane; SUB > 1: one set per phase
                            [[maybe_unused]] __align__(8) __half sc[(SUB > 1 ? SUB : 1) * (Q + 1)];
                            if constexpr (SUB > 1) {
                                const uint32_t *sp = reinterpret_cast<const uint32_t *>(tile + Q * 512 + lane * (2 * SUB * (Q + 1)));
#pragma unroll
                                for (int k = 0; k < SUB * (Q + 1) / 2; ++k) reinterpret_cast<uint32_t *>(sc)[k] = sp[k];
                            } else if constexpr (GROUPED) {
                                const unsigned char *sp = tile + Q * 512 + lane * (2 * (Q + 1));
                                if constexpr (Q == 3) {
                                    *reinterpret_cast<uint2 *>(sc) = *reinterpret_cast<const uint2 *>(sp);
                                } else if constexpr (Q == 1) {
                                    *reinterpret_cast<uint32_t *>(sc) = *reinterpret_cast<const uint32_t *>(sp);
                                } else {
#pragma unroll
                                    for (int i = 0; i <= Q; ++i) sc[i] = reinterpret_cast<const __half *>(sp)[i];
                                }
                            }
                            if (tt == nt - 1) {   // the slot's last tile is in registers: hand the slot back
                                __syncwarp();
                                if (lane == 0) mbar_arrive(empty0 + 8 * slot);
                            }
                            float sum[Q], sum1[NB == 2 ? Q : 1];
                            [[maybe_unused]] float vsub = acc[a][0];   // SUB > 1: the row's sum, a scaling unit at a time
                            static_for<0, 16>([&](auto S) {
                                constexpr int st = decltype(S)::value;
                                static_for<0, Q>([&](auto I) {
                                    constexpr int i = decltype(I)::value;
                                    constexpr int pb = i * 16 + st;
                                    const uint32_t addr = __byte_perm(wbuf[pb >> 2], off[st >> 1], 0x7604 | ((pb & 3) << 4));
                                    if constexpr (NB == 1) {
                                        if constexpr (st % kPhase == 0)
                                            sum[i] = lut_first<(st & 1) * 2>(addr);
                                        else
                                            lut_add<(st & 1) * 2>(sum[i], addr);
                                    } else {
                                        if constexpr (st == 0)
                                            lut_first2<0>(sum[i], sum1[i], addr);
                                        else
                                            lut_add2<(st & 1) * 128>(sum[i], sum1[i], addr);
                                    }
                                });
                                if constexpr (SUB > 1 && st % kPhase == kPhase - 1) {   // a scaling unit is complete
                                    constexpr int ph = st / kPhase;
                                    vsub = fmaf(__half2float(sc[ph * (Q + 1) + Q]), xs[ph], vsub);
#pragma unroll
                                    for (int i = 0; i < Q; ++i) vsub = fmaf(__half2float(sc[ph * (Q + 1) + i]), sum[i], vsub);
                                }
                            });
                            if constexpr (SUB > 1) {
                                acc[a][0] = vsub;
                            } else if constexpr (GROUPED) {
                                float v = fmaf(__half2float(sc[Q]), xsum, acc[a][0]);
#pragma unroll
                                for (int i = 0; i < Q; ++i) v = fmaf(__half2float(sc[i]), sum[i], v);
                                acc[a][0] = v;
                                if constexpr (NB == 2) {
                                    float v1 = fmaf(__half2float(sc[Q]), xsum1, acc1[a]);
#pragma unroll
                                    for (int i = 0; i < Q; ++i) v1 = fmaf(__half2float(sc[i]), sum1[i], v1);
                                    acc1[a] = v1;
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < Q; ++i) acc[a][i] += sum[i];
                            }
                        }
                    });
                    if (++slot == kD) {
                        slot = 0;
                        ++fill;
                    }
                }
            }
        });
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tab_free + 8 * b);
    }
    if (!alive) return;   // the block is giving up: y is undefined (bcq_poll_status reports it)

    // ---- a unit's row j is spread over the 4 lanes 8 g + j: add them up (all four end up with the sum).
    // One K split: lanes 0..7 store y.  Several: lane 8 g + j adds the rows j of the warp's accumulator slots
    // g and g + 4 to their split-K words (32 rows per atomic instruction); whoever completes a word stores
    // that row of y and clears the word.
    // (Two columns: the second column's words follow the first column's, N further on; its rows of y start
    // after the operand's own rows.) ----------------------------------------------------------------------
    const bool split = p.k_splits > 1;
    bool finish = false;   // something follows the product (one operand, one column only)
    if constexpr (NB == 1 && !MULTI) finish = p.bias != nullptr || p.residual != nullptr || p.activation != BCQ_ACT_NONE || p.bf16 != 0;
    unsigned long long *accum = split ? p.accum + row0 : nullptr;
    const size_t Nop = size_t(U) * kUnitRows;   // rows of this operand: its second column of y starts there
    float tot[kUnitsPerWarp], tot1[NB == 2 ? kUnitsPerWarp : 1];
    // one scale per row: all the rows' alphas and offsets are asked for together, before the first is used
    // (one trip to L2 for the block's last step instead of one per unit)
    [[maybe_unused]] __half row_scale[GROUPED ? 1 : kUnitsPerWarp][Q + 1];
    if constexpr (!GROUPED) {
#pragma unroll
        for (int a = 0; a < kUnitsPerWarp; ++a) {
            const int ul = kJ * (cw + kCons * (a / kJ)) + a % kJ;
            const int u = u0 + (ul < V ? ul : 0);
#pragma unroll
            for (int i = 0; i < Q; ++i) row_scale[a][i] = alpha[(size_t(u) * Q + i) * kUnitRows + jr];
            row_scale[a][Q] = zoff[size_t(u) * kUnitRows + jr];
        }
    }
#pragma unroll
    for (int a = 0; a < kUnitsPerWarp; ++a) {
        const int ul = kJ * (cw + kCons * (a / kJ)) + a % kJ;   // the unit, counted inside the block
        tot[a] = 0.f;
        if constexpr (NB == 2) tot1[a] = 0.f;
        if (ul >= V) continue;                                  // (the same for the whole warp)
        float v = acc[a][0];
        if constexpr (!GROUPED) {
            // apply the row's alphas and offset to the sums over this block's K range
            v = 0.f;
#pragma unroll
            for (int i = 0; i < Q; ++i) v = fmaf(__half2float(row_scale[a][i]), acc[a][i % NACC], v);
            v = fmaf(__half2float(row_scale[a][Q]), xacc, v);
        }
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        tot[a] = v;
        if constexpr (NB == 2) {
            float v1 = acc1[a];
            v1 += __shfl_xor_sync(0xffffffffu, v1, 8);
            v1 += __shfl_xor_sync(0xffffffffu, v1, 16);
            tot1[a] = v1;
        }
        if (!split && lane < 8) {
            const size_t n = size_t(u0 + ul) * kUnitRows + jr;   // row inside the operand
            y[n] = finish ? lut_finish(v, p, n) : __float2half_rn(v);
            if constexpr (NB == 2) y[Nop + n] = __float2half_rn(tot1[a]);
        }
    }
    if (split) {
        // two passes over the warp's accumulator slots, 32 rows each: lane 8 g + j takes row j of slot 4 h + g
#pragma unroll
        for (int h = 0; h < kUnitsPerWarp / 4; ++h) {
            const int a = 4 * h + g4;
            const int ul = kJ * (cw + kCons * (a / kJ)) + a % kJ;
            if (ul < V) {
                const size_t n = size_t(u0 + ul) * kUnitRows + jr;
                const float v = g4 == 0 ? tot[4 * h] : (g4 == 1 ? tot[4 * h + 1] : (g4 == 2 ? tot[4 * h + 2] : tot[4 * h + 3]));
                const unsigned long long mine = splitk_encode(v);
                const unsigned long long before = atomicAdd(accum + n, mine);
                if (splitk_arrivals(before) == p.k_splits - 1) {
                    y[n] = finish ? lut_finish(splitk_decode_f32(before + mine, p.k_splits), p, n) : splitk_decode(before + mine, p.k_splits);
                    accum[n] = 0;
                }
                if constexpr (NB == 2) {
                    const float v1 = g4 == 0 ? tot1[4 * h] : (g4 == 1 ? tot1[4 * h + 1] : (g4 == 2 ? tot1[4 * h + 2] : tot1[4 * h + 3]));
                    const unsigned long long mine1 = splitk_encode(v1);
                    const unsigned long long before1 = atomicAdd(accum + size_t(p.N) + n, mine1);
                    if (splitk_arrivals(before1) == p.k_splits - 1) {
                        y[Nop + n] = splitk_decode(before1 + mine1, p.k_splits);
                        accum[size_t(p.N) + n] = 0;
                    }
                }
            }
        }
    }
}

template <int Q, int SUB, int NB, bool MULTI, bool TEST>
static cudaError_t launch_lut_inst(const typename LutParamsOf<MULTI>::type &prm, cudaStream_t st)
{
    // The opt-in to more than 48 KB of dynamic shared memory is per function and per device:
    // done on the first launch on each device, remembered afterwards.
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(lut_gemv_kernel<Q, SUB, NB, MULTI, TEST>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLutSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(lut_one(prm).row_blocks, lut_one(prm).k_splits);
    cfg.blockDim = dim3(kLutThreads);
    cfg.dynamicSmemBytes = kLutSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, lut_gemv_kernel<Q, SUB, NB, MULTI, TEST>, prm);
}

// Read and clear this translation unit's device status word.
static cudaError_t lut_status_take_here(int *status)
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

// All instantiations for one number of planes: one column or two (grouped scales), one operand or several
// (one column), and the test instantiation (one operand, one column).
template <int Q>
static cudaError_t launch_lut_for_q(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st)
{
    if (sub == 2 || sub == 4) {   // groups of 64 and 32: one operand, one column
        if (many || cols != 1 || test) return cudaErrorInvalidValue;
        return sub == 2 ? launch_lut_inst<Q, 2, 1, false, false>(*one, st) : launch_lut_inst<Q, 4, 1, false, false>(*one, st);
    }
    if (many) {
        if (cols != 1 || test) return cudaErrorInvalidValue;
        return sub ? launch_lut_inst<Q, 1, 1, true, false>(*many, st) : launch_lut_inst<Q, 0, 1, true, false>(*many, st);
    }
    if (cols == 2) {
        if (!sub || test) return cudaErrorInvalidValue;
        return launch_lut_inst<Q, 1, 2, false, false>(*one, st);
    }
    if (test) return sub ? launch_lut_inst<Q, 1, 1, false, true>(*one, st) : launch_lut_inst<Q, 0, 1, false, true>(*one, st);
    return sub ? launch_lut_inst<Q, 1, 1, false, false>(*one, st) : launch_lut_inst<Q, 0, 1, false, false>(*one, st);
}

}  // namespace bcq

// The extern "C" boundary of libbcq: argument validation, the default decomposition, the
// host-side table of the linear-int -> binary-code conversion, and dispatch to the kernels.
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "bcq_internal.cuh"

using namespace bcq;

namespace {
thread_local char g_cuda_error[256] = "";
}

// Remember the text of a failed CUDA runtime call for bcq_last_cuda_error(); returns BCQ_ERR_CUDA.
int bcq::record_cuda_error(cudaError_t e)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return BCQ_ERR_CUDA;
}

namespace {

int cuda_fail(cudaError_t e) { return bcq::record_cuda_error(e); }

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_desc(const bcq_desc *d)
{
    if (!d) return BCQ_ERR_INVALID_ARG;
    if (d->N <= 0 || d->K <= 0 || d->q < 1 || d->q > 4 || d->group < 0) return BCQ_ERR_INVALID_ARG;
    if (d->layout != BCQ_LAYOUT_CANONICAL && d->layout != BCQ_LAYOUT_TILED) return BCQ_ERR_INVALID_ARG;
    if (d->K % 32 != 0) return BCQ_ERR_UNSUPPORTED_SHAPE;
    if (d->group != 0 && (d->K % d->group != 0 || d->group % 32 != 0)) return BCQ_ERR_UNSUPPORTED_SHAPE;
    if (d->layout == BCQ_LAYOUT_TILED) {
        if (d->K % kWindow != 0 || d->N % kUnitRows != 0) return BCQ_ERR_UNSUPPORTED_SHAPE;
        if (d->group != 0 && d->group != 128 && d->group != 64 && d->group != 32) return BCQ_ERR_UNSUPPORTED_SHAPE;
    }
    return BCQ_OK;
}

bool same_problem(const bcq_desc *a, const bcq_desc *b)
{
    return a->N == b->N && a->K == b->K && a->q == b->q && a->group == b->group;
}

int device_sm_count(int *out)
{
    int dev = 0, sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    *out = sm;
    return BCQ_OK;
}

// From this many columns on the default plan is the tensor-core kernel.  With the scales in the tiles the
// lookup-table kernel takes two columns per pass, and two such passes (4 columns) are still faster than one
// pass of the tensor-core kernel (measured on Llama-2-70B-shaped layers: 1.73 against 2.03 ms per 8 layers).
constexpr int kSmallBatchMin = 4;
constexpr int kSmallBatchMinPairs = 5;
// column pairs and the tensor-core kernel exist for groups of 128 (and, the latter, one scale per row); groups of
// 64 and 32 run the lookup-table kernel column by column
bool pairs_ok(const bcq_desc *d) { return d->layout == BCQ_LAYOUT_TILED && d->group == 128; }
bool mma_ok(const bcq_desc *d) { return d->layout == BCQ_LAYOUT_TILED && (d->group == 128 || d->group == 0); }
int small_batch_min(const bcq_desc *d) { return !mma_ok(d) ? 17 : (pairs_ok(d) ? kSmallBatchMinPairs : kSmallBatchMin); }

bool lut_kernel_covers(const bcq_desc *d) { return d->layout == BCQ_LAYOUT_TILED; }   // group 128 or one scale per row

// tiled layout with grouped scales: alpha and z live inside `packed`
bool interleaved(const bcq_desc *d) { return d->layout == BCQ_LAYOUT_TILED && d->group != 0; }

// Row units one block of the lookup-table kernel can take for `cols` columns per launch (B >= 2 with the
// scales in the tiles runs column pairs, and a last single column with the same plan).
int lut_max_units(const bcq_desc *d, int B)
{
    const int sub = scale_subs(d->group);
    int cons = lut_consumer_warps(d->q, sub, 1);
    if (B >= 2 && pairs_ok(d)) {
        const int c2 = lut_consumer_warps(d->q, sub, 2);
        if (c2 < cons) cons = c2;
    }
    return cons * kLutUnitsPerWarp;
}

// Time model of the lookup-table kernel in nanoseconds, fitted to sweeps of decompositions over the 19 layer
// shapes of the workloads on B200 (its pick is within 0.4 % of the fastest measured plan on average, 3.5 % at
// worst).  A block walks its windows; the work of a window is dealt to the consumer warps in jobs, so a window
// costs between its tiles and whole rounds of jobs; the table of the next window is built meanwhile by three
// warps (about 2.2 us from the previous table, and not before the buffer it overwrites is free), so blocks
// with short windows wait for tables; a K split costs little (one atomic per row).  It ranks decompositions;
// it does not predict time exactly.
double lut_cost(int U, int W, int rb, int ks, int sm, int cons, int tiles_per_job, int cols)
{
    // (two columns: twice the table entries to build, 4 instead of 3 instructions per lookup)
    const double per_tile = cols == 2 ? 50.0 : 38.0, table_build = 2200.0 * cols, split_fixed = 500.0, per_split = 10.0, round_weight = 0.3,
                 per_reuse = 100.0;   // measured on the long-K shapes (56 and 72 windows): fewer, longer windows per block lose
    const long long blocks = static_cast<long long>(rb) * ks;
    const long long waves = (blocks + sm - 1) / sm;
    const int wc = (W + ks - 1) / ks;
    const int units = (U + rb - 1) / rb;
    const int jobs = (units + tiles_per_job - 1) / tiles_per_job;
    const int rounds = (jobs + cons - 1) / cons;
    const double tiles = (1.0 - round_weight) * units + round_weight * double(rounds) * tiles_per_job * cons;
    const double window = tiles * per_tile;
    double end_prev = window;      // the first window (its table is built by the whole block)
    double ready = table_build;    // when the second window's table stands
    for (int w = 1; w < wc; ++w) {
        const double start = end_prev > ready ? end_prev : ready;
        ready = (ready > end_prev ? ready : end_prev) + table_build;   // the table after this one reuses the buffer of the window before
        end_prev = start + window;
    }
    const int reuses = wc > 2 ? wc - 2 : 0;   // tables built into a buffer that consumers have to hand back first
    return double(waves) * (end_prev + per_reuse * reuses + (ks > 1 ? split_fixed + per_split * ks : 0.0));
}

int plan_lut(const bcq_desc *d, int B, int sm, bcq_plan *out)
{
    const int U = d->N / kUnitRows, W = d->K / kWindow;
    const int max_units = lut_max_units(d, B);
    const int rb_min = (U + max_units - 1) / max_units;
    double best = -1.0;
    const int cols = (B >= 2 && pairs_ok(d)) ? 2 : 1;
    const int cons = lut_consumer_warps(d->q, scale_subs(d->group), cols), per_job = lut_tiles_per_job(d->q, scale_subs(d->group), cols);
    for (int ks = (W + kMaxWindowsPerBlock - 1) / kMaxWindowsPerBlock; ks <= W && ks <= 64; ++ks) {
        // row blocks that fill whole waves of the GPU, or a little less than that, and the fewest possible
        for (int k = 0; k <= 16; ++k) {
            for (int j = 0; j <= (k == 1 ? 8 : 0); ++j) {
                const int rb = k == 0 ? rb_min : (k * sm) / ks - j;
                if (rb < rb_min || rb < 1 || rb > U || rb > kMaxRowBlocks) continue;
                if (j > 0 && 10LL * rb * ks < 7LL * sm) continue;   // the fit covers plans down to 0.7 of the GPU
                double c = lut_cost(U, W, rb, ks, sm, cons, per_job, cols);
                if (static_cast<long long>(rb) * ks > sm) c *= 1.25;   // (the fit saw single waves only: measured, a second wave costs more than its blocks)
                if (best < 0 || c < best) {
                    best = c;
                    out->kernel = 1;
                    out->row_blocks = rb;
                    out->k_splits = ks;
                    out->reserved = 0;
                }
            }
        }
    }
    return best < 0 ? BCQ_ERR_UNSUPPORTED_SHAPE : BCQ_OK;
}

// The same kind of model for the small-batch kernel, fitted to sweeps at 8 and 16 columns over the
// OPT-30B and Llama-2-70B layer shapes (pick within 0.5 % of the fastest measured plan on average, 3.5 %
// at worst): a round is one pair of row units per consumer warp; the combine grows with splits x rows x
// columns.
long long mma_cost(int U, int W, int rb, int ks, int sm, int B)
{
    const long long per_window = 300, round = 1500, per_pair = 200, per_split = 100, combine = 24;
    const long long waves = (static_cast<long long>(rb) * ks + sm - 1) / sm;
    const long long wc = (W + ks - 1) / ks;
    const long long units = (U + rb - 1) / rb;
    const long long pairs = (units + 1) / 2;
    long long rounds = (pairs + kMmaWarps - 1) / kMmaWarps;
    if (rounds < 1) rounds = 1;
    long long work = rounds * round + pairs * per_pair;
    if (B > 8) work += work / 2;   // a second MMA per expanded operand
    long long t = wc * (per_window + work);
    if (ks > 1) t += per_split * ks + combine * ks * units * B / 8;
    return waves * t;
}

int plan_mma(const bcq_desc *d, int sm, int B, bcq_plan *out)
{
    const int U = d->N / kUnitRows, W = d->K / kWindow;
    const int rb_min = (U + kMmaMaxUnitsPerBlock - 1) / kMmaMaxUnitsPerBlock;
    long long best = -1;
    for (int ks = (W + kMaxWindowsPerBlock - 1) / kMaxWindowsPerBlock; ks <= W && ks <= 64; ++ks) {
        for (int k = 0; k <= 16; ++k) {
            for (int j = 0; j <= (k == 1 ? 8 : 0); ++j) {
                const int rb = k == 0 ? rb_min : (k * sm) / ks - j;
                if (rb < rb_min || rb < 1 || rb > U || rb > kMaxRowBlocks) continue;
                if (j > 0 && 10LL * rb * ks < 7LL * sm) continue;
                const long long c = mma_cost(U, W, rb, ks, sm, B);
                if (best < 0 || c < best) {
                    best = c;
                    out->kernel = 2;
                    out->row_blocks = rb;
                    out->k_splits = ks;
                    out->reserved = 0;
                }
            }
        }
    }
    return best < 0 ? BCQ_ERR_UNSUPPORTED_SHAPE : BCQ_OK;
}

// The search above costs a few microseconds; products are launched far more often than shapes change,
// so the last plans are remembered (a small table, replaced round-robin).
int cached_plan(const bcq_desc *d, int B, int sm, bcq_plan *out)
{
    struct Entry {
        bcq_desc d;
        int B, sm;
        bcq_plan plan;
    };
    static Entry table[32];
    static int used = 0, next = 0;
    static std::mutex lock;
    {
        std::lock_guard<std::mutex> g(lock);
        for (int i = 0; i < used; ++i) {
            const Entry &e = table[i];
            if (e.B == B && e.sm == sm && e.d.N == d->N && e.d.K == d->K && e.d.q == d->q && e.d.group == d->group &&
                e.d.layout == d->layout) {
                *out = e.plan;
                return BCQ_OK;
            }
        }
    }
    const int rc = B < small_batch_min(d) ? plan_lut(d, B, sm, out) : plan_mma(d, sm, B, out);
    if (rc != BCQ_OK) return rc;
    std::lock_guard<std::mutex> g(lock);
    Entry &e = table[next];
    e.d = *d, e.B = B, e.sm = sm, e.plan = *out;
    next = (next + 1) % 32;
    if (used < 32) ++used;
    return BCQ_OK;
}

// B: the number of columns the plan is for (kernel 1 handles one column per launch, kernel 2 needs 2..16)
int check_plan(const bcq_desc *d, const bcq_plan *p, int B)
{
    if (p->kernel == 0) return BCQ_OK;
    if ((p->kernel != 1 && p->kernel != 2) || !lut_kernel_covers(d)) return BCQ_ERR_INVALID_ARG;
    if (p->reserved & ~(BCQ_PLAN_TEST_SHORT_WAITS | BCQ_PLAN_TEST_WITHHOLD_TABLE)) return BCQ_ERR_INVALID_ARG;
    if (p->reserved != 0 && d->group != 0 && d->group != 128) return BCQ_ERR_INVALID_ARG;   // the test instantiations
    if (p->kernel == 2 && (B < 2 || !mma_ok(d))) return BCQ_ERR_INVALID_ARG;
    const int U = d->N / kUnitRows, W = d->K / kWindow;
    const int max_units = p->kernel == 1 ? lut_max_units(d, B) : kMmaMaxUnitsPerBlock;
    if (p->row_blocks < 1 || p->row_blocks > U || p->row_blocks > kMaxRowBlocks) return BCQ_ERR_INVALID_ARG;
    if (p->k_splits < 1 || p->k_splits > W) return BCQ_ERR_INVALID_ARG;
    if ((W + p->k_splits - 1) / p->k_splits > kMaxWindowsPerBlock) return BCQ_ERR_INVALID_ARG;
    if ((U + p->row_blocks - 1) / p->row_blocks > max_units) return BCQ_ERR_INVALID_ARG;
    return BCQ_OK;
}

size_t plan_workspace(const bcq_desc *d, const bcq_plan *p, int B)
{
    if (p->k_splits <= 1) return 0;
    // kernel 1 runs one column per launch, or two when the scales live in the tiles
    if (p->kernel == 1) return lut_workspace_bytes(d->N, (B >= 2 && pairs_ok(d)) ? 2 : 1);
    if (p->kernel == 2) return kCounterBytes + size_t(p->k_splits) * B * d->N * sizeof(float);
    return 0;
}

// cols: 1, or 2 (lookup-table kernel with the scales in the tiles): x and y hold two columns
int run_gemv(const bcq_desc *desc, const bcq_plan *plan, const void *packed, const uint16_t *alpha, const uint16_t *z,
             const uint16_t *x, uint16_t *y, void *ws, size_t ws_bytes, void *stream, int cols = 1,
             const bcq_epilogue *epilogue = nullptr, bool bf16 = false)
{
    if (!packed || !x || !y) return BCQ_ERR_INVALID_ARG;
    if (interleaved(desc))
        alpha = z = nullptr;
    else if (!alpha || !z)
        return BCQ_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(alpha, 16) || !aligned(z, 16) || !aligned(x, 16) || !aligned(y, 2))
        return BCQ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (plan->kernel == 0) {
        if (epilogue || bf16) return BCQ_ERR_INVALID_ARG;   // the fused and bfloat16 forms exist in the lookup-table kernel only
        e = launch_generic(*desc, packed, alpha, z, x, y, 1, st);
    } else {
        const size_t need = plan_workspace(desc, plan, cols);
        if (need > 0) {
            if (!ws) return BCQ_ERR_INVALID_ARG;
            if (!aligned(ws, 16)) return BCQ_ERR_MISALIGNED;
            if (ws_bytes < need) return BCQ_ERR_WORKSPACE_TOO_SMALL;
        }
        e = launch_lut_gemv(*desc, *plan, packed, alpha, z, x, y, need ? ws : nullptr, st, cols, epilogue, bf16);
    }
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

// Share the plan's row blocks out among operands of N[o] rows in proportion to their rows (largest remainders,
// at least one each); BCQ_ERR_INVALID_ARG when that is impossible or a block would get too many row units.
int share_row_blocks(const bcq_desc *d, const bcq_plan *plan, const int32_t *N, int count, int32_t *out)
{
    const int max_units = lut_max_units(d, 1);
    long long total = 0;
    for (int o = 0; o < count; ++o) {
        if (N[o] <= 0 || N[o] % kUnitRows != 0) return BCQ_ERR_INVALID_ARG;
        total += N[o];
    }
    if (total != d->N || plan->row_blocks < count) return BCQ_ERR_INVALID_ARG;
    long long rem[kLutMaxOperands];
    int given = 0;
    for (int o = 0; o < count; ++o) {
        const long long share = static_cast<long long>(plan->row_blocks) * N[o];
        out[o] = static_cast<int32_t>(share / total);
        rem[o] = share % total;
        if (out[o] < 1) out[o] = 1, rem[o] = -1;
        given += out[o];
    }
    while (given < plan->row_blocks) {   // hand the rest to the largest remainders (ties: the earlier operand)
        int best = 0;
        for (int o = 1; o < count; ++o)
            if (rem[o] > rem[best]) best = o;
        ++out[best], rem[best] = -1, ++given;
        bool all_used = true;
        for (int o = 0; o < count; ++o) all_used = all_used && rem[o] < 0;
        if (all_used)
            for (int o = 0; o < count; ++o) rem[o] = N[o];   // more left than operands: go round again by size
    }
    if (given != plan->row_blocks) return BCQ_ERR_INVALID_ARG;   // the one-block minimum exceeded the plan
    for (int o = 0; o < count; ++o) {
        const int U = N[o] / kUnitRows;
        if (out[o] > U || (U + out[o] - 1) / out[o] > max_units) return BCQ_ERR_INVALID_ARG;
    }
    return BCQ_OK;
}

int run_multi(const bcq_desc *desc, const bcq_plan *plan, const bcq_operand *ops, int count, const uint16_t *x, void *ws,
              size_t ws_bytes, void *stream)
{
    if (!ops || !x || count < 1 || count > kLutMaxOperands) return BCQ_ERR_INVALID_ARG;
    if (!lut_kernel_covers(desc) || plan->kernel != 1) return BCQ_ERR_INVALID_ARG;
    if (count > 1 && desc->group != 0 && desc->group != 128) return BCQ_ERR_INVALID_ARG;   // several operands: groups of 128 or per row
    int32_t N[kLutMaxOperands], rb[kLutMaxOperands];
    for (int o = 0; o < count; ++o) N[o] = ops[o].N;
    int rc = share_row_blocks(desc, plan, N, count, rb);
    if (rc != BCQ_OK) return rc;
    LutOperand lo[kLutMaxOperands];
    for (int o = 0; o < count; ++o) {
        const bcq_operand &op = ops[o];
        if (!op.packed_dev || !op.y_dev) return BCQ_ERR_INVALID_ARG;
        lo[o].alpha = lo[o].z = nullptr;
        if (!interleaved(desc)) {
            if (!op.alpha_dev || !op.z_dev) return BCQ_ERR_INVALID_ARG;
            lo[o].alpha = op.alpha_dev, lo[o].z = op.z_dev;
        }
        if (!aligned(op.packed_dev, 16) || !aligned(lo[o].alpha, 16) || !aligned(lo[o].z, 16) || !aligned(op.y_dev, 2))
            return BCQ_ERR_MISALIGNED;
        lo[o].packed = op.packed_dev, lo[o].y = op.y_dev, lo[o].N = op.N, lo[o].row_blocks = rb[o];
    }
    if (!aligned(x, 16)) return BCQ_ERR_MISALIGNED;
    const size_t need = plan_workspace(desc, plan, 1);
    if (need > 0) {
        if (!ws) return BCQ_ERR_INVALID_ARG;
        if (!aligned(ws, 16)) return BCQ_ERR_MISALIGNED;
        if (ws_bytes < need) return BCQ_ERR_WORKSPACE_TOO_SMALL;
    }
    const cudaError_t e = launch_lut_multi(*desc, *plan, lo, count, x, need ? ws : nullptr, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

// The host-side table of the linear-int -> binary-code conversion (Eq. fuse_step2, Eq. round):
// plane weights m_j and, for every step-1 integer, the code of the nearest reachable integer.
int merge_table(int q, int n_bits, const uint8_t *bit_to_plane, double (&weight)[4], uint8_t (&code_of_int)[256])
{
    // A sign pattern (code) drives all step-1 bits of a plane together, so the integers it can
    // reach are those whose binary digit (i-1) equals the code's bit for the plane of step-1 bit i.
    for (int j = 0; j < 4; ++j) weight[j] = 0.0;
    for (int i = 0; i < n_bits; ++i) {
        if (bit_to_plane[i] >= q) return BCQ_ERR_INVALID_ARG;
        weight[bit_to_plane[i]] += double(1u << i) * 0.5;  // step-1 bit i+1 weighs 2^(i-1)
    }
    for (int j = 0; j < q; ++j)
        if (weight[j] == 0.0) return BCQ_ERR_INVALID_ARG;
    int reach[16];
    for (int c = 0; c < (1 << q); ++c) {
        int v = 0;
        for (int i = 0; i < n_bits; ++i) v |= ((c >> bit_to_plane[i]) & 1) << i;
        reach[c] = v;
    }
    for (int t = 0; t < 256; ++t) {
        int best = 0;
        for (int c = 1; c < (1 << q); ++c) {
            const int dc = abs(t - reach[c]), db = abs(t - reach[best]);
            if (dc < db || (dc == db && reach[c] < reach[best])) best = c;
        }
        code_of_int[t] = uint8_t(best);
    }
    return BCQ_OK;
}

// lut[v] = the integer the planes of bit_to_plane reach that is nearest to the step-1 integer v (ties: the smaller)
int nearest_reachable(int q, int n_bits, const uint8_t *bit_to_plane, float *lut /*[64]*/)
{
    double weight[4];
    uint8_t code_of_int[256];
    const int rc = merge_table(q, n_bits, bit_to_plane, weight, code_of_int);
    if (rc != BCQ_OK) return rc;
    for (int v = 0; v < 64; ++v) {
        int reach = 0;
        if (v < (1 << n_bits))
            for (int i = 0; i < n_bits; ++i) reach |= ((code_of_int[v] >> bit_to_plane[i]) & 1) << i;
        lut[v] = float(reach);
    }
    return BCQ_OK;
}

// bit_to_plane arrays of all splits of n bits into q non-empty planes: planes numbered by their lowest bit,
// arrays in lexicographic order.  Returns the count; writes the index-th array when out is given.
int enumerate_partitions(int n, int q, int index, uint8_t *out)
{
    uint8_t cur[8];
    int count = 0;
    // iterative depth-first walk over restricted-growth strings
    int pos = 0, used[9];
    used[0] = 0;
    cur[0] = 0;
    int next[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    while (pos >= 0) {
        const int limit = used[pos] + 1 < q ? used[pos] + 1 : q;   // values 0 .. limit-1 are allowed here
        if (next[pos] >= limit) {
            --pos;
            continue;
        }
        cur[pos] = uint8_t(next[pos]++);
        const int u = cur[pos] + 1 > used[pos] ? cur[pos] + 1 : used[pos];
        if (pos == n - 1) {
            if (u == q) {
                if (out && count == index)
                    for (int i = 0; i < n; ++i) out[i] = cur[i];
                ++count;
            }
        } else {
            ++pos;
            used[pos] = u;
            next[pos] = 0;
        }
    }
    return count;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Scale factors are searched several per launch (a launch of 128-row blocks x groups of candidates alone leaves the
// last wave of blocks partly empty): step 1's outputs of kSearchScalesPerLaunch factors sit side by side.
constexpr int kSearchScalesPerLaunch = 8;
struct SearchLayout {
    size_t lut, w_int, S, qbias, packed, alpha, z, err, err_rows, total;
    size_t w_int_each, S_each;   // bytes of one scale factor's W_int; of its S (and of its qbias)
    int together;                // scale factors per launch
};
SearchLayout search_layout(const bcq_desc &d, int P, int n_scales, bool own_rows)
{
    SearchLayout L;
    const size_t G = size_t(n_groups(d));
    L.together = n_scales < kSearchScalesPerLaunch ? n_scales : kSearchScalesPerLaunch;
    L.w_int_each = size_t(d.N) * d.K, L.S_each = round_up(size_t(d.N) * G * 2, 256);
    size_t at = 0;
    L.lut = at, at += round_up(size_t(P) * 64 * sizeof(float), 256);
    L.w_int = at, at += round_up(L.w_int_each * L.together, 256);
    L.S = at, at += L.S_each * L.together;
    L.qbias = at, at += L.S_each * L.together;
    L.packed = at, at += round_up(size_t(d.q) * d.N * (d.K / 8), 256);
    L.alpha = at, at += round_up(size_t(d.q) * d.N * G * 2, 256);
    L.z = at, at += round_up(size_t(d.N) * G * 2, 256);
    L.err = at, at += round_up(size_t(n_scales) * P * sizeof(double), 256);
    L.err_rows = at, at += own_rows ? round_up(size_t(L.together) * P * d.N * sizeof(float), 256) : 0;
    L.total = at;
    return L;
}

int check_search(const bcq_desc *desc, int T, int n_bits, int P, int n_scales)
{
    const int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (n_bits < 1 || n_bits > 6 || desc->q > n_bits || P < 1 || P > 4096 || n_scales < 1 || n_scales > 4096) return BCQ_ERR_INVALID_ARG;
    if (T < 16 || T > 65536 || T % 16 != 0) return BCQ_ERR_INVALID_ARG;
    if (desc->K % 64 != 0 || (desc->group != 0 && desc->group % 64 != 0)) return BCQ_ERR_UNSUPPORTED_SHAPE;
    return BCQ_OK;
}

}  // namespace

extern "C" {

int bcq_version(void) { return BCQ_VERSION; }

const char *bcq_last_cuda_error(void) { return g_cuda_error; }

const char *bcq_status_string(int s)
{
    switch (s) {
        case BCQ_OK: return "ok";
        case BCQ_ERR_INVALID_ARG: return "invalid argument";
        case BCQ_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case BCQ_ERR_MISALIGNED: return "misaligned pointer";
        case BCQ_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case BCQ_ERR_CUDA: return "CUDA error";
        case BCQ_ERR_SCRATCH_LIMIT: return "product needs more scratch than bcq_gemv_noalloc has built in";
        case BCQ_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    }
    return "unknown status";
}

int bcq_poll_status(void)
{
    int v = 0;
    int w = 0;
    int u = 0;
    cudaError_t e = cudaDeviceSynchronize();   // kernels on non-blocking streams included
    if (e == cudaSuccess) e = lut_status_take(&v);
    if (e == cudaSuccess) e = mma_status_take(&w);
    if (e == cudaSuccess) e = search_status_take(&u);
    if (e != cudaSuccess) return cuda_fail(e);
    if (v != 0 || w != 0 || u != 0) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: bounded wait %d ran out",
                 v ? "lut_gemv_kernel" : (w ? "mma_gemm_kernel" : "search_error_kernel"), v ? v : (w ? w : u));
        return BCQ_ERR_TIMEOUT;
    }
    return BCQ_OK;
}

int bcq_check_desc(const bcq_desc *desc) { return check_desc(desc); }

size_t bcq_packed_bytes(const bcq_desc *d)
{
    if (check_desc(d) != BCQ_OK) return 0;
    size_t bytes = size_t(d->q) * d->N * (d->K / 8);
    if (interleaved(d)) bytes += (size_t(d->q) + 1) * d->N * n_groups(*d) * sizeof(uint16_t);
    return bytes;
}
size_t bcq_alpha_elems(const bcq_desc *d) { return check_desc(d) == BCQ_OK ? size_t(d->q) * d->N * n_groups(*d) : 0; }
size_t bcq_offset_elems(const bcq_desc *d) { return check_desc(d) == BCQ_OK ? size_t(d->N) * n_groups(*d) : 0; }

int bcq_plan_default(const bcq_desc *desc, int B, int sm_count, bcq_plan *out)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!out || B < 1 || B > 16) return BCQ_ERR_INVALID_ARG;
    out->kernel = 0;
    out->row_blocks = (desc->N + 7) / 8;
    out->k_splits = 1;
    out->reserved = 0;
    if (lut_kernel_covers(desc)) {
        if (sm_count <= 0) {
            rc = device_sm_count(&sm_count);
            if (rc != BCQ_OK) return rc;
        }
        return cached_plan(desc, B, sm_count, out);
    }
    return BCQ_OK;
}

size_t bcq_workspace_bytes(const bcq_desc *desc, int B, const bcq_plan *plan)
{
    bcq_plan def;
    if (check_desc(desc) != BCQ_OK) return 0;
    if (!plan) {
        if (bcq_plan_default(desc, B, 0, &def) != BCQ_OK) return 0;
        plan = &def;
    }
    if (B < 1 || B > 16 || check_plan(desc, plan, B) != BCQ_OK) return 0;
    return plan_workspace(desc, plan, B);
}

int bcq_workspace_init(void *ws, size_t bytes, void *stream)
{
    if (bytes == 0) return BCQ_OK;
    if (!ws) return BCQ_ERR_INVALID_ARG;
    cudaError_t e = cudaMemsetAsync(ws, 0, bytes, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_merge_linear(const bcq_desc *desc, const uint8_t *w_int, const uint16_t *S, const uint16_t *qbias, int n_bits,
                     const uint8_t *bit_to_plane, uint8_t *codes, uint16_t *alpha, uint16_t *z, void *stream)
{
    bcq_desc d;
    if (!desc) return BCQ_ERR_INVALID_ARG;
    d = *desc;
    d.layout = BCQ_LAYOUT_CANONICAL;
    int rc = check_desc(&d);
    if (rc != BCQ_OK) return rc;
    if (!w_int || !S || !qbias || !bit_to_plane || !codes || !alpha || !z) return BCQ_ERR_INVALID_ARG;
    if (n_bits < 1 || n_bits > 8 || d.q > n_bits) return BCQ_ERR_INVALID_ARG;
    if (!aligned(w_int, 16) || !aligned(codes, 16) || !aligned(S, 2) || !aligned(qbias, 2) || !aligned(alpha, 2) ||
        !aligned(z, 2))
        return BCQ_ERR_MISALIGNED;

    double weight[4];
    uint8_t code_of_int[256];
    rc = merge_table(d.q, n_bits, bit_to_plane, weight, code_of_int);
    if (rc != BCQ_OK) return rc;
    cudaError_t e = launch_merge(d, w_int, S, qbias, n_bits, code_of_int, weight, codes, alpha, z,
                                 static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_quantize_rtn(const bcq_desc *desc, const uint16_t *W, int n_bits, const uint8_t *bit_to_plane, double s_factor,
                     uint16_t *S, uint16_t *qbias, uint8_t *w_int, void *packed, uint16_t *alpha, uint16_t *z, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!W || !bit_to_plane || !S || !qbias || !packed) return BCQ_ERR_INVALID_ARG;
    if (n_bits < 1 || n_bits > 8 || desc->q > n_bits) return BCQ_ERR_INVALID_ARG;
    if (!(s_factor > 0.0) || !(s_factor < 1e30)) return BCQ_ERR_INVALID_ARG;
    if (interleaved(desc))
        alpha = z = nullptr;
    else if (!alpha || !z)
        return BCQ_ERR_INVALID_ARG;
    if (!aligned(W, 16) || !aligned(packed, 16) || !aligned(w_int, 8) || !aligned(S, 2) || !aligned(qbias, 2) ||
        !aligned(alpha, 2) || !aligned(z, 2))
        return BCQ_ERR_MISALIGNED;
    double weight[4];
    uint8_t code_of_int[256];
    rc = merge_table(desc->q, n_bits, bit_to_plane, weight, code_of_int);
    if (rc != BCQ_OK) return rc;
    cudaError_t e = launch_quantize_rtn(W, n_bits, s_factor, code_of_int, weight, S, qbias, w_int,
                                        make_view(*desc, packed, alpha, z), static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_pack(const bcq_desc *desc, const uint8_t *codes, const uint16_t *alpha_in, const uint16_t *z_in, void *packed,
             uint16_t *alpha_out, uint16_t *z_out, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!codes || !packed) return BCQ_ERR_INVALID_ARG;
    bool scales;
    if (interleaved(desc)) {
        if (!alpha_in || !z_in) return BCQ_ERR_INVALID_ARG;  // the tiles carry the scales
        alpha_out = z_out = nullptr;
        scales = true;
    } else {
        scales = alpha_in || z_in || alpha_out || z_out;
        if (scales && !(alpha_in && z_in && alpha_out && z_out)) return BCQ_ERR_INVALID_ARG;
    }
    if (!aligned(codes, 16) || !aligned(packed, 16) || !aligned(alpha_in, 2) || !aligned(z_in, 2) ||
        !aligned(alpha_out, 2) || !aligned(z_out, 2))
        return BCQ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const View dst = make_view(*desc, packed, alpha_out, z_out);
    cudaError_t e = launch_pack(codes, dst, st);
    if (e == cudaSuccess && scales) {
        bcq_desc canon = *desc;
        canon.layout = BCQ_LAYOUT_CANONICAL;
        e = launch_permute_scales(make_view(canon, nullptr, alpha_in, z_in), dst, st);
    }
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_repack(const bcq_desc *src, const void *packed_src, const uint16_t *alpha_src, const uint16_t *z_src,
               const bcq_desc *dst, void *packed_dst, uint16_t *alpha_dst, uint16_t *z_dst, void *stream)
{
    int rc = check_desc(src);
    if (rc != BCQ_OK) return rc;
    rc = check_desc(dst);
    if (rc != BCQ_OK) return rc;
    if (!same_problem(src, dst)) return BCQ_ERR_INVALID_ARG;
    if (!packed_src || !packed_dst || packed_src == packed_dst) return BCQ_ERR_INVALID_ARG;
    if (interleaved(src)) alpha_src = z_src = nullptr;
    if (interleaved(dst)) alpha_dst = z_dst = nullptr;
    if ((alpha_src == nullptr) != (z_src == nullptr) || (alpha_dst == nullptr) != (z_dst == nullptr)) return BCQ_ERR_INVALID_ARG;
    const bool have_scales = interleaved(src) || alpha_src;
    const bool want_scales = interleaved(dst) || alpha_dst;
    if (interleaved(dst) && !have_scales) return BCQ_ERR_INVALID_ARG;  // a tiled operand cannot exist without its scales
    if ((alpha_src && alpha_src == alpha_dst) || (z_src && z_src == z_dst)) return BCQ_ERR_INVALID_ARG;
    if (!aligned(packed_src, 16) || !aligned(packed_dst, 16) || !aligned(alpha_src, 2) || !aligned(alpha_dst, 2) ||
        !aligned(z_src, 2) || !aligned(z_dst, 2))
        return BCQ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const View vs = make_view(*src, packed_src, alpha_src, z_src), vd = make_view(*dst, packed_dst, alpha_dst, z_dst);
    cudaError_t e = launch_permute_planes(vs, vd, st);
    if (e == cudaSuccess && have_scales && want_scales) e = launch_permute_scales(vs, vd, st);
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_gemv_plan(const bcq_desc *desc, const bcq_plan *plan, const void *packed, const uint16_t *alpha,
                  const uint16_t *z, const uint16_t *x, uint16_t *y, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!plan) return BCQ_ERR_INVALID_ARG;
    rc = check_plan(desc, plan, 1);
    if (rc != BCQ_OK) return rc;
    return run_gemv(desc, plan, packed, alpha, z, x, y, ws, ws_bytes, stream);
}

int bcq_gemv(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z, const uint16_t *x,
             uint16_t *y, void *ws, size_t ws_bytes, void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, 1, 0, &plan);
    if (rc != BCQ_OK) return rc;
    return run_gemv(desc, &plan, packed, alpha, z, x, y, ws, ws_bytes, stream);
}

int bcq_gemv_bf16(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z, const uint16_t *x,
                  uint16_t *y, const bcq_epilogue *epilogue, void *ws, size_t ws_bytes, void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, 1, 0, &plan);
    if (rc != BCQ_OK) return rc;
    if (epilogue) {
        if (epilogue->reserved != 0 || epilogue->activation < BCQ_ACT_NONE || epilogue->activation > BCQ_ACT_SILU) return BCQ_ERR_INVALID_ARG;
        if (!aligned(epilogue->bias_dev, 2) || !aligned(epilogue->residual_dev, 2)) return BCQ_ERR_MISALIGNED;
    }
    return run_gemv(desc, &plan, packed, alpha, z, x, y, ws, ws_bytes, stream, 1, epilogue, true);
}

int bcq_gemv_dequant(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z, const uint16_t *x,
                     uint16_t *y, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!lut_kernel_covers(desc) || (desc->group != 0 && desc->group != 128)) return BCQ_ERR_INVALID_ARG;
    if (!packed || !x || !y) return BCQ_ERR_INVALID_ARG;
    if (interleaved(desc))
        alpha = z = nullptr;
    else if (!alpha || !z)
        return BCQ_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(alpha, 2) || !aligned(z, 2) || !aligned(x, 16) || !aligned(y, 2)) return BCQ_ERR_MISALIGNED;
    const cudaError_t e = launch_dequant_gemv(*desc, packed, alpha, z, x, y, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_gemv_fused(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z, const uint16_t *x,
                   uint16_t *y, const bcq_epilogue *epilogue, void *ws, size_t ws_bytes, void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, 1, 0, &plan);
    if (rc != BCQ_OK) return rc;
    if (!epilogue || epilogue->reserved != 0 || epilogue->activation < BCQ_ACT_NONE || epilogue->activation > BCQ_ACT_SILU)
        return BCQ_ERR_INVALID_ARG;
    if (!aligned(epilogue->bias_dev, 2) || !aligned(epilogue->residual_dev, 2)) return BCQ_ERR_MISALIGNED;
    return run_gemv(desc, &plan, packed, alpha, z, x, y, ws, ws_bytes, stream, 1, epilogue);
}

int bcq_multi_row_blocks(const bcq_desc *desc, const bcq_plan *plan, const int32_t *N, int count, int32_t *out)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!plan || !N || !out || count < 1 || count > kLutMaxOperands) return BCQ_ERR_INVALID_ARG;
    rc = check_plan(desc, plan, 1);
    if (rc != BCQ_OK) return rc;
    if (plan->kernel != 1) return BCQ_ERR_INVALID_ARG;
    return share_row_blocks(desc, plan, N, count, out);
}

int bcq_gemv_multi_plan(const bcq_desc *desc, const bcq_plan *plan, const bcq_operand *ops, int count, const uint16_t *x,
                        void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!plan) return BCQ_ERR_INVALID_ARG;
    if (plan->kernel != 1 || !lut_kernel_covers(desc)) return BCQ_ERR_INVALID_ARG;
    // the limits on row units per block apply per operand (share_row_blocks); the rest as for one product
    if (plan->reserved != 0 && count > 1) return BCQ_ERR_INVALID_ARG;   // the test bits apply to single products
    if (plan->reserved & ~(BCQ_PLAN_TEST_SHORT_WAITS | BCQ_PLAN_TEST_WITHHOLD_TABLE)) return BCQ_ERR_INVALID_ARG;
    const int W = desc->K / kWindow;
    if (plan->row_blocks < 1 || plan->row_blocks > kMaxRowBlocks || plan->k_splits < 1 || plan->k_splits > W ||
        (W + plan->k_splits - 1) / plan->k_splits > kMaxWindowsPerBlock)
        return BCQ_ERR_INVALID_ARG;
    return run_multi(desc, plan, ops, count, x, ws, ws_bytes, stream);
}

int bcq_gemv_multi(const bcq_desc *desc, const bcq_operand *ops, int count, const uint16_t *x, void *ws, size_t ws_bytes,
                   void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, 1, 0, &plan);
    if (rc != BCQ_OK) return rc;
    if (plan.kernel != 1 || !ops || count < 1 || count > kLutMaxOperands) return BCQ_ERR_INVALID_ARG;
    // the default plan of the rows taken together, with more row blocks if an operand would not fit its share
    int32_t N[kLutMaxOperands], rb[kLutMaxOperands];
    for (int o = 0; o < count; ++o) N[o] = ops[o].N;
    while ((rc = share_row_blocks(desc, &plan, N, count, rb)) != BCQ_OK && plan.row_blocks < desc->N / kUnitRows &&
           plan.row_blocks < kMaxRowBlocks)
        ++plan.row_blocks;
    if (rc != BCQ_OK) return rc;
    return run_multi(desc, &plan, ops, count, x, ws, ws_bytes, stream);
}

int bcq_gemm_smallbatch_plan(const bcq_desc *desc, const bcq_plan *plan, const void *packed, const uint16_t *alpha,
                             const uint16_t *z, const uint16_t *X, uint16_t *Y, int B, void *ws, size_t ws_bytes,
                             void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!plan || B < 1 || B > 16) return BCQ_ERR_INVALID_ARG;
    rc = check_plan(desc, plan, B);
    if (rc != BCQ_OK) return rc;
    if (!packed || !X || !Y) return BCQ_ERR_INVALID_ARG;
    if (interleaved(desc))
        alpha = z = nullptr;
    else if (!alpha || !z)
        return BCQ_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(alpha, 16) || !aligned(z, 16) || !aligned(X, 16) || !aligned(Y, 2))
        return BCQ_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (plan->kernel == 1) {
        // The lookup-table kernel column by column -- or, with the scales in the tiles, two columns at a
        // time (tables that hold both columns' sums side by side: one pass over the weights per pair).
        const int step = pairs_ok(desc) ? 2 : 1;
        for (int b = 0; b < B; b += step) {
            const int cols = (b + step <= B) ? step : 1;
            rc = run_gemv(desc, plan, packed, alpha, z, X + size_t(b) * desc->K, Y + size_t(b) * desc->N, ws, ws_bytes, stream,
                          cols);
            if (rc != BCQ_OK) return rc;
        }
        return BCQ_OK;
    }
    cudaError_t e;
    if (plan->kernel == 2) {
        const size_t need = plan_workspace(desc, plan, B);
        if (need > 0) {
            if (!ws) return BCQ_ERR_INVALID_ARG;
            if (!aligned(ws, 16)) return BCQ_ERR_MISALIGNED;
            if (ws_bytes < need) return BCQ_ERR_WORKSPACE_TOO_SMALL;
        }
        e = launch_mma_gemm(*desc, *plan, packed, alpha, z, X, Y, B, need ? ws : nullptr, st);
    } else {
        e = launch_generic(*desc, packed, alpha, z, X, Y, B, st);
    }
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_gemm_smallbatch(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z,
                        const uint16_t *X, uint16_t *Y, int B, void *ws, size_t ws_bytes, void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, B, 0, &plan);
    if (rc != BCQ_OK) return rc;
    return bcq_gemm_smallbatch_plan(desc, &plan, packed, alpha, z, X, Y, B, ws, ws_bytes, stream);
}

int bcq_gemv_host(const bcq_desc *desc, const void *packed, const uint16_t *alpha, const uint16_t *z,
                  const uint16_t *x_host, uint16_t *y_host, uint16_t *x_stage, uint16_t *y_stage, void *ws,
                  size_t ws_bytes, void *stream)
{
    int rc = check_desc(desc);
    if (rc != BCQ_OK) return rc;
    if (!x_host || !y_host || !x_stage || !y_stage) return BCQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(x_stage, x_host, size_t(desc->K) * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
    // Page-locked host memory is addressable from the device: the kernel then stores y there itself
    // (N fp16 values over the bus, once) and the copy back, a stream operation of its own, is saved.
    cudaPointerAttributes attr;
    uint16_t *y_direct = nullptr;
    if (cudaPointerGetAttributes(&attr, y_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
        y_direct = static_cast<uint16_t *>(attr.devicePointer);
    else
        (void)cudaGetLastError();   // pageable memory is not an error here
    rc = bcq_gemv(desc, packed, alpha, z, x_stage, y_direct ? y_direct : y_stage, ws, ws_bytes, stream);
    if (rc != BCQ_OK || y_direct) return rc;
    e = cudaMemcpyAsync(y_host, y_stage, size_t(desc->N) * 2, cudaMemcpyDeviceToHost, st);
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

int bcq_partition_count(int n_bits, int q)
{
    if (n_bits < 1 || n_bits > 8 || q < 1 || q > 4 || q > n_bits) return 0;
    return enumerate_partitions(n_bits, q, -1, nullptr);
}

int bcq_partition_get(int n_bits, int q, int index, uint8_t *bit_to_plane_out)
{
    if (!bit_to_plane_out || n_bits < 1 || n_bits > 8 || q < 1 || q > 4 || q > n_bits) return BCQ_ERR_INVALID_ARG;
    if (index < 0 || index >= enumerate_partitions(n_bits, q, -1, nullptr)) return BCQ_ERR_INVALID_ARG;
    enumerate_partitions(n_bits, q, index, bit_to_plane_out);
    return BCQ_OK;
}

int bcq_reexplore_factors(int n_bits, int count, double *s_factors_out)
{
    if (!s_factors_out || n_bits < 2 || n_bits > 8 || count < 1) return BCQ_ERR_INVALID_ARG;
    const double full = double((1u << n_bits) - 1u);
    const double lo = full / double((1u << (n_bits + 1)) - 1u), hi = full / double((1u << (n_bits - 1)) - 1u);
    for (int i = 0; i < count; ++i) s_factors_out[i] = lo + (hi - lo) * double(i + 1) / double(count + 1);
    return BCQ_OK;
}

size_t bcq_grid_search_workspace(const bcq_desc *desc, int T, int n_bits, int P, int n_scales, int rows_given)
{
    bcq_desc d;
    if (!desc) return 0;
    d = *desc;
    d.layout = BCQ_LAYOUT_CANONICAL;
    if (check_search(&d, T, n_bits, P, n_scales) != BCQ_OK) return 0;
    return search_layout(d, P, n_scales, rows_given == 0).total;
}

int bcq_grid_search(const bcq_desc *desc, const uint16_t *W, const uint16_t *X, int T, int n_bits, const uint8_t *partitions,
                    int P, const double *s_factors, int n_scales, double *err, float *err_rows, int32_t *best, void *ws,
                    size_t ws_bytes, void *stream)
{
    if (!desc) return BCQ_ERR_INVALID_ARG;
    bcq_desc d = *desc;
    d.layout = BCQ_LAYOUT_CANONICAL;
    int rc = check_search(&d, T, n_bits, P, n_scales);
    if (rc != BCQ_OK) return rc;
    if (!W || !X || !partitions || !s_factors || !err || !best || !ws) return BCQ_ERR_INVALID_ARG;
    if (!aligned(W, 16) || !aligned(X, 16) || !aligned(err, 8) || !aligned(err_rows, 4) || !aligned(best, 4) || !aligned(ws, 256))
        return BCQ_ERR_MISALIGNED;
    const SearchLayout L = search_layout(d, P, n_scales, err_rows == nullptr);
    if (ws_bytes < L.total) return BCQ_ERR_WORKSPACE_TOO_SMALL;
    for (int s = 0; s < n_scales; ++s)
        if (!(s_factors[s] > 0.0) || !(s_factors[s] < 1e30)) return BCQ_ERR_INVALID_ARG;

    std::vector<float> lut(size_t(P) * 64);
    for (int c = 0; c < P; ++c) {
        rc = nearest_reachable(d.q, n_bits, partitions + size_t(c) * n_bits, lut.data() + size_t(c) * 64);
        if (rc != BCQ_OK) return rc;
    }
    double weight[4];
    uint8_t code_of_int[256];
    rc = merge_table(d.q, n_bits, partitions, weight, code_of_int);   // step 1 does not depend on the BCchoice: any will do
    if (rc != BCQ_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *base = static_cast<unsigned char *>(ws);
    float *lut_dev = reinterpret_cast<float *>(base + L.lut);
    uint8_t *w_int = base + L.w_int;
    uint16_t *S = reinterpret_cast<uint16_t *>(base + L.S), *qbias = reinterpret_cast<uint16_t *>(base + L.qbias);
    double *err_all = reinterpret_cast<double *>(base + L.err);
    // (pageable host memory: the copy has left the vector when the call returns)
    cudaError_t e = cudaMemcpyAsync(lut_dev, lut.data(), lut.size() * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
    const View scratch = make_view(d, base + L.packed, reinterpret_cast<uint16_t *>(base + L.alpha), reinterpret_cast<uint16_t *>(base + L.z));
    for (int s0 = 0; s0 < n_scales; s0 += L.together) {
        const int count = n_scales - s0 < L.together ? n_scales - s0 : L.together;
        for (int i = 0; i < count; ++i) {
            e = launch_quantize_rtn(W, n_bits, s_factors[s0 + i], code_of_int, weight, S + i * (L.S_each / 2), qbias + i * (L.S_each / 2),
                                    w_int + i * L.w_int_each, scratch, st, false);   // the search needs no packed operand
            if (e != cudaSuccess) return cuda_fail(e);
        }
        float *rows = err_rows ? err_rows + size_t(s0) * P * d.N : reinterpret_cast<float *>(base + L.err_rows);
        e = launch_search_errors(W, w_int, S, qbias, L.S_each / 2, X, d.N, d.K, d.group, T, n_bits, lut_dev, P, count, rows,
                                 err_all + size_t(s0) * P, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    e = launch_search_argmin(err_all, n_scales * P, P, best, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaMemcpyAsync(err, err_all, size_t(n_scales) * P * sizeof(double), cudaMemcpyDeviceToDevice, st);
    return e == cudaSuccess ? BCQ_OK : cuda_fail(e);
}

}  // extern "C"

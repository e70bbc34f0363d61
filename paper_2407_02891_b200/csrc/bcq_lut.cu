// Host side of the lookup-table BCQ GEMV: geometry queries, parameter marshalling and dispatch to the
// instantiations (bcq_lut_kernel.cuh holds the kernel; bcq_lut_q1.cu .. q4.cu instantiate it per plane count).
#include "bcq_lut_kernel.cuh"

namespace bcq {

cudaError_t launch_lut_q1(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st);
cudaError_t launch_lut_q2(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st);
cudaError_t launch_lut_q3(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st);
cudaError_t launch_lut_q4(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st);
cudaError_t lut_status_take_q1(int *status);
cudaError_t lut_status_take_q2(int *status);
cudaError_t lut_status_take_q3(int *status);
cudaError_t lut_status_take_q4(int *status);

template <int Q>
static void lut_geometry(int sub, int cols, int *cons, int *per_job)
{
    switch (sub * 4 + cols) {
        case 1: *cons = LutCfg<Q, 0, 1>::kCons, *per_job = LutCfg<Q, 0, 1>::kJ; break;
        case 5: *cons = LutCfg<Q, 1, 1>::kCons, *per_job = LutCfg<Q, 1, 1>::kJ; break;
        case 6: *cons = LutCfg<Q, 1, 2>::kCons, *per_job = LutCfg<Q, 1, 2>::kJ; break;
        case 9: *cons = LutCfg<Q, 2, 1>::kCons, *per_job = LutCfg<Q, 2, 1>::kJ; break;
        case 17: *cons = LutCfg<Q, 4, 1>::kCons, *per_job = LutCfg<Q, 4, 1>::kJ; break;
        default: *cons = 0, *per_job = 1; break;
    }
}
static void lut_geometry_any(int q, int sub, int cols, int *cons, int *per_job)
{
    *cons = 0, *per_job = 1;
    switch (q) {
        case 1: lut_geometry<1>(sub, cols, cons, per_job); break;
        case 2: lut_geometry<2>(sub, cols, cons, per_job); break;
        case 3: lut_geometry<3>(sub, cols, cons, per_job); break;
        case 4: lut_geometry<4>(sub, cols, cons, per_job); break;
    }
}
int lut_consumer_warps(int q, int sub, int cols)
{
    int cons, per_job;
    lut_geometry_any(q, sub, cols, &cons, &per_job);
    return cons;
}
int lut_tiles_per_job(int q, int sub, int cols)
{
    int cons, per_job;
    lut_geometry_any(q, sub, cols, &cons, &per_job);
    return per_job;
}

static cudaError_t launch_lut_any(int q, int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st)
{
    switch (q) {
        case 1: return launch_lut_q1(sub, cols, test, one, many, st);
        case 2: return launch_lut_q2(sub, cols, test, one, many, st);
        case 3: return launch_lut_q3(sub, cols, test, one, many, st);
        case 4: return launch_lut_q4(sub, cols, test, one, many, st);
    }
    return cudaErrorInvalidValue;
}

static void fill_common(LutOne &one, const bcq_desc &d, const bcq_plan &plan, const uint16_t *x, void *workspace)
{
    one.x = reinterpret_cast<const __half *>(x);
    one.accum = static_cast<unsigned long long *>(workspace);
    one.N = d.N;
    one.K = d.K;
    one.row_blocks = plan.row_blocks;
    one.k_splits = plan.k_splits;
    const int U = d.N / kUnitRows, W = d.K / kWindow;
    one.u_base = U / plan.row_blocks, one.u_rem = U % plan.row_blocks;   // (several operands: per operand, see launch_lut_multi)
    one.w_base = W / plan.k_splits, one.w_rem = W % plan.k_splits;
    one.test_flags = plan.reserved;
}

// cols = 1: y = W x.  cols = 2 (grouped scales only): x and y hold two columns, K and N elements apart.
// A plan with test bits set runs the test instantiation (one column only).
cudaError_t launch_lut_gemv(const bcq_desc &d, const bcq_plan &plan, const void *packed, const uint16_t *alpha,
                            const uint16_t *z, const uint16_t *x, uint16_t *y, void *workspace, cudaStream_t st, int cols,
                            const bcq_epilogue *epilogue, bool bf16)
{
    LutOne one = {};
    one.tiles = static_cast<const uint8_t *>(packed);
    one.alpha = reinterpret_cast<const __half *>(alpha);   // used with per-row scales only
    one.z = reinterpret_cast<const __half *>(z);
    one.y = reinterpret_cast<__half *>(y);
    fill_common(one, d, plan, x, workspace);
    if (bf16 && cols != 1) return cudaErrorInvalidValue;
    one.bf16 = bf16 ? 1 : 0;
    if (epilogue) {
        if (cols != 1) return cudaErrorInvalidValue;
        one.bias = reinterpret_cast<const __half *>(epilogue->bias_dev);
        one.residual = reinterpret_cast<const __half *>(epilogue->residual_dev);
        one.activation = epilogue->activation;
    }
    return launch_lut_any(d.q, scale_subs(d.group), cols, plan.reserved != 0, &one, nullptr, st);
}

// Several operands that share x in one launch (batch 1); d.N is the sum of their rows and ops[o].row_blocks the
// row blocks given to operand o (they add up to plan.row_blocks).  One operand is launch_lut_gemv.
cudaError_t launch_lut_multi(const bcq_desc &d, const bcq_plan &plan, const LutOperand *ops, int count, const uint16_t *x,
                             void *workspace, cudaStream_t st)
{
    if (count < 1 || count > kLutMaxOperands) return cudaErrorInvalidValue;
    int rows = 0, rb = 0;
    for (int o = 0; o < count; ++o) rows += ops[o].N, rb += ops[o].row_blocks;
    if (rows != d.N || rb != plan.row_blocks) return cudaErrorInvalidValue;
    if (count == 1) return launch_lut_gemv(d, plan, ops[0].packed, ops[0].alpha, ops[0].z, x, ops[0].y, workspace, st, 1);
    if (plan.reserved != 0) return cudaErrorInvalidValue;   // the test instantiation takes one operand
    LutMany many = {};
    rows = rb = 0;
    for (int o = 0; o < count; ++o) {
        many.tiles[o] = static_cast<const uint8_t *>(ops[o].packed);
        many.alpha[o] = reinterpret_cast<const __half *>(ops[o].alpha);   // used with per-row scales only
        many.z[o] = reinterpret_cast<const __half *>(ops[o].z);
        many.y[o] = reinterpret_cast<__half *>(ops[o].y);
        many.U[o] = ops[o].N / kUnitRows;
        many.u_base[o] = many.U[o] / ops[o].row_blocks;
        many.u_rem[o] = many.U[o] % ops[o].row_blocks;
        many.row0[o] = rows;
        many.rb_first[o] = rb;
        rows += ops[o].N;
        rb += ops[o].row_blocks;
    }
    for (int o = count; o <= kLutMaxOperands; ++o) many.rb_first[o] = rb;
    many.count = count;
    fill_common(many.one, d, plan, x, workspace);
    return launch_lut_any(d.q, scale_subs(d.group), 1, false, nullptr, &many, st);
}

// Read and clear the device status words of the kernels (one per translation unit that instantiates them).
cudaError_t lut_status_take(int *status)
{
    int v[4] = {0, 0, 0, 0};
    cudaError_t e = lut_status_take_q1(&v[0]);
    if (e == cudaSuccess) e = lut_status_take_q2(&v[1]);
    if (e == cudaSuccess) e = lut_status_take_q3(&v[2]);
    if (e == cudaSuccess) e = lut_status_take_q4(&v[3]);
    *status = v[0] ? v[0] : (v[1] ? v[1] : (v[2] ? v[2] : v[3]));
    return e;
}

}  // namespace bcq

// On-device quantiser front end: fp16 weights -> packed binary-coded operand in one call.
//
//   step 1 (Eq. gptqt, with the scale of section "Re-explore Scaling Factor"), per (row, group):
//       qbias = Wmin,  S = fp16( s_factor (Wmax - Wmin) / (2^n - 1) ),
//       W_int = clamp( round((W - qbias) / S), 0, 2^n - 1 )        (nearest, ties to even)
//   step 2 (Eq. round): W_int -> code of the nearest integer the merged planes reach
//   fusion (Eq. fuse_step3): alpha_j = S m_j,  z = S (2^n - 1)/2 + qbias
//   packing: code bit i -> plane i, written straight into the layout of the descriptor.
//
// The quantiser is the inverse of the dequantisation S W_int + qbias and uses the fp16 S that is
// stored.  The integer is defined in fp64: W - qbias is exact there, the quotient is rounded once,
// so the decision does not depend on evaluation order.  Groups of 128 take one pass over W (a
// group's 16 chunks sit in 16 lanes); other group lengths take a range pass and an encode pass.
#include "bcq_internal.cuh"

namespace bcq {

constexpr int kQuantRows = 16;   // rows a block walks: the block's table set-up is shared by them

struct QuantTable {
    uint8_t code_of_int[256];
    double plane_weight[4];
    double centre;      // (2^n - 1) / 2
    double top;         // 2^n - 1
    double s_factor;
};

// One warp per (row, group): the range of the group's weights, then S and qbias.
__global__ void __launch_bounds__(256) rtn_range_kernel(const __half *__restrict__ W, int N, int K, int L, QuantTable tab,
                                                        __half *__restrict__ S, __half *__restrict__ qbias)
{
    const int G = K / L;
    const size_t unit = (size_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (unit >= size_t(N) * G) return;
    const __half *w = W + (unit / G) * size_t(K) + (unit % G) * size_t(L);
    float lo = __half2float(w[0]), hi = lo;
#pragma unroll 4
    for (int k = 8 * lane; k < L; k += 256) {   // L is a multiple of 32: whole 16-byte pieces
        const uint4 raw = *reinterpret_cast<const uint4 *>(w + k);
        const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(h[j]);
            lo = fminf(lo, fminf(f.x, f.y));
            hi = fmaxf(hi, fmaxf(f.x, f.y));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
        if (lo == 0.f) lo = 0.f;   // a zero minimum is stored as +0
        const double range = double(hi) - double(lo);   // exact
        S[unit] = __double2half(__ddiv_rn(__dmul_rn(tab.s_factor, range), tab.top));
        qbias[unit] = __float2half_rn(lo);              // exact: lo is an fp16 value
    }
}

// Shared-memory table of a block: entry t = the code of step-1 integer t with code bit i moved to
// bit 8 i, so that OR-ing (entry << j) over the 8 weights j of a chunk leaves plane i's byte in byte i.
__device__ __forceinline__ void load_spread_table(const QuantTable &tab, uint32_t *lut)
{
    for (int t = threadIdx.x; t < 256; t += blockDim.x) {
        const uint32_t c = tab.code_of_int[t];
        lut[t] = (c & 1u) | ((c & 2u) << 7) | ((c & 4u) << 14) | ((c & 8u) << 21);
    }
    __syncthreads();
}

// Integers, codes and plane bytes of one chunk of 8 weights (row n, bytes kb of the planes).
// The integer is DEFINED by the fp64 quotient (W - qbias)/S, rounded to nearest, ties to even.  An
// fp32 estimate t of the quotient (three roundings, relative error below 1.8e-7) decides whenever it
// is further from a rounding boundary than its own error bound; the few weights that are not (and
// exact ties) take the fp64 division.  Same integers, a fraction of the fp64 work.  Rounding t: adding
// 1.5 * 2^23 leaves the nearest integer in the low mantissa bits (valid below 2^22; larger t clamp).
// PACK = false (the search over scale factors wants the integers only): no codes, no plane bytes.
template <bool PACK>
__device__ __forceinline__ void encode_chunk(const uint4 raw, __half s_h, __half b_h, const QuantTable &tab,
                                             const uint32_t *lut, uint8_t *__restrict__ w_int, const View &dst, int n, int kb)
{
    const float sf = __half2float(s_h), bf = __half2float(b_h);
    const float inv_s = sf > 0.f ? __frcp_rn(sf) : 0.f;   // S = 0: every t is 0, every integer 0
    const float topf = float(tab.top);
    const int topi = int(tab.top);
    const float magic = 12582912.f;
    const uint32_t word[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t spread = 0u, ints_lo = 0u, ints_hi = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const __half hw = __ushort_as_half(uint16_t(word[j >> 1] >> (16 * (j & 1))));
        const float w = __half2float(hw);
        const float t = __fmul_rn(__fsub_rn(w, bf), inv_s);   // >= 0: qbias is the minimum
        const float err = fmaf(t, 4e-7f, 1e-6f);
        int r;
        if (t - err > topf + 0.5f) {
            r = topi;
        } else {
            const float shifted = __fadd_rn(t, magic);
            const float nearest = __fsub_rn(shifted, magic);
            if (fabsf(t - nearest) < 0.5f - err) {
                r = min(__float_as_int(shifted) - __float_as_int(magic), topi);
            } else {
                const double r64 = rint(__ddiv_rn(double(w) - double(bf), double(sf)));   // the subtraction is exact in fp64
                r = int(fmin(fmax(r64, 0.0), tab.top));
            }
        }
        if (PACK) spread |= lut[r] << j;
        if (j < 4)
            ints_lo |= uint32_t(r) << (8 * j);
        else
            ints_hi |= uint32_t(r) << (8 * (j - 4));
    }
    if (PACK) {
        unsigned char *out = dst.plane_byte(0, n, kb);
        const size_t stride = dst.plane_stride();
        for (int i = 0; i < dst.q; ++i) out[i * stride] = uint8_t(spread >> (8 * i));
    }
    if (w_int) *reinterpret_cast<uint2 *>(w_int + size_t(n) * dst.K + size_t(kb) * 8) = make_uint2(ints_lo, ints_hi);
}

// alpha_j = S m_j and z = S centre + qbias of one (row, group): exact in fp64, rounded once.
__device__ __forceinline__ void write_scales(__half s_h, __half b_h, const QuantTable &tab, const View &dst, int n, int g)
{
    const double s = double(__half2float(s_h)), b = double(__half2float(b_h));
    for (int j = 0; j < dst.q; ++j) *dst.alpha_elem(j, n, g) = __half_as_ushort(__double2half(s * tab.plane_weight[j]));
    *dst.z_elem(n, g) = __half_as_ushort(__double2half(s * tab.centre + b));
}

__device__ __forceinline__ void range_to_scale(float lo, float hi, const QuantTable &tab, __half &s_h, __half &b_h)
{
    if (lo == 0.f) lo = 0.f;   // a zero minimum is stored as +0
    const double range = double(hi) - double(lo);   // exact
    s_h = __double2half(__ddiv_rn(__dmul_rn(tab.s_factor, range), tab.top));
    b_h = __float2half_rn(lo);                      // exact: lo is an fp16 value
}

// Any group length: one thread per (row, chunk), S and qbias from the range kernel.  Block (x, y) covers
// rows kQuantRows x .. + kQuantRows - 1 and chunks 256 y .. + 255.
template <bool PACK>
__global__ void __launch_bounds__(256) rtn_encode_kernel(const __half *__restrict__ W, const __half *__restrict__ S,
                                                         const __half *__restrict__ qbias, int L, QuantTable tab,
                                                         uint8_t *__restrict__ w_int, const View dst)
{
    __shared__ uint32_t lut[256];
    load_spread_table(tab, lut);
    const int kb = blockIdx.y * 256 + threadIdx.x;
    if (kb >= dst.K / 8) return;
    const int G = dst.K / L, g = (kb * 8) / L;
    for (int n = blockIdx.x * kQuantRows; n < min(dst.N, (blockIdx.x + 1) * kQuantRows); ++n) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(W + size_t(n) * dst.K + size_t(kb) * 8);
        encode_chunk<PACK>(raw, S[size_t(n) * G + g], qbias[size_t(n) * G + g], tab, lut, w_int, dst, n, kb);
    }
    __threadfence();   // operands visible device-wide before the block counts as finished (products fetch them early)
}

// Groups of 128: everything in one pass.  A group is 16 chunks = 16 consecutive lanes, each holding
// its chunk in registers: range by shuffles, S and qbias by the group's first lane, then the encoding.
template <bool PACK>
__global__ void __launch_bounds__(256) rtn_fused128_kernel(const __half *__restrict__ W, QuantTable tab,
                                                           __half *__restrict__ S, __half *__restrict__ qbias,
                                                           uint8_t *__restrict__ w_int, const View dst)
{
    __shared__ uint32_t lut[256];
    load_spread_table(tab, lut);
    const int kbytes = dst.K / 8;   // a multiple of 16: a half-warp is inside the row or outside
    const int kb = blockIdx.y * 256 + threadIdx.x;
    const bool in = kb < kbytes;
    for (int n = blockIdx.x * kQuantRows; n < min(dst.N, (blockIdx.x + 1) * kQuantRows); ++n) {
        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
        if (in) raw = *reinterpret_cast<const uint4 *>(W + size_t(n) * dst.K + size_t(kb) * 8);
        const __half2 *h2 = reinterpret_cast<const __half2 *>(&raw);
        float lo, hi;
        {
            const float2 f = __half22float2(h2[0]);
            lo = fminf(f.x, f.y), hi = fmaxf(f.x, f.y);
#pragma unroll
            for (int j = 1; j < 4; ++j) {
                const float2 e = __half22float2(h2[j]);
                lo = fminf(lo, fminf(e.x, e.y));
                hi = fmaxf(hi, fmaxf(e.x, e.y));
            }
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        // S and qbias by the group's first lane, handed to the other 15; then lanes 0 .. q of the group
        // each produce one fused scale (alpha_0 .. alpha_{q-1}, z = S centre + qbias) in the same pass.
        __half s_h = __float2half_rn(0.f), b_h = s_h;
        const int sub = threadIdx.x & 15;
        const int g = kb >> 4, G = dst.K / 128;
        if (sub == 0 && in) {
            range_to_scale(lo, hi, tab, s_h, b_h);
            S[size_t(n) * G + g] = s_h;
            qbias[size_t(n) * G + g] = b_h;
        }
        const unsigned pair = uint32_t(__half_as_ushort(s_h)) | (uint32_t(__half_as_ushort(b_h)) << 16);
        const unsigned got = __shfl_sync(0xffffffffu, pair, (threadIdx.x & 31) & 16);
        s_h = __ushort_as_half(uint16_t(got & 0xffffu));
        b_h = __ushort_as_half(uint16_t(got >> 16));
        if (PACK && in && sub <= dst.q) {
            const double mult = sub < dst.q ? tab.plane_weight[sub & 3] : tab.centre;
            const double add = sub < dst.q ? 0.0 : double(__half2float(b_h));
            const uint16_t v = __half_as_ushort(__double2half(double(__half2float(s_h)) * mult + add));   // exact, rounded once
            if (sub < dst.q)
                *dst.alpha_elem(sub, n, g) = v;
            else
                *dst.z_elem(n, g) = v;
        }
        if (in) encode_chunk<PACK>(raw, s_h, b_h, tab, lut, w_int, dst, n, kb);
    }
    __threadfence();   // operands visible device-wide before the block counts as finished (products fetch them early)
}

// One thread per (row, group): the fused scales, written where the destination layout keeps them.
__global__ void __launch_bounds__(256) rtn_scales_kernel(const __half *__restrict__ S, const __half *__restrict__ qbias,
                                                         QuantTable tab, const View dst)
{
    const int G = dst.G();
    const size_t t = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= size_t(dst.N) * G) return;
    write_scales(S[t], qbias[t], tab, dst, int(t / G), int(t % G));
    __threadfence();   // as in the encoding kernels
}

cudaError_t launch_quantize_rtn(const uint16_t *W, int n_bits, double s_factor, const uint8_t *code_of_int /*[256]*/,
                                const double *plane_weight /*[q]*/, uint16_t *S, uint16_t *qbias, uint8_t *w_int,
                                const View &dst, cudaStream_t st, bool pack)
{
    QuantTable tab;
    for (int t = 0; t < 256; ++t) tab.code_of_int[t] = code_of_int[t];
    for (int j = 0; j < 4; ++j) tab.plane_weight[j] = j < dst.q ? plane_weight[j] : 0.0;
    tab.top = double((1u << n_bits) - 1u);
    tab.centre = tab.top / 2.0;
    tab.s_factor = s_factor;
    const int L = dst.group == 0 ? dst.K : dst.group;
    const size_t units = size_t(dst.N) * dst.G();
    const __half *w = reinterpret_cast<const __half *>(W);
    __half *s = reinterpret_cast<__half *>(S), *b = reinterpret_cast<__half *>(qbias);
    const dim3 grid(unsigned((dst.N + kQuantRows - 1) / kQuantRows), unsigned((dst.K / 8 + 255) / 256));   // kQuantRows rows per block
    if (L == 128) {
        if (pack)
            rtn_fused128_kernel<true><<<grid, 256, 0, st>>>(w, tab, s, b, w_int, dst);
        else
            rtn_fused128_kernel<false><<<grid, 256, 0, st>>>(w, tab, s, b, w_int, dst);
        return cudaGetLastError();
    }
    rtn_range_kernel<<<unsigned((units + 7) / 8), 256, 0, st>>>(w, dst.N, dst.K, L, tab, s, b);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (pack)
        rtn_encode_kernel<true><<<grid, 256, 0, st>>>(w, s, b, L, tab, w_int, dst);
    else
        rtn_encode_kernel<false><<<grid, 256, 0, st>>>(w, s, b, L, tab, w_int, dst);
    e = cudaGetLastError();
    if (e != cudaSuccess || !pack) return e;
    rtn_scales_kernel<<<unsigned((units + 255) / 256), 256, 0, st>>>(s, b, tab, dst);
    return cudaGetLastError();
}

}  // namespace bcq

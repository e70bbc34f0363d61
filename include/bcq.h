/*
 * bcq.h -- C ABI of the B200 (sm_100a) library for GPTQT inference (arxiv 2407.02891).
 *
 * After GPTQT's two quantisation steps are merged (section "Intermediate Steps Can be
 * Fused in Inference", Eq. fuse_step1..3), a linear layer is pure binary coding
 *
 *     W[n][k] = sum_{i<q} alpha[i][n][g(k)] * b_i[n][k] + z[n][g(k)],   b_i in {-1,+1}
 *     y[n]    = sum_k W[n][k] x[k]
 *             = sum_g ( sum_i alpha[i][n][g] * sum_{k in g} b_i[n][k] x[k] + z[n][g] * sum_{k in g} x[k] )
 *
 * (Eq. bcw gives the dequantisation  w = sum_i alpha_i b_i ; Eq. fuse_step3 adds the
 * offset).  g(k) = k / group is the scaling unit along K; group == 0 means one scale per
 * row, which is the granularity the paper states.  This library computes y at batch 1
 * (bcq_gemv) and for 2..16 activation vectors (bcq_gemm_smallbatch), and prepares the
 * operands (bcq_quantize_rtn from fp16 weights; bcq_merge_linear, bcq_pack, bcq_repack).
 *
 * Conventions
 *   - Every pointer named *_dev is DEVICE memory owned by the caller; *_host is host memory.
 *     Nothing is allocated or freed by the library and no pointer is retained after a call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; they never synchronise.  Errors found on the host return before any
 *     launch.  The current CUDA device must be the one that owns the pointers.
 *   - fp16 values are IEEE binary16 bit patterns in uint16_t.  Accumulation is fp32;
 *     y is rounded to fp16 (nearest even) once, at the end.  The lookup-table kernel keeps
 *     its table of 8-activation partial sums in fp16: each signed sum of 8 consecutive
 *     activations x[8c .. 8c+7] is computed in fp32 and rounded once (relative 2^-11 per table
 *     entry; everything added afterwards is fp32).  Input range: such a sum must stay finite in
 *     fp16, i.e. |x[8c]| + ... + |x[8c+7]| < 65520 for every chunk c; beyond that the entry becomes
 *     infinite and so does every y that uses it (the generic kernel, plan kernel 0, has no table
 *     and no such limit).
 *   - Packed operands are constants to the products: bcq_gemv and bcq_gemm_smallbatch start
 *     fetching them before they wait for the previous kernel in the stream (programmatic dependent
 *     launch).  Operands written by this library's calls (bcq_pack, bcq_repack, bcq_quantize_rtn)
 *     or by copies may be multiplied right away on the same stream.  A kernel of your own that
 *     writes packed operands immediately in front of a product must make its writes visible
 *     before its blocks end (__threadfence() after the last store), or be separated from the
 *     product by any other stream operation; x, y and the workspace are ordered as usual.
 *   - Device pointers must be 16-byte aligned (y: 2-byte) or BCQ_ERR_MISALIGNED is returned.
 *   - Return value: BCQ_OK (0) or a negative bcq_status.  No exceptions, no exit().
 *
 * Canonical layout (BCQ_LAYOUT_CANONICAL), row-major, last index fastest:
 *   codes   uint8  [N][K]        bit i of a code is 1  <=>  b_i = +1        (codes < 2^q)
 *   packed  uint8  [q][N][K/8]   bit (k mod 8) of byte (k div 8), LSB = lowest k, 1 <=> b = +1
 *   alpha   fp16   [q][N][G]     G = K / group, or 1 when group == 0
 *   z       fp16   [N][G]
 *   x       fp16   [B][K],   y fp16 [B][N]
 *
 * Tiled layout (BCQ_LAYOUT_TILED): the same bytes and the same fp16 values, permuted so that
 * the batch-1 kernel fetches everything it needs for 8 rows x 512 weights with ONE contiguous
 * bulk copy, and so that the 32 lanes of a warp always look up 32 different shared-memory
 * banks.  It needs K % 512 == 0, N % 8 == 0 and group in {0, 128, 64, 32}.  With U = N/8 row units
 * and K/512 windows, `packed` is a sequence of tiles, tile (w, u) at byte (w*U + u) * T.  Inside a
 * tile, lane l = 8 g + j (g < 4, j < 8) stands for row 8u + j and the g-th segment of 128 weights
 * of window w.  SUB = 128 / group is the number of scaling units in a segment (1 for group 128 and,
 * for the walk below, for group 0):
 *   bytes [0, q*512)      planes as [i < q][lane < 32][s < 16]: byte s of lane l in plane i holds
 *                         plane i of the 8 weights  k = 512 w + 128 g + 8 c .. + 7  (bit order as
 *                         canonical) of chunk c of the segment, where
 *                           SUB = 1:     c = (s + 2 j) mod 16
 *                           SUB = 2, 4:  the lane walks its segment unit by unit.  With C = 16/SUB chunks
 *                                        and P = 8/SUB chunk pairs per unit, ph = s div C, t = s mod C:
 *                                        unit  sg = (ph + j div P) mod SUB,
 *                                        c = 2 (P sg + ((t div 2 + j) mod P)) + (t mod 2)
 *   group != 0, T = q*512 + 64*SUB*(q+1): the tile continues with the lanes' scales,
 *     bytes [q*512, T)    fp16 [lane < 32][ph < SUB][alpha_0 .. alpha_{q-1}, z]: the ph-th set is that of
 *                         the unit the lane walks in phase ph,
 *                         <- alpha[i][8u + j][(4w + g) SUB + sg], z[8u + j][(4w + g) SUB + sg]
 *     and the alpha / z arguments of every call are ignored for this layout (pass NULL);
 *   group 0 (one scale per row), T = q*512: alpha and z stay in arrays of their own,
 *     alpha [u][i][r], z [u][r].
 * Groups of 64 and 32 run the lookup-table kernel one column at a time (no column pairs, no
 * tensor-core kernel, no bcq_gemv_multi, no bcq_gemv_dequant).
 * bcq_packed_bytes gives the size of `packed` for the descriptor's layout (it includes the
 * scales exactly when they live in the tiles); bcq_alpha_elems and bcq_offset_elems give the
 * element counts of separate alpha / z arrays (the canonical counts).
 */
#ifndef BCQ_H
#define BCQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BCQ_VERSION 220

typedef enum bcq_status {
    BCQ_OK = 0,
    BCQ_ERR_INVALID_ARG = -1,        /* NULL pointer, q outside 1..4, N or K <= 0, B outside 1..16, ...   */
    BCQ_ERR_UNSUPPORTED_SHAPE = -2,  /* K % 32 != 0; group != 0 and (K % group != 0 or group % 32 != 0);   */
                                     /* or a shape the tiled layout does not cover                        */
    BCQ_ERR_MISALIGNED = -3,         /* a device pointer is not aligned as required                       */
    BCQ_ERR_WORKSPACE_TOO_SMALL = -4,
    BCQ_ERR_CUDA = -5,               /* a CUDA runtime call failed; text via bcq_last_cuda_error()        */
    BCQ_ERR_SCRATCH_LIMIT = -6,      /* bcq_gemv_noalloc: the product needs more than the built-in scratch */
    BCQ_ERR_TIMEOUT = -7             /* bcq_poll_status: a bounded wait inside a kernel ran out           */
} bcq_status;

enum { BCQ_LAYOUT_CANONICAL = 0, BCQ_LAYOUT_TILED = 1 };

/* One quantised linear layer: N output rows, K inputs, q bit-planes, `group` weights per
 * scaling unit along K (0 = one unit per row), and the memory layout of its operands. */
typedef struct bcq_desc {
    int32_t N;
    int32_t K;
    int32_t q;
    int32_t group;
    int32_t layout;
} bcq_desc;

/* How a product is decomposed over the GPU.  kernel: 0 = generic (one warp per row; any valid
 * shape, either layout), 1 = lookup-table kernel (tiled layout, one or two columns per launch),
 * 2 = tensor-core small-batch kernel (tiled layout, 2..16 columns per launch); kernels 1 and 2
 * are launched as row_blocks x k_splits thread blocks; k_splits > 1 needs the workspace.
 * Limits: at most 184 (kernel 1; 160 for q = 4 with two columns per launch) or 176 (kernel 2)
 * row units of 8 rows per block, at most 32 windows of 512 weights per K split.
 * reserved: 0.  The library's own tests set BCQ_PLAN_TEST_* bits there (kernel 1 only) to see a
 * bounded wait inside the kernel run out without anything faulting: SHORT_WAITS shortens the
 * limit of every wait to about a millisecond, WITHHOLD_TABLE makes the table builders keep a
 * completed table to themselves, so that the warps waiting for it give up.  y is then undefined
 * and bcq_poll_status reports BCQ_ERR_TIMEOUT. */
typedef struct bcq_plan {
    int32_t kernel;
    int32_t row_blocks;
    int32_t k_splits;
    int32_t reserved;
} bcq_plan;
enum { BCQ_PLAN_TEST_SHORT_WAITS = 1, BCQ_PLAN_TEST_WITHHOLD_TABLE = 2 };

/* ---- sizes (pure host functions; 0 when the descriptor is invalid) -------------------- */
size_t bcq_packed_bytes(const bcq_desc *desc);   /* q*N*K/8, plus 2*(q+1)*N*G when tiled with grouped scales */
size_t bcq_alpha_elems(const bcq_desc *desc);    /* q * N * G                              */
size_t bcq_offset_elems(const bcq_desc *desc);   /* N * G                                  */

/* Validate a descriptor: BCQ_OK, BCQ_ERR_INVALID_ARG or BCQ_ERR_UNSUPPORTED_SHAPE. */
int bcq_check_desc(const bcq_desc *desc);

/* The decomposition bcq_gemv / bcq_gemm_smallbatch use by default for batch B on a GPU with
 * `sm_count` multiprocessors (sm_count <= 0: ask the current device).  Pure host logic when
 * sm_count > 0. */
int bcq_plan_default(const bcq_desc *desc, int B, int sm_count, bcq_plan *plan_out);

/* Bytes of workspace the plan needs (0 when k_splits == 1 and the generic kernel).  The
 * workspace holds the split-K partial sums and arrival counts (kernel 1: one 64-bit word per
 * row and column, in which the K splits' sums meet as fixed-point numbers in units of 2^-26;
 * a split's partial sum beyond +-131071 saturates).  It must be zero-filled once
 * (bcq_workspace_init) before its first use; every call leaves it zero where it has to be, so
 * it can be reused by later calls ON THE SAME STREAM.  Two products in flight at once
 * need two workspaces.  After a call that bcq_poll_status reported as timed out the counters
 * may be left non-zero: zero-fill the workspace again before the next use. */
size_t bcq_workspace_bytes(const bcq_desc *desc, int B, const bcq_plan *plan /* NULL = default */);
int bcq_workspace_init(void *workspace_dev, size_t bytes, void *stream);

/* ---- operand preparation (offline, once per layer) ------------------------------------ */

/*
 * Linear-int -> merged binary code (Eq. round, Eq. fuse_step1..3).
 * w_int holds step-1 integers 0 .. 2^n_bits - 1; S and qbias ([N][G], canonical) dequantise
 * them as S * w_int + qbias.  bit_to_plane_host[i-1] in 0..q-1 assigns step-1 bit i (weight
 * 2^(i-2)) to a plane; every plane needs at least one bit.  Outputs, all canonical:
 *   codes  [N][K]   code of the reachable integer nearest to w_int (ties: the smaller one)
 *   alpha  [q][N][G] = S * sum_{i in plane j} 2^(i-2)          (rounded once to fp16)
 *   z      [N][G]    = S * (2^n_bits - 1)/2 + qbias            (rounded once to fp16)
 * desc->layout is ignored.  n_bits in 1..8, q <= n_bits.
 */
int bcq_merge_linear(const bcq_desc *desc, const uint8_t *w_int_dev, const uint16_t *S_dev,
                     const uint16_t *qbias_dev, int n_bits, const uint8_t *bit_to_plane_host,
                     uint8_t *codes_dev, uint16_t *alpha_dev, uint16_t *z_dev, void *stream);

/*
 * fp16 weights -> packed binary-coded operand in desc->layout, in one call: step-1 linear
 * quantisation (Eq. gptqt step 1 with the scale of section "Re-explore Scaling Factor"),
 * nearest reachable integer (Eq. round), fusion (Eq. fuse_step3) and packing.
 * Per (row, group) of W [N][K] (fp16, device, 16-byte aligned, finite values):
 *   qbias = Wmin,   S = fp16( s_factor * (Wmax - Wmin) / (2^n_bits - 1) )
 *   w_int = clamp( round((W - qbias) / S), 0, 2^n_bits - 1 )   nearest, ties to even, decided
 *           in fp64 from the stored fp16 S; a group of equal weights gets S = 0, w_int = 0
 * s_factor = 1 is the step-1 scale; Eq. reexplore searches s_factor between
 * (2^n - 1)/(2^(n+1) - 1) and (2^n - 1)/(2^(n-1) - 1).  bit_to_plane_host as in bcq_merge_linear.
 * Outputs (device, caller-owned): S, qbias [N][G] canonical (always written; they are also
 * the kernels' scratch); w_int [N][K] or NULL; packed / alpha / z exactly as bcq_merge_linear
 * followed by bcq_pack would produce them for desc->layout (alpha and z ignored when the tiles
 * carry the scales).  Asynchronous on `stream`, no allocation.  The paper times no quantiser;
 * this one reads W once for groups of 128 (2 bytes per weight plus the operand written) and
 * twice (range, then encode) for every other group length.
 */
int bcq_quantize_rtn(const bcq_desc *desc, const uint16_t *W_dev, int n_bits,
                     const uint8_t *bit_to_plane_host, double s_factor, uint16_t *S_dev,
                     uint16_t *qbias_dev, uint8_t *w_int_dev, void *packed_dev, uint16_t *alpha_dev,
                     uint16_t *z_dev, void *stream);

/*
 * Codes + canonical scales -> packed bit-planes and scales in desc->layout.
 * Bit-exact: only bit extraction and permutation.  Canonical, or tiled with group 0:
 * alpha_in/z_in may be NULL together with alpha_out/z_out to pack the planes only.  Tiled with
 * group 128: alpha_in and z_in are required (they go into the tiles); alpha_out/z_out are
 * ignored.  Outputs must not overlap inputs.
 */
int bcq_pack(const bcq_desc *desc, const uint8_t *codes_dev, const uint16_t *alpha_in_dev,
             const uint16_t *z_in_dev, void *packed_out_dev, uint16_t *alpha_out_dev,
             uint16_t *z_out_dev, void *stream);

/*
 * Re-lay-out packed operands from src->layout to dst->layout (N, K, q, group must agree).
 * Bit-exact permutation; canonical -> tiled -> canonical is the identity.  The packed pointers
 * are required.  Scales move when the source has them (inside its tiles, or alpha_src and z_src
 * given) and the destination takes them (inside its tiles, or alpha_dst and z_dst given); a
 * destination that keeps its scales in the tiles cannot be made without them.  Scale pointers of
 * a side whose scales live in the tiles are ignored.  No in-place operation.
 */
int bcq_repack(const bcq_desc *src, const void *packed_src_dev, const uint16_t *alpha_src_dev,
               const uint16_t *z_src_dev, const bcq_desc *dst, void *packed_dst_dev,
               uint16_t *alpha_dst_dev, uint16_t *z_dst_dev, void *stream);

/* ---- the products --------------------------------------------------------------------- */

/*
 * y = W x at batch 1 (the definition at the top of this file; Eq. bcw + Eq. fuse_step3).
 * x [K], y [N] fp16.  y is overwritten.  workspace may be NULL when bcq_workspace_bytes is 0.
 * bcq_gemv_plan is the same product with an explicit decomposition (for tuning and tests):
 * the plan must have 1 <= row_blocks, 1 <= k_splits <= K/512, at most 184 row units (1472 rows)
 * per row block and at most 32 windows (16384 weights along K) per K split.
 */
int bcq_gemv(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
             const uint16_t *z_dev, const uint16_t *x_dev, uint16_t *y_dev,
             void *workspace_dev, size_t workspace_bytes, void *stream);
int bcq_gemv_plan(const bcq_desc *desc, const bcq_plan *plan, const void *packed_dev,
                  const uint16_t *alpha_dev, const uint16_t *z_dev, const uint16_t *x_dev,
                  uint16_t *y_dev, void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * Several layers that read the SAME activation, in one launch: y_o = W_o x for o < count (batch 1).
 * At decode the query, key and value projections of a layer (and the gate and up projections of a
 * gated feed-forward block) multiply one and the same vector -- the per-token measurement of the
 * paper's section "Setup" runs every linear module of every decoder layer once per token -- and
 * launching them together builds each window's lookup table once per thread block instead of once
 * per projection and pays the fixed cost of a launch once.  Every operand keeps its own packed
 * tensor and its own y; nothing is concatenated.
 *   desc   K, q, group and layout (BCQ_LAYOUT_TILED) of all operands; desc->N = sum of ops[o].N
 *   ops    host array of 1..4 operands: packed_dev (and alpha_dev / z_dev when the scales are not in
 *          the tiles), y_dev [N] and N (a multiple of 8) of each; read during the call only
 *   plan   kernel 1; its row_blocks are shared out among the operands in proportion to their rows
 *          (largest remainders; bcq_multi_row_blocks tells how), its k_splits apply to all.  An operand
 *          that would get no row block, or more than 184 row units per block, makes the plan invalid.
 *          bcq_gemv_multi uses bcq_plan_default of `desc` (enlarged, if need be, until it is valid).
 * Workspace: bcq_workspace_bytes(desc, 1, plan), as for a single product of desc->N rows.
 * With the same k_splits and the same row blocks per operand as a bcq_gemv_plan call on that operand
 * alone, y_o is bit-identical to that call's result.  Errors as bcq_gemv.
 */
typedef struct bcq_operand {
    const void *packed_dev;
    const uint16_t *alpha_dev;
    const uint16_t *z_dev;
    uint16_t *y_dev;
    int32_t N;
    int32_t reserved;   /* 0 */
} bcq_operand;
int bcq_gemv_multi(const bcq_desc *desc, const bcq_operand *ops_host, int count, const uint16_t *x_dev,
                   void *workspace_dev, size_t workspace_bytes, void *stream);
int bcq_gemv_multi_plan(const bcq_desc *desc, const bcq_plan *plan, const bcq_operand *ops_host, int count,
                        const uint16_t *x_dev, void *workspace_dev, size_t workspace_bytes, void *stream);
/* The row blocks each operand gets under `plan` (pure host logic): row_blocks_out[o], o < count. */
int bcq_multi_row_blocks(const bcq_desc *desc, const bcq_plan *plan, const int32_t *N_host, int count,
                         int32_t *row_blocks_out);

/*
 * Y[b] = W X[b] for b < B, 1 <= B <= 16; X [B][K], Y [B][N] row-major fp16.  Every column is
 * an independent product (the paper defines batch 1 only; Eq. bcw + Eq. fuse_step3 per column).
 * B == 1 is bcq_gemv.  Tiled layout: by default B >= 4 takes ONE pass over the packed weights
 * for all columns (plan kernel 2, the tensor-core kernel: a weight bit becomes the fp16 value
 * +-alpha of its row and group, the products with x are exact, all sums fp32; the offset term
 * uses the fp32 group sums of x, kept to 22 bits) and B == 2, 3 run the lookup-table kernel on
 * column pairs (plan kernel 1 with tables that hold two columns' sums side by side: one pass
 * over the weights and one 4-byte lookup per weight byte for both columns of a pair; every
 * column is bit-identical to bcq_gemv on it), which is faster there (bcq_plan_default tells
 * which).  The workspace depends on B: bcq_workspace_bytes(desc, B, plan).
 * Canonical layout: one pass of the generic kernel for all columns.
 * bcq_gemm_smallbatch_plan takes the decomposition from the caller; a plan with kernel 1 runs
 * the lookup-table kernel on two columns at a time when the scales live in the tiles (group
 * 128: ceil(B/2) passes) and column by column otherwise (one scale per row: B passes).
 */
int bcq_gemm_smallbatch(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                        const uint16_t *z_dev, const uint16_t *X_dev, uint16_t *Y_dev, int B,
                        void *workspace_dev, size_t workspace_bytes, void *stream);
int bcq_gemm_smallbatch_plan(const bcq_desc *desc, const bcq_plan *plan, const void *packed_dev,
                             const uint16_t *alpha_dev, const uint16_t *z_dev, const uint16_t *X_dev,
                             uint16_t *Y_dev, int B, void *workspace_dev, size_t workspace_bytes,
                             void *stream);

/*
 * bcq_gemv with the activation and the result in HOST memory: enqueues x_host -> x_stage_dev,
 * the product, y_stage_dev -> y_host on `stream` and returns without synchronising (the
 * caller synchronises the stream before reading y_host).  Use page-locked host memory for
 * the copies to be asynchronous; when y_host is page-locked the kernel stores y into it
 * directly and y_stage_dev is not used.  x_stage_dev [K] and y_stage_dev [N] are caller-owned
 * device buffers.
 */
int bcq_gemv_host(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                  const uint16_t *z_dev, const uint16_t *x_host, uint16_t *y_host,
                  uint16_t *x_stage_dev, uint16_t *y_stage_dev,
                  void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * The product with what follows it in a decoder layer fused into its last step (the per-token decode of the
 * paper's section "Setup" runs bias, activation and residual additions as steps of their own):
 *     y = act(W x + bias) + residual
 * evaluated in fp32 from the complete sum and rounded once to fp16.  bias_dev, residual_dev: [N] fp16 device
 * arrays or NULL; residual_dev may be y_dev itself (every row is read before it is written, by the same
 * thread).  activation: BCQ_ACT_NONE, BCQ_ACT_RELU, BCQ_ACT_GELU (x/2 (1 + erf(x/sqrt 2))), BCQ_ACT_SILU
 * (x / (1 + exp(-x))).  Tiled layout only (the lookup-table kernel); otherwise as bcq_gemv.
 */
enum { BCQ_ACT_NONE = 0, BCQ_ACT_RELU = 1, BCQ_ACT_GELU = 2, BCQ_ACT_SILU = 3 };
typedef struct bcq_epilogue {
    const uint16_t *bias_dev;
    const uint16_t *residual_dev;
    int32_t activation;
    int32_t reserved;   /* 0 */
} bcq_epilogue;
int bcq_gemv_fused(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                   const uint16_t *z_dev, const uint16_t *x_dev, uint16_t *y_dev, const bcq_epilogue *epilogue,
                   void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * bcq_gemv with bfloat16 activations and outputs: x [K] and y [N] (and the epilogue's bias and residual, when an
 * epilogue is given; NULL = none) are bfloat16 bit patterns; the packed operand and its fp16 scales are
 * unchanged.  The sums of 8 activations in the lookup tables are still rounded to fp16, so eight activations of
 * one sign must not add up beyond 65504; accumulation is fp32, the result is rounded once to bfloat16
 * (2^-9 relative).  Tiled layout only.
 */
int bcq_gemv_bf16(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                  const uint16_t *z_dev, const uint16_t *x_bf16_dev, uint16_t *y_bf16_dev,
                  const bcq_epilogue *epilogue_or_null, void *workspace_dev, size_t workspace_bytes, void *stream);

/*
 * Ablation: the product of bcq_gemv computed without lookup tables.  Every weight is dequantised to fp16
 * (Eq. bcw dequantisation + Eq. fuse_step3: w = sum_i alpha_i b_i + z, fp16 additions) and multiplied with its
 * activation (fp32 accumulation), the way a kernel for linearly quantised weights works; operand, layout
 * (tiled only) and bytes read are those of bcq_gemv.  Its time against bcq_gemv shows, on this GPU, the shape
 * of the paper's speed claim for binary-coded weights (Tab. "The speed up of GPTQT").  No workspace.
 */
int bcq_gemv_dequant(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                     const uint16_t *z_dev, const uint16_t *x_dev, uint16_t *y_dev, void *stream);

/*
 * bcq_gemv without a workspace argument and without any allocation.  (The paper has no
 * counterpart; this entry point exists for the library's users.)
 *
 * Who it is for: callers that must not, or cannot, obtain device memory at the point where
 * they need the product -- a plugin running inside a host application that owns all device
 * memory and hands none out, a serving loop where an allocation would stall the whole device,
 * a process whose memory budget is already fully committed.  Such callers cannot create the
 * workspace bcq_gemv wants for its split-K partial sums.
 *
 * Here the scratch is a fixed array of BCQ_NOALLOC_SCRATCH_BYTES inside the library image.
 * Consequences to know about:
 *   - every GPU on which this library is loaded gives up that much memory until the process
 *     exits, whether or not this function is ever called;
 *   - a product whose default decomposition needs more scratch (8 bytes per row when K is
 *     split, i.e. more than 262144 rows) is refused with BCQ_ERR_SCRATCH_LIMIT and nothing is
 *     launched;
 *   - the first call on each device looks up the array's device address (a host-side runtime
 *     query, done with that device current) and keeps it for as long as the device's primary
 *     context lives (a cudaDeviceReset invalidates it).  Make that first call during start-up,
 *     before any stream capture is begun;
 *   - all calls on a device share the one array.  Calls on the same stream are ordered and
 *     safe; calls whose kernels can overlap on the GPU (different streams, no dependency)
 *     race on it and give wrong results.  The array keeps the previous call's contents; the
 *     function clears the part that has to start at zero on every call.
 * Neither this function nor anything it calls uses cudaMalloc, cudaFree or an allocating
 * library routine.  Result and error behaviour are otherwise those of bcq_gemv.
 */
#define BCQ_NOALLOC_SCRATCH_BYTES (2u << 20)
int bcq_gemv_noalloc(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                     const uint16_t *z_dev, const uint16_t *x_dev, uint16_t *y_dev, void *stream);

/*
 * The search of GPTQT's second step on calibration inputs (section "Quantize Weight Twice", Eq. gptqt step 2:
 * the BCchoice of Eq. round is the one with the smallest output error; section "Re-explore Scale Factor",
 * Eq. reexplore: so is the scale of step 1).  For every scale factor s (outer loop) and every candidate split
 * p of the n_bits step-1 bits into desc->q planes (inner loop):
 *     step 1 as in bcq_quantize_rtn with s_factor = s  ->  W_int, S, qbias per (row, scaling unit)
 *     W_q = the integer of BCchoice p nearest to W_int (Eq. round; ties: the smaller)
 *     err_rows[s][p][n] = sum_t ( sum_k (S W_q[n][k] + qbias - W[n][k]) X[t][k] )^2
 *     err[s][p]         = sum_n err_rows[s][p][n]
 * and best = (s, p) of the first candidate, in loop order, whose err is below all earlier ones.
 * The contraction runs on the tensor cores with fp16 operands (a weight difference is formed as
 * S (W_q - W_int) + r, r = S W_int + qbias - W computed in fp32 and rounded to fp16, by one fp16 fused
 * multiply-add) and fp32 accumulation; the error values agree with an fp64 evaluation to about 1e-3 relative, so
 * candidates closer than that may swap places.  GPTQ's error compensation is not part of this call.
 *   W [N][K] fp16 weights, X [T][K] fp16 calibration inputs (device, 16-byte aligned); T a multiple of 16,
 *   16..65536 (the error is a sum over tokens: more than 256 tokens run as pieces of at most 256, one launch
 *   each, on the same stream); K a multiple of 64; desc->group 0 or a multiple of 64; n_bits 1..6; desc->layout is ignored.
 *   partitions_host [P][n_bits]: bit_to_plane arrays as in bcq_merge_linear (bcq_partition_get lists them all);
 *   s_factors_host [n_scales] (bcq_reexplore_factors gives an even grid inside the interval of Eq. reexplore).
 *   err_dev [n_scales][P] fp64; err_rows_dev [n_scales][P][N] fp32 or NULL; best_dev [2] int32.
 *   workspace: bcq_grid_search_workspace(desc, T, n_bits, P, n_scales, err_rows_dev != NULL) bytes, 256-byte
 *   aligned; holds W_int, S and qbias of up to 8 scale factors (searched together in one launch: N * K bytes
 *   each) and a scratch operand.  Asynchronous on `stream`.
 */
size_t bcq_grid_search_workspace(const bcq_desc *desc, int T, int n_bits, int P, int n_scales, int rows_given);
int bcq_grid_search(const bcq_desc *desc, const uint16_t *W_dev, const uint16_t *X_dev, int T, int n_bits,
                    const uint8_t *partitions_host, int P, const double *s_factors_host, int n_scales,
                    double *err_dev, float *err_rows_dev, int32_t *best_dev, void *workspace_dev,
                    size_t workspace_bytes, void *stream);
/* Every split of n_bits step-1 bits into q non-empty planes (the candidates Eq. fuse_step2 can build), each
 * once: planes numbered by their lowest bit, arrays in lexicographic order.  Host functions. */
int bcq_partition_count(int n_bits, int q);                                      /* 0 when the arguments are invalid */
int bcq_partition_get(int n_bits, int q, int index, uint8_t *bit_to_plane_out);  /* [n_bits] */
/* `count` evenly spaced scale factors strictly inside the interval of Eq. reexplore, as multiples of the
 * step-1 scale (Wmax - Wmin)/(2^n - 1): between (2^n - 1)/(2^(n+1) - 1) and (2^n - 1)/(2^(n-1) - 1). */
int bcq_reexplore_factors(int n_bits, int count, double *s_factors_out);

/*
 * Every wait inside the kernels (on an mbarrier fed by an asynchronous copy or by other warps)
 * is bounded.  If one ever runs out, the block stops waiting, lets its outstanding copies land,
 * returns without a fault, and records the event in a device status word; y is then undefined.
 * bcq_poll_status waits for all work submitted to the current device (cudaDeviceSynchronize:
 * non-blocking streams included), returns BCQ_ERR_TIMEOUT if a wait ran out since the last poll
 * (detail via bcq_last_cuda_error) and clears the word; BCQ_OK otherwise.
 */
int bcq_poll_status(void);

/* ---- misc ----------------------------------------------------------------------------- */
const char *bcq_status_string(int status);   /* static string                              */
const char *bcq_last_cuda_error(void);       /* text of the last CUDA error seen, "" if none */
int bcq_version(void);                       /* BCQ_VERSION                                 */

#ifdef __cplusplus
}
#endif
#endif /* BCQ_H */

/*
 * scalebits.h -- C ABI of the B200 (sm_100a) hot path of ScaleBITS' bitwidth search
 * (arxiv 2602.17698): score every hardware-aligned weight block at every candidate
 * bitwidth, then allocate bits globally under a memory budget.
 *
 * Conventions (all entry points):
 *   - Every tensor pointer is CALLER-OWNED DEVICE memory on the context's device,
 *     valid until the context's stream has passed the call.  The only host pointers
 *     are `bits` arrays (read during the call), `sb_alloc_report*` and out-params of
 *     sb_create / sb_kernel_launches.
 *   - Calls enqueue work on the context's stream and return without waiting, except
 *     sb_allocate_bits and sb_sync, which synchronise that stream.
 *   - Return value: SB_OK, or an argument / shape / budget error detected on the host
 *     (nothing was enqueued).  Conditions detected on the device (non-finite input,
 *     packed capacity exceeded, a bounded wait that ran out) are latched in a device
 *     status word and returned by the next sb_sync / sb_allocate_bits.
 *   - bf16 matrices are row-major with a leading dimension in elements; the base
 *     must be 16-byte aligned and the leading dimension a multiple of 8.
 *   - A permutation is int32 perm[new] = old.  NULL means identity.
 *   - The library owns one scratch arena per context, grown on demand; after the
 *     first call of each shape nothing allocates.  An outgrown arena stays allocated
 *     until sb_destroy, so launches already enqueued, or captured in a CUDA graph by
 *     the caller, keep valid scratch pointers (a growth cannot happen during capture:
 *     run every captured call once eagerly first).
 *   - No call falls back to the CPU.
 */
#ifndef SCALEBITS_H_
#define SCALEBITS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sb_ctx sb_ctx;

typedef enum {
    SB_OK = 0,
    SB_ERR_INVALID = 1,     /* NULL / out-of-range argument, bad bit list            */
    SB_ERR_SHAPE = 2,       /* sizes not divisible as required, misaligned pointer   */
    SB_ERR_BUDGET = 3,      /* budget below the smallest candidate bitwidth          */
    SB_ERR_SCRATCH = 4,     /* scratch allocation failed / capacity too small        */
    SB_ERR_CUDA = 5,        /* a CUDA runtime call failed (see sb_last_error)        */
    SB_ERR_NOCONVERGE = 6,  /* Algorithm 2 hit the iteration cap (4096)              */
    SB_ERR_NONFINITE = 7,   /* a non-finite score or error was produced on device    */
    SB_ERR_TIMEOUT = 8      /* a bounded device-side wait (scan look-back) ran out   */
} sb_status;

enum { SB_ALLOC_SCALEBITS = 0, SB_ALLOC_GREEDY = 1 };
enum { SB_ACC_ROW = 1, SB_ACC_COL = 2 };

/* Context: device, stream (a cudaStream_t passed as void*, NULL = default stream),
 * scratch arena, device status word.  One context per stream; not thread-safe.      */
sb_status sb_create(sb_ctx** ctx, int device, void* cuda_stream);
sb_status sb_destroy(sb_ctx* ctx);
/* Waits for the stream, returns and clears the latched device status.               */
sb_status sb_sync(sb_ctx* ctx);
/* Static / context-owned string describing the last host-side error.                */
const char* sb_last_error(const sb_ctx* ctx);

/* Test hook for the one device-side wait of the path, the look-back of the chained scans
 * (prefix sums of Algorithm 1's step costs and of the packed block sizes; the paper has no
 * counterpart).  wait_ns: how long a tile may wait for a predecessor before it gives up, latches
 * SB_ERR_TIMEOUT and lets the kernel return (negative: the default, 250 ms).  mute_tile: the tile
 * of that index publishes nothing, like a predecessor that never arrives (negative: none).  With
 * a muted tile the results of the call are undefined; the status is returned by sb_sync /
 * sb_allocate_bits, which also clears it.  Synchronises the stream.  Use only with calls whose
 * later kernels index by block id (SB_ALLOC_GREEDY with at most 65536 steps): a scan whose
 * prefix feeds addresses (sb_pack_blocks, the multi-launch sort) must not run with a muted tile. */
sb_status sb_debug_lookback(sb_ctx* ctx, int64_t wait_ns, int64_t mute_tile);
/* Number of kernels this context has launched so far (for launch accounting).       */
int64_t sb_kernel_launches(const sb_ctx* ctx);
/* 1 if the library was built with -DSB_CHECKED (data-dependent indices bounds-checked on the device,
 * a failing one latched as SB_ERR_INVALID with the index in sb_last_error), else 0.           */
int sb_checked_build(void);

/* Calibration second moments -- the column factor |x_j| of the element sensitivity
 * (Section 3.2, the equation after Eq. 3), aggregated over tokens as a second moment:
 *     sumsq[j] = (accumulate ? sumsq[j] : 0) + scale * sum_t X[t][j]^2
 * X: bf16 [T][K], leading dimension ldx.  sumsq: fp32 [K].  K % 8 == 0.
 * fp32 accumulation in a fixed order (run-to-run deterministic).                    */
sb_status sb_calib_moments(sb_ctx* ctx, const void* X_bf16, int64_t T, int64_t K, int64_t ldx,
                           float* sumsq, int accumulate, float scale);

/* Bi-directional channel reordering (Section 4.1; coupling rules of Appendix D).
 * Phase 1 (W != NULL): fake-quantise W on its ORIGINAL layout at ref_bits (round to
 * nearest, asymmetric min-max, groups of `group` consecutive columns; Section 5
 * "Implementation"), element sensitivity s_rj = a_r c_j (W_rj - Q(W)_rj)^2, and
 *     row_score[r] (+)= sum_j s_rj,   col_score[j] (+)= sum_r s_rj
 * (accumulate is a bit mask: SB_ACC_ROW adds to what row_score holds, SB_ACC_COL to what
 * col_score holds, otherwise the buffer is overwritten; matrices that must share a
 * permutation pass the same buffer).  Either score pointer may be NULL.
 * Phase 2 (per axis, when *_segment > 0 and *_perm != NULL): sort the channels of the
 * score buffer by score, descending, ties to the lower index, independently inside
 * each run of *_segment channels (*_segment = axis length: whole axis; head_dim: within
 * each attention head).  Phase 2 sees the scores after phase 1.
 * W == NULL skips phase 1 ("sort only"); R / C still give the axis lengths.
 * C % group == 0, group in {16,32,64,128}.  col_moment: fp32 [C]; row_weight: fp32
 * [R] or NULL (= 1).                                                                 */
sb_status sb_reorder_channels(sb_ctx* ctx, const void* W_bf16, int64_t R, int64_t C, int64_t ldw,
                              const float* col_moment, const float* row_weight,
                              int ref_bits, int group,
                              float* row_score, float* col_score, int accumulate,
                              int64_t row_segment, int64_t col_segment,
                              int32_t* row_perm, int32_t* col_perm);

/* Appendix D (the residual-stream permutation also shuffles what is not quantised: the columns
 * of the embedding and of the language-model head, the rows of anything that writes the stream):
 * out[r][j] = W[row_perm[r]][col_perm[j]] for a bf16 matrix that is only moved, not scored.
 * W [R][ldw] device, row-major, ldw >= C, C a multiple of 8, 16-byte aligned; row_perm [R] /
 * col_perm [C] device (perm[new] = old) or NULL = identity; out [R][C] device, dense, must not
 * overlap W.  Asynchronous on the context's stream.  SB_ERR_INVALID: null pointers;
 * SB_ERR_SHAPE: alignment, or rows longer than 34133 columns.                                  */
sb_status sb_permute_matrix(sb_ctx* ctx, const void* W_bf16, int64_t R, int64_t C, int64_t ldw,
                            const int32_t* row_perm, const int32_t* col_perm, void* out_bf16);

/* Helpers for grouped-query attention (Appendix D: value / output projections are
 * reordered inside each head; query heads that read one value head share its order):
 *   fold:   dst[h*seg + d] += sum_{u<reps} src[(h*reps + u)*seg + d],  n_dst = len(dst)
 *   expand: out[(h*reps + u)*seg + d] = (h*reps + u)*seg + (perm[h*seg + d] - h*seg)   */
sb_status sb_fold_segment_scores(sb_ctx* ctx, float* dst, const float* src, int64_t n_dst,
                                 int reps, int64_t seg);
sb_status sb_expand_segment_perm(sb_ctx* ctx, int32_t* out, const int32_t* perm, int64_t n_src,
                                 int reps, int64_t seg);

/* Score vectors of the matrices of one coupled channel set (Appendix D), each written by an
 * sb_reorder_channels call of its own -- possibly on another context's stream, so that the
 * calls overlap -- added in a fixed order:
 *   dst[i] = (accumulate ? dst[i] : 0) + src[0][i] + src[1][i] + ... + src[n_src-1][i],
 * left to right in fp32, which is the order (and the result, bit for bit) of the same calls
 * accumulating into dst one after the other.  src: HOST array of 1..8 device pointers to
 * fp32 [n] (read during the call); dst: device fp32 [n].  The caller orders this call after
 * the calls that wrote the sources (stream order, or an event).                          */
sb_status sb_sum_scores(sb_ctx* ctx, float* dst, const float* const* src, int n_src, int64_t n,
                        int accumulate);

/* Block scores -- the hot loop (block partition: Section 4.1; marginal gains of one
 * precision step: Section 4.2, Eq. 6).  On the permuted layout
 * W'[r][j] = W[row_perm[r]][col_perm[j]], for every block i of block_rows x block_cols
 * (row-major over the block grid) and every candidate b_l = bits[l]:
 *     err[i][l]  = sum_{(r,j) in block i} a_r c_j (W'_rj - Q_{b_l}(W')_rj)^2
 *     gain[i][l] = (err[i][l] - err[i][l+1]) / ((b_{l+1} - b_l) * block_rows*block_cols)
 * with the same quantizer as above on groups of `group` consecutive columns of W'.
 * col_moment / row_weight are indexed by ORIGINAL column / row.  All candidates are
 * evaluated from registers in one pass over W; fp32 arithmetic, fixed summation order.
 * bits: host array, strictly ascending, each in 1..8, 1 <= n_bits <= 8.
 * R % block_rows == 0, C % block_cols == 0, block_cols % group == 0, block_rows % 4 == 0,
 * block_cols in {32,64} or a multiple of 128.
 * err: fp32 [(R/br)*(C/bc)][n_bits]; gain: fp32 [..][n_bits-1] or NULL;
 * W_perm_out: bf16 [R][C] (ld = C) receives W' or NULL.                              */
sb_status sb_block_scores(sb_ctx* ctx, const void* W_bf16, int64_t R, int64_t C, int64_t ldw,
                          const int32_t* row_perm, const int32_t* col_perm,
                          const float* col_moment, const float* row_weight,
                          int block_rows, int block_cols, int group,
                          const int* bits, int n_bits,
                          float* err, float* gain, void* W_perm_out_bf16);

typedef struct {
    int64_t cap_bits;            /* floor(budget * sum M_i), code bits only            */
    int64_t used_bits;           /* sum M_i * bits[level_i] of the result              */
    int32_t iterations;          /* Algorithm 2 loop iterations (greedy: steps taken)  */
    int32_t accepted;            /* accepted exchange steps                            */
    int32_t rejected;            /* rejected exchange steps (each halves k)            */
    int32_t expansions;          /* expansion steps                                    */
    double proxy_loss_init;      /* sum_i err[i][warm start]                           */
    double proxy_loss_final;     /* sum_i err[i][level_i]                              */
    int64_t level_hist[8];       /* blocks per level                                   */
} sb_alloc_report;

/* Global allocation (Eq. 1 with blocks weighted by their sizes M_i) on the separable
 * proxy loss L(level) = sum_i err[i][level_i].
 *   SB_ALLOC_SCALEBITS: Algorithm 2 -- warm start at the largest candidate <= budget,
 *     batches of k = floor(gamma N) blocks ranked by the gain of their next step up /
 *     down, expansion while the budget is slack (truncated so it is never exceeded),
 *     balanced exchange when it is active, accepted only if the proxy loss strictly
 *     falls, else k halves; stops when k < floor(gammaT N).
 *   SB_ALLOC_GREEDY: Algorithm 1 from the lowest candidate along each block's lower
 *     convex hull: all hull steps sorted by gain per bit, longest affordable prefix.
 * Ranking keys are IEEE binary64 quotients of the fp32 table entries; ties go to the
 * lower block index.  err: fp32 [N][n_bits].  block_elems: int64 [N] or NULL (then every
 * block has uniform_block_elems weights).  level: uint8 [N], index into bits[].
 * report: HOST struct, filled before return (the call synchronises the stream).        */
sb_status sb_allocate_bits(sb_ctx* ctx, const float* err, int64_t N,
                           const int64_t* block_elems, int64_t uniform_block_elems,
                           const int* bits, int n_bits, double budget_avg_bits,
                           int mode, double gamma0, double gammaT,
                           uint8_t* level, sb_alloc_report* report);

/* The same allocation (Algorithm 2 / Algorithm 1, same kernels, same results) without the
 * host round trip: everything is enqueued on the context's stream and the call returns, so
 * it can be captured in a CUDA graph between sb_block_scores and sb_pack_blocks.
 * report_dev: DEVICE struct, written in stream order after `level`; copy it back after a
 * synchronisation.  What the synchronous form reports after reading the device -- a lowest
 * candidate that does not fit the budget in greedy mode (SB_ERR_BUDGET; `level` is then all
 * zero), the iteration cap (SB_ERR_NOCONVERGE) -- is latched in the device status word and
 * returned by the next sb_sync.  Errors in the arguments are returned at once, as above.   */
sb_status sb_allocate_bits_async(sb_ctx* ctx, const float* err, int64_t N,
                                 const int64_t* block_elems, int64_t uniform_block_elems,
                                 const int* bits, int n_bits, double budget_avg_bits,
                                 int mode, double gamma0, double gammaT,
                                 uint8_t* level, sb_alloc_report* report_dev);

/* Pack (Section 5.3: one bitwidth per tile).  Quantise each block of W' at
 * bits[level[block]] with the same quantizer, evaluated in IEEE binary64 so that the
 * integer codes are reproducible: lo = min, range = max - min, inv = qmax / range,
 * q = clamp(rint((v - lo) * inv), 0, qmax) (round half to even), scale = range / qmax.
 * Layout: blocks in grid row-major order; inside a block the codes in block-row-major
 * order, code k in bits [k*b, (k+1)*b) of a little-endian stream of 32-bit words;
 * block_off_words[i] = first word of block i (exclusive prefix sum, [nb+1] entries);
 * meta[(r*(C/group) + g)] = {(float)scale, (float)lo} for group g of permuted row r.
 * If block_off_words[nb] > packed_capacity_words nothing beyond the capacity is written
 * and SB_ERR_SCRATCH is latched.  block_rows*block_cols*bits % 32 == 0 is required,
 * group in {16,32,64,128}, block_rows % 4 == 0.                                           */
sb_status sb_pack_blocks(sb_ctx* ctx, const void* W_bf16, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* row_perm, const int32_t* col_perm,
                         int block_rows, int block_cols, int group,
                         const int* bits, int n_bits, const uint8_t* level,
                         uint32_t* packed, int64_t packed_capacity_words,
                         int64_t* block_off_words, float* meta);

/* Fused mixed-precision dequantisation + matrix product on the output of sb_pack_blocks
 * (Section 5.3 and Table 4: dequantise tile by tile, one bitwidth per tile, and multiply):
 *     Y[t][r] = sum_c X[t][c] * (lo[r][g(c)] + scale[r][g(c)] * q[r][c])
 * in the packed (permuted) row and column order: X's columns are the packed columns, Y's
 * columns the packed rows.  The contraction runs on the integer codes (exact in bf16) on the
 * tensor cores with fp32 accumulation, one block at a time, and scale and lo are applied per
 * row and block in fp32; nothing else is rounded.
 *   - X: device bf16 [T][C], leading dimension ldx >= C; T >= 1 (tokens are processed in
 *     slices of 32, padded to 8, 16 or 32; decode batches are the intended use).
 *   - packed, block_off_words, meta, level, bits: as written by / given to sb_pack_blocks;
 *     packed 16-byte aligned.  Blocks of 64 x 128 (the paper's partition, Section 5
 *     "Implementation") or 128 x 128 with group = 128 are required.
 *   - Y: device fp32 [T][R], leading dimension ldy >= R, overwritten.
 * A pipeline wait that does not complete within 2 s latches SB_ERR_TIMEOUT.  Asynchronous. */
sb_status sb_dequant_gemm(sb_ctx* ctx, const void* X_bf16, int64_t T, int64_t ldx,
                          const uint32_t* packed, const int64_t* block_off_words, const float* meta,
                          const uint8_t* level, int64_t R, int64_t C,
                          int block_rows, int block_cols, int group, const int* bits, int n_bits,
                          float* Y, int64_t ldy);

/* Full calibration second-moment matrix on the tensor cores (Section 3.2: sb_calib_moments
 * returns the diagonal of this matrix; a sensitivity that keeps the cross terms between input
 * channels needs all of it):
 *     H[i][j] = (accumulate ? H[i][j] : 0) + scale * sum_t X[t][i] X[t][j]
 * X: device bf16 [T][K], leading dimension ldx (K % 8 == 0, ldx % 8 == 0, 16-byte aligned
 * base); H: device fp32 [K][K], row-major, both triangles written.  bf16 products are exact in
 * fp32, the sum over tokens is accumulated in fp32 by the tensor cores.  A pipeline wait that
 * does not complete within 2 s latches SB_ERR_TIMEOUT and the kernel returns.  Asynchronous. */
sb_status sb_calib_gram(sb_ctx* ctx, const void* X_bf16, int64_t T, int64_t K, int64_t ldx,
                        float* H, int accumulate, float scale);

/* Block error table with the full second-moment matrix (Section 3.2 with the cross terms
 * between input channels kept), on the permuted layout W' = W[row_perm][:, col_perm]:
 *     err[i][l]  = sum over rows r of block i of  d_r H'_JJ d_r^T,
 *                  d_r = (W' - Q_{b_l}(W'))[r, J],  J = the block's columns,
 *                  H'_JJ[a][b] = H[col_perm[J0 + a]][col_perm[J0 + b]]
 *     gain[i][l] = (err[i][l] - err[i][l+1]) / ((b_{l+1} - b_l) * block_rows * block_cols)
 * H: device fp32 [C][C] in the ORIGINAL column order (sb_calib_gram); symmetric.  With a
 * diagonal H this is sb_block_scores with col_moment = diag(H).  row_weight: [R] device fp32
 * by ORIGINAL row (non-negative) or NULL = 1: err sums a_r d_r H'_JJ d_r^T.  Blocks are 64, 128
 * or 256 rows x 64 or 128 columns (64 x 128 is the paper's default partition, Section 5
 * "Implementation"; C must be a multiple of 128), group in {16,32,64,128} and at most the block
 * width.  The 128 x 128 Gram matrix of every (128 rows x 128 columns, candidate) residual is a
 * tensor-core contraction of two bf16 terms of the residual (relative error about 2^-16); a
 * 64-row block contracts 64 zero rows along, a 256-row block is the sum of two units, two
 * 64-column blocks side by side take the two diagonal quadrants of one Gram matrix.  err, gain
 * (or NULL) and W_perm_out (or NULL) as in sb_block_scores.  A pipeline wait that does not
 * complete within 2 s latches SB_ERR_TIMEOUT.  Asynchronous.                                  */
sb_status sb_block_scores_full(sb_ctx* ctx, const void* W_bf16, int64_t R, int64_t C, int64_t ldw,
                               const int32_t* row_perm, const int32_t* col_perm, const float* H,
                               const float* row_weight, int block_rows, int block_cols, int group,
                               const int* bits, int n_bits, float* err, float* gain, void* W_perm_out_bf16);

/* First-order mode (Appendix E.3, "choice of sensitivity statistics"): the paper's own scores
 * for Algorithm 2 from a caller-supplied gradient G = dL/dw taken at the current quantized
 * model.  Every block is quantized at ITS current bitwidth b = bits[level[block]] on the
 * permuted layout W' = W[row_perm][:, col_perm], G' likewise:
 *     s_up[i]   = - sum over block i of G' (W' - Q_b(W'))      (gain of restoring the block; the
 *                                                               paper prints g^T (w - w^Q) and
 *                                                               ranks the largest first)
 *     s_down[i] = 2^-b * sum over block i of |G' Q_b(W')|
 *     s_l1[i]   = sum over block i of |G' (W' - Q_b(W'))|      (p = 1 element sensitivities of
 *                                                               Section 3.2, summed; optional)
 *   - W, G: device bf16 [R][C] row-major, leading dimensions ldw / ldg (multiples of 8,
 *     16-byte aligned bases); level: device uint8 [(R/br)*(C/bc)], blocks row-major over the
 *     grid; s_up, s_down, s_l1 (or NULL): device fp32 of the same length.
 *   - Shapes as sb_block_scores (group in {16,32,64,128} dividing block_cols, block_rows % 4
 *     == 0, block_cols in {32, 64} or a multiple of 128, C % 128 == 0).
 *   - fp32 accumulation: compare the signed sum at the scale of s_l1.  Non-finite sums latch
 *     SB_ERR_NONFINITE, a level >= n_bits latches SB_ERR_INVALID.  Asynchronous.             */
sb_status sb_first_order_scores(sb_ctx* ctx, const void* W_bf16, const void* G_bf16, int64_t R,
                                int64_t C, int64_t ldw, int64_t ldg, const int32_t* row_perm,
                                const int32_t* col_perm, int block_rows, int block_cols, int group,
                                const int* bits, int n_bits, const uint8_t* level, float* s_up,
                                float* s_down, float* s_l1);

/* Reorder statistics in the first-order form (Section 3.2 with p = 1, l1 channel aggregation
 * of Section 4.1): element sensitivity |G_rj (W_rj - Q(W)_rj)| at ref_bits on the ORIGINAL
 * layout, summed per row and per column.  Everything else (accumulate mask, segments, "sort
 * only" calls with W == NULL, permutations) as in sb_reorder_channels; G: device bf16 [R][C],
 * leading dimension ldg (a multiple of 8, 16-byte aligned base).                           */
sb_status sb_reorder_channels_first_order(sb_ctx* ctx, const void* W_bf16, const void* G_bf16,
                                          int64_t R, int64_t C, int64_t ldw, int64_t ldg,
                                          int ref_bits, int group,
                                          float* row_score, float* col_score, int accumulate,
                                          int64_t row_segment, int64_t col_segment,
                                          int32_t* row_perm, int32_t* col_perm);

/* One iteration of Algorithm 2 (lines 6-10) on per-block scores AT THE CURRENT LEVELS; the
 * caller refreshes the scores, evaluates the loss of level_out and decides on acceptance
 * (line 11) itself.  Rules as in sb_allocate_bits: one move = one level of the candidate list;
 * ranking keys per stored bit, s / ((b' - b) M_i) as a binary64 quotient of the fp32 scores,
 * ties to the lower block; up-eligible: not at the top level and s_up > 0; down-eligible:
 * not at the bottom level.  If the budget is not used up, the first k up-candidates are
 * raised, truncated to the longest prefix that fits (expansion); if nothing fits, or the
 * budget is used up, the first h = max(1, k/2) up-candidates and the first h down-candidates
 * outside that set are exchanged, the up set truncated to what the freed bits and the slack
 * pay for; an exchange with an empty side moves nothing.
 *   - s_up, s_down: device fp32 [N]; level, level_out: device uint8 [N] (may be the same
 *     buffer); block_elems: device int64 [N] or NULL with uniform_block_elems; budget in
 *     average code bits per weight; report: HOST memory, filled after an internal stream
 *     synchronisation (this call is synchronous).                                          */
typedef struct {
    int64_t cap_bits, used_in, used_out;
    int32_t expansion;      /* 1: expansion step, 0: exchange step                         */
    int32_t moved;          /* 0: level_out == level (nothing eligible or nothing fits)    */
    int64_t n_up, n_down;
    double sum_up, sum_down;    /* first-order change promised: sum_down - sum_up          */
} sb_step_report;
sb_status sb_exchange_step(sb_ctx* ctx, const float* s_up, const float* s_down, const uint8_t* level,
                           int64_t N, const int64_t* block_elems, int64_t uniform_block_elems,
                           const int* bits, int n_bits, double budget_avg_bits, int64_t k,
                           uint8_t* level_out, sb_step_report* report);

/* Allocation-free variant of sb_calib_moments (the paper has no counterpart: this entry
 * point exists for deployment, not for the method).  It is for callers that cannot allocate
 * device memory when they need the moments: a serving process whose device memory was
 * handed out in full at start-up, code running under a framework's caching allocator where
 * a raw cudaMalloc would synchronise the device and fragment the pool, a latency-critical
 * loop.  It needs no context and calls no cudaMalloc / cudaFree or any allocating routine:
 * its per-split partial sums live in a fixed 4 MiB array inside the library image, which
 * every GPU that loads the library holds until the process exits.
 *   - Same arithmetic, argument meaning and layout as sb_calib_moments; X, sumsq are DEVICE
 *     pointers on the CURRENT device (the caller makes it current); cuda_stream is a
 *     cudaStream_t (NULL = default stream).  Work is enqueued, not waited for.
 *   - K <= 65536; larger K returns SB_ERR_SCRATCH (and says so on stderr): split the columns
 *     across calls or use sb_calib_moments.  Other argument errors as in sb_calib_moments.
 *   - The first call on each device looks up the array's device address and asks the occupancy
 *     calculator how many CTAs of the kernel are resident per SM (the grid is one wave of them);
 *     neither allocates.  Make that first call before any stream capture begins.
 *   - All calls share the array and it keeps the previous call's contents.  Every partial
 *     that a call reads it has written first, so nothing needs clearing; but two calls whose
 *     kernels overlap on the GPU (e.g. on different streams) race on it and must be ordered
 *     by the caller.                                                                      */
sb_status sb_calib_moments_noalloc(void* cuda_stream, const void* X_bf16, int64_t T, int64_t K,
                                   int64_t ldx, float* sumsq, int accumulate, float scale);

#ifdef __cplusplus
}
#endif
#endif /* SCALEBITS_H_ */

/*
 * ScaleBITS bitwidth-search hot path -- CPU ORACLE (test infrastructure).
 *
 * A plain, slow, fp64 restatement of what the path computes, written from the
 * paper (arxiv 2602.17698).  It exists only so that tests, the smoke check and
 * the benchmark's cpu_baseline leg can compare the CUDA library against it.
 * It shares no code, header, table or helper with the CUDA path and is never
 * reached from the product.
 *
 * Every function takes HOST pointers.  bf16 tensors are passed as uint16_t bit
 * patterns.  All arithmetic is IEEE binary64, compiled with -ffp-contract=off.
 * Loops over independent rows / blocks carry an OpenMP pragma; nothing else is
 * blocked, fused or reordered.
 *
 * What the paper fixes and what is a reading of it:
 *   - Section 2 (Eq. 1): allocation problem; the budget is weighted by the block
 *     sizes M_i (identical to Eq. 1's 1/N sum when blocks are equal) and counts
 *     code bits only.
 *   - Section 3.2 (the two equations after Eq. 3): element sensitivity is a row
 *     factor times a column factor times the local distortion.  On this path the
 *     column factor is the calibration second moment c_j, the row factor an
 *     optional caller vector a_r, the distortion squared:
 *     sigma_rj = a_r c_j (W_rj - Q(W)_rj)^2.
 *   - Section 4.1: block-wise partition; bi-directional reordering = sort the
 *     channels by their summed element sensitivities, most sensitive first.
 *   - Section 5 "Implementation": round-to-nearest uniform scalar quantizer with
 *     groups along the input (column) axis.  The paper prints no formula; the
 *     reading here is asymmetric min-max, min-anchored, 2^b levels,
 *     round-half-to-even.
 *   - Algorithm 1 (classic greedy) and Algorithm 2 (scalable greedy) on the
 *     separable proxy loss L(b) = sum_i E[i][level_i].
 *   - Appendix E.3: the paper's own first-order scores s_up / s_down from a caller's
 *     gradient, and one iteration of Algorithm 2 on such scores
 *     (sbo_first_order_scores, sbo_exchange_step).
 *
 * Parity pins: see tests/test_oracle_*.py.  The exact trajectory of
 * sbo_allocate_scalebits (tie rules, odd k, budget truncation) is a reading of
 * Algorithm 2 that the paper does not pin: "parity unpinned" beyond the
 * invariants and tiny-instance optimum bounds tested there.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { SBO_OK = 0, SBO_ERR_INVALID = 1, SBO_ERR_SHAPE = 2, SBO_ERR_BUDGET = 3,
       SBO_ERR_NOCONVERGE = 6, SBO_ERR_NONFINITE = 7 };

typedef struct {
    int64_t cap_bits, used_bits;
    int32_t iterations, accepted, rejected, expansions;
    double proxy_loss_init, proxy_loss_final;
    int64_t level_hist[8];
    double min_margin;   /* smallest |dU-dD|/max(dU,dD) over exchange decisions */
} sbo_alloc_report;

int sbo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* bf16 = the upper 16 bits of an IEEE binary32 */
double sbo_bf16_to_f64(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---- calibration second moments: column factor of Section 3.2 ------------- */
/* out[j] (+)= scale * sum_t X[t][j]^2 */
void sbo_calib_moments(const uint16_t* X, int64_t T, int64_t K, int64_t ldx,
                       double scale, int accumulate, double* out) {
    #pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < K; ++j) {
        double s = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            double x = sbo_bf16_to_f64(X[t * ldx + j]);
            s += x * x;
        }
        s *= scale;
        out[j] = accumulate ? out[j] + s : s;
    }
}

/* ---- full calibration second-moment matrix -------------------------------- */
/* H[i][j] = scale * sum_t X[t][i] X[t][j]: the matrix whose diagonal sbo_calib_moments
 * returns (Section 3.2: the sensitivity "needs more than its diagonal" when cross terms
 * between input channels are kept).  Plain triple loop, upper triangle mirrored.          */
void sbo_calib_gram(const uint16_t* X, int64_t T, int64_t K, int64_t ldx, double scale, double* H) {
    #pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < K; ++i) {
        for (int64_t j = i; j < K; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t)
                s += sbo_bf16_to_f64(X[t * ldx + i]) * sbo_bf16_to_f64(X[t * ldx + j]);
            H[i * K + j] = s * scale;
        }
    }
    for (int64_t i = 0; i < K; ++i)
        for (int64_t j = 0; j < i; ++j) H[i * K + j] = H[j * K + i];
}

/* ---- the quantizer Q(., b) on one group (Section 5 "Implementation") ------ */
/* asymmetric min-max RTN, min-anchored:
 *   lo = min v, hi = max v, range = hi - lo, qmax = 2^b - 1
 *   range == 0: codes 0, scale 0, vhat = lo
 *   else inv = qmax / range; t = (v - lo) * inv; q = clamp(rint(t), 0, qmax)
 *        scale = range / qmax; vhat = lo + q * scale                          */
int sbo_quantize_group(const double* v, int g, int bits, int32_t* code, double* vhat,
                       double* scale_out, double* lo_out) {
    if (g <= 0 || bits < 1 || bits > 16) return SBO_ERR_INVALID;
    double lo = v[0], hi = v[0];
    for (int k = 1; k < g; ++k) {
        if (v[k] < lo) lo = v[k];
        if (v[k] > hi) hi = v[k];
    }
    const double qmax = (double)((1 << bits) - 1);
    const double range = hi - lo;
    double scale = 0.0;
    if (range == 0.0) {
        for (int k = 0; k < g; ++k) {
            if (code) code[k] = 0;
            if (vhat) vhat[k] = lo;
        }
    } else {
        const double inv = qmax / range;
        scale = range / qmax;
        for (int k = 0; k < g; ++k) {
            double t = (v[k] - lo) * inv;
            double q = nearbyint(t);            /* round-half-to-even */
            if (q < 0.0) q = 0.0;
            if (q > qmax) q = qmax;
            if (code) code[k] = (int32_t)q;
            if (vhat) {
                double prod = q * scale;
                vhat[k] = lo + prod;
            }
        }
    }
    if (scale_out) *scale_out = scale;
    if (lo_out) *lo_out = lo;
    return SBO_OK;
}

static int check_bits(const int* bits, int L) {
    if (L < 1 || L > 8) return 0;
    for (int l = 0; l < L; ++l) {
        if (bits[l] < 1 || bits[l] > 8) return 0;
        if (l > 0 && bits[l] <= bits[l - 1]) return 0;
    }
    return 1;
}

/* ---- reorder statistics (Section 4.1, Appendix D) -------------------------- */
/* On the ORIGINAL layout: fake-quantize every group of `group` consecutive
 * columns of a row at ref_bits, sigma_rj = a_r c_j (W_rj - What_rj)^2,
 * row_score[r] (+)= sum_j sigma_rj, col_score[j] (+)= sum_r sigma_rj.         */
int sbo_reorder_scores(const uint16_t* W, int64_t R, int64_t C, int64_t ldw,
                       const double* c, const double* a, int ref_bits, int group,
                       double* row_score, double* col_score, int accumulate) {
    if (group <= 0 || C % group != 0 || ref_bits < 1 || ref_bits > 8) return SBO_ERR_SHAPE;
    if (!accumulate) {
        if (row_score) for (int64_t r = 0; r < R; ++r) row_score[r] = 0.0;
        if (col_score) for (int64_t j = 0; j < C; ++j) col_score[j] = 0.0;
    }
    double* v = (double*)malloc(sizeof(double) * group);
    double* vh = (double*)malloc(sizeof(double) * group);
    /* rows in order: column sums accumulate in row order, row sums in column order */
    for (int64_t r = 0; r < R; ++r) {
        const double ar = a ? a[r] : 1.0;
        double rs = 0.0;
        for (int64_t j0 = 0; j0 < C; j0 += group) {
            for (int k = 0; k < group; ++k) v[k] = sbo_bf16_to_f64(W[r * ldw + j0 + k]);
            sbo_quantize_group(v, group, ref_bits, NULL, vh, NULL, NULL);
            for (int k = 0; k < group; ++k) {
                double d = v[k] - vh[k];
                double sigma = ar * c[j0 + k] * (d * d);
                rs += sigma;
                if (col_score) col_score[j0 + k] += sigma;
            }
        }
        if (row_score) row_score[r] += rs;
    }
    free(v); free(vh);
    return SBO_OK;
}

/* stable argsort, descending score, ties -> lower original index, independently
 * inside each segment of `segment` consecutive channels; perm[new] = old        */
static const double* g_sort_key;
static int cmp_desc_idx(const void* pa, const void* pb) {
    int32_t ia = *(const int32_t*)pa, ib = *(const int32_t*)pb;
    double ka = g_sort_key[ia], kb = g_sort_key[ib];
    if (ka > kb) return -1;
    if (ka < kb) return 1;
    return (ia > ib) - (ia < ib);
}
int sbo_argsort_desc_segments(const double* score, int64_t K, int64_t segment, int32_t* perm) {
    if (segment <= 0 || K % segment != 0) return SBO_ERR_SHAPE;
    for (int64_t i = 0; i < K; ++i) perm[i] = (int32_t)i;
    g_sort_key = score;
    for (int64_t s0 = 0; s0 < K; s0 += segment)
        qsort(perm + s0, (size_t)segment, sizeof(int32_t), cmp_desc_idx);
    return SBO_OK;
}

/* dst[h*seg + d] += sum_{u<reps} src[(h*reps + u)*seg + d]   (grouped-query heads
 * that share one value head share its channel permutation, Appendix D)          */
void sbo_fold_segment_scores(double* dst, const double* src, int64_t n_dst, int reps, int64_t seg) {
    for (int64_t i = 0; i < n_dst; ++i) {
        int64_t h = i / seg, d = i % seg;
        for (int u = 0; u < reps; ++u) dst[i] += src[(h * reps + u) * seg + d];
    }
}
/* out[(h*reps + u)*seg + d] = (h*reps + u)*seg + (perm[h*seg + d] - h*seg)     */
void sbo_expand_segment_perm(int32_t* out, const int32_t* perm, int64_t n_src, int reps, int64_t seg) {
    for (int64_t i = 0; i < n_src; ++i) {
        int64_t h = i / seg, d = i % seg;
        for (int u = 0; u < reps; ++u)
            out[(h * reps + u) * seg + d] = (int32_t)((h * reps + u) * seg + (perm[i] - h * seg));
    }
}

/* ---- block error table and marginal gains (Sections 4.1, 4.2) -------------- */
/* On the permuted layout W'[r][j] = W[rp[r]][cp[j]]:
 *   E[i][l]    = sum over block i of a_{rp[r]} c_{cp[j]} (W' - Q_{b_l}(W'))^2
 *   gain[i][l] = (E[i][l] - E[i][l+1]) / ((b_{l+1} - b_l) * M_i)
 * blocks row-major over the (R/br) x (C/bc) grid; groups are `group` consecutive
 * columns of the PERMUTED row and never straddle a block.                       */
int sbo_block_scores(const uint16_t* W, int64_t R, int64_t C, int64_t ldw,
                     const int32_t* row_perm, const int32_t* col_perm,
                     const double* c, const double* a,
                     int br, int bc, int group, const int* bits, int L,
                     double* err, double* gain) {
    if (!check_bits(bits, L)) return SBO_ERR_INVALID;
    if (br <= 0 || bc <= 0 || group <= 0 || R % br || C % bc || bc % group) return SBO_ERR_SHAPE;
    const int64_t nbr = R / br, nbc = C / bc;
    #pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * group);
        double* vh = (double*)malloc(sizeof(double) * group);
        #pragma omp for schedule(dynamic, 1)
        for (int64_t blk = 0; blk < nbr * nbc; ++blk) {
            const int64_t bi = blk / nbc, bj = blk % nbc;
            for (int l = 0; l < L; ++l) {
                double e = 0.0;
                for (int rr = 0; rr < br; ++rr) {
                    const int64_t r = bi * br + rr;
                    const int64_t rs = row_perm ? row_perm[r] : r;
                    const double ar = a ? a[rs] : 1.0;
                    for (int g0 = 0; g0 < bc; g0 += group) {
                        for (int k = 0; k < group; ++k) {
                            const int64_t j = bj * bc + g0 + k;
                            const int64_t js = col_perm ? col_perm[j] : j;
                            v[k] = sbo_bf16_to_f64(W[rs * ldw + js]);
                        }
                        sbo_quantize_group(v, group, bits[l], NULL, vh, NULL, NULL);
                        for (int k = 0; k < group; ++k) {
                            const int64_t j = bj * bc + g0 + k;
                            const int64_t js = col_perm ? col_perm[j] : j;
                            double d = v[k] - vh[k];
                            e += ar * c[js] * (d * d);
                        }
                    }
                }
                err[blk * L + l] = e;
            }
            if (gain) {
                const double M = (double)br * (double)bc;
                for (int l = 0; l + 1 < L; ++l)
                    gain[blk * (L - 1) + l] =
                        (err[blk * L + l] - err[blk * L + l + 1]) / ((double)(bits[l + 1] - bits[l]) * M);
            }
        }
        free(v); free(vh);
    }
    return SBO_OK;
}

/* ---- block error table with the full second-moment matrix ------------------- */
/* The sensitivity of Section 3.2 with the cross terms between input channels kept: for block i
 * with columns J (permuted layout) and candidate b_l,
 *   E[i][l] = sum over rows r of block i of  d_r H'_JJ d_r^T,   d_r = (W' - Q_{b_l}(W'))_{r,J},
 * where H' = H[cp][:, cp] is the calibration second-moment matrix (sbo_calib_gram) in the
 * permuted column order.  With a diagonal H this is sbo_block_scores with c = diag(H).         */
int sbo_block_scores_full(const uint16_t* W, int64_t R, int64_t C, int64_t ldw,
                          const int32_t* row_perm, const int32_t* col_perm, const double* H,
                          int br, int bc, int group, const int* bits, int L, double* err,
                          const double* row_weight /* [R] by original row, or NULL = 1 */) {
    if (!check_bits(bits, L)) return SBO_ERR_INVALID;
    if (br <= 0 || bc <= 0 || group <= 0 || R % br || C % bc || bc % group) return SBO_ERR_SHAPE;
    const int64_t nbr = R / br, nbc = C / bc;
    #pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * group);
        double* vh = (double*)malloc(sizeof(double) * group);
        double* d = (double*)malloc(sizeof(double) * bc);
        #pragma omp for schedule(dynamic, 1)
        for (int64_t blk = 0; blk < nbr * nbc; ++blk) {
            const int64_t bi = blk / nbc, bj = blk % nbc;
            for (int l = 0; l < L; ++l) {
                double e = 0.0;
                for (int rr = 0; rr < br; ++rr) {
                    const int64_t r = bi * br + rr;
                    const int64_t rs = row_perm ? row_perm[r] : r;
                    for (int g0 = 0; g0 < bc; g0 += group) {
                        for (int k = 0; k < group; ++k) {
                            const int64_t j = bj * bc + g0 + k;
                            const int64_t js = col_perm ? col_perm[j] : j;
                            v[k] = sbo_bf16_to_f64(W[rs * ldw + js]);
                        }
                        sbo_quantize_group(v, group, bits[l], NULL, vh, NULL, NULL);
                        for (int k = 0; k < group; ++k) d[g0 + k] = v[k] - vh[k];
                    }
                    for (int a = 0; a < bc; ++a) {
                        const int64_t ja = bj * bc + a;
                        const int64_t jas = col_perm ? col_perm[ja] : ja;
                        double s = 0.0;
                        for (int b = 0; b < bc; ++b) {
                            const int64_t jb = bj * bc + b;
                            const int64_t jbs = col_perm ? col_perm[jb] : jb;
                            s += H[jas * C + jbs] * d[b];
                        }
                        e += (row_weight ? row_weight[rs] : 1.0) * (d[a] * s);   /* a_r d_r H d_r^T */
                    }
                }
                err[blk * L + l] = e;
            }
        }
        free(v); free(vh); free(d);
    }
    return SBO_OK;
}

/* ---- allocation ------------------------------------------------------------ */
static inline int64_t blk_elems(const int64_t* block_elems, int64_t uniform, int64_t i) {
    return block_elems ? block_elems[i] : uniform;
}
/* per stored bit: (E[from] - E[to]) / ((b_to - b_from) * M_i), from < to */
static inline double step_gain(const double* err, int L, const int* bits, int64_t M, int64_t i,
                               int from, int to) {
    return (err[i * L + from] - err[i * L + to]) / ((double)(bits[to] - bits[from]) * (double)M);
}
static void fill_report(sbo_alloc_report* rep, const uint8_t* level, int64_t N) {
    for (int l = 0; l < 8; ++l) rep->level_hist[l] = 0;
    for (int64_t i = 0; i < N; ++i) rep->level_hist[level[i]]++;
}
static int64_t budget_cap(double budget, const int64_t* block_elems, int64_t uniform, int64_t N) {
    int64_t total = 0;
    for (int64_t i = 0; i < N; ++i) total += blk_elems(block_elems, uniform, i);
    return (int64_t)floor(budget * (double)total);
}

/* next step of block i on the lower convex hull of (b_l, E[i][l]) from level p:
 * the level q > p with E[q] < E[p] of largest slope (E[p]-E[q])/((b_q-b_p) M),
 * exact ties -> the farthest q.  Returns -1 when no level lowers E.             */
static int hull_next(const double* err, int L, const int* bits, int64_t M, int64_t i, int p,
                     double* slope_out) {
    int best = -1;
    double bs = 0.0;
    for (int q = p + 1; q < L; ++q) {
        if (!(err[i * L + q] < err[i * L + p])) continue;
        double s = step_gain(err, L, bits, M, i, p, q);
        if (best < 0 || s >= bs) { best = q; bs = s; }
    }
    if (slope_out) *slope_out = bs;
    return best;
}

/* Algorithm 1 (classic greedy) on the separable proxy: start every block at the
 * lowest candidate (0 bits is not a candidate), repeatedly give the step of
 * largest marginal gain per bit to one block, stop at the first step that does
 * not fit the budget.  Literal: one arg-max scan over all blocks per step.      */
int sbo_allocate_greedy(const double* err, int64_t N, const int64_t* block_elems, int64_t uniform,
                        const int* bits, int L, double budget, uint8_t* level,
                        sbo_alloc_report* rep) {
    if (!check_bits(bits, L) || N <= 0) return SBO_ERR_INVALID;
    memset(rep, 0, sizeof *rep);
    rep->min_margin = INFINITY;
    const int64_t cap = budget_cap(budget, block_elems, uniform, N);
    int64_t used = 0;
    double loss = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        level[i] = 0;
        used += blk_elems(block_elems, uniform, i) * bits[0];
        loss += err[i * L];
    }
    rep->cap_bits = cap; rep->proxy_loss_init = loss;
    if (used > cap) { rep->used_bits = used; return SBO_ERR_BUDGET; }
    for (;;) {
        int64_t bi = -1; int bq = -1; double bs = 0.0;
        for (int64_t i = 0; i < N; ++i) {
            double s;
            int q = hull_next(err, L, bits, blk_elems(block_elems, uniform, i), i, level[i], &s);
            if (q < 0) continue;
            if (bi < 0 || s > bs) { bi = i; bq = q; bs = s; }   /* ties -> lower block id */
        }
        if (bi < 0) break;
        int64_t cost = blk_elems(block_elems, uniform, bi) * (bits[bq] - bits[level[bi]]);
        if (cost > cap - used) break;
        loss += err[bi * L + bq] - err[bi * L + level[bi]];
        used += cost;
        level[bi] = (uint8_t)bq;
        rep->iterations++;
    }
    rep->accepted = rep->iterations;
    rep->used_bits = used; rep->proxy_loss_final = loss;
    fill_report(rep, level, N);
    return SBO_OK;
}

/* Same selection rule as sbo_allocate_greedy with the arg-max kept in a binary
 * heap ordered by (slope desc, block id asc); for sizes where the literal scan is
 * too slow.  Pinned against the literal version in the tests.                   */
typedef struct { double s; int64_t i; int q; } heap_item;
static int heap_before(const heap_item* x, const heap_item* y) {
    if (x->s != y->s) return x->s > y->s;
    return x->i < y->i;
}
static void heap_push(heap_item* h, int64_t* n, heap_item it) {
    int64_t k = (*n)++;
    h[k] = it;
    while (k > 0) {
        int64_t p = (k - 1) / 2;
        if (!heap_before(&h[k], &h[p])) break;
        heap_item t = h[k]; h[k] = h[p]; h[p] = t; k = p;
    }
}
static heap_item heap_pop(heap_item* h, int64_t* n) {
    heap_item top = h[0];
    h[0] = h[--(*n)];
    int64_t k = 0;
    for (;;) {
        int64_t l = 2 * k + 1, r = l + 1, m = k;
        if (l < *n && heap_before(&h[l], &h[m])) m = l;
        if (r < *n && heap_before(&h[r], &h[m])) m = r;
        if (m == k) break;
        heap_item t = h[k]; h[k] = h[m]; h[m] = t; k = m;
    }
    return top;
}
int sbo_allocate_greedy_heap(const double* err, int64_t N, const int64_t* block_elems,
                             int64_t uniform, const int* bits, int L, double budget,
                             uint8_t* level, sbo_alloc_report* rep) {
    if (!check_bits(bits, L) || N <= 0) return SBO_ERR_INVALID;
    memset(rep, 0, sizeof *rep);
    rep->min_margin = INFINITY;
    const int64_t cap = budget_cap(budget, block_elems, uniform, N);
    int64_t used = 0;
    double loss = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        level[i] = 0;
        used += blk_elems(block_elems, uniform, i) * bits[0];
        loss += err[i * L];
    }
    rep->cap_bits = cap; rep->proxy_loss_init = loss;
    if (used > cap) { rep->used_bits = used; return SBO_ERR_BUDGET; }
    heap_item* h = (heap_item*)malloc(sizeof(heap_item) * (size_t)N);
    int64_t n = 0;
    for (int64_t i = 0; i < N; ++i) {
        heap_item it; it.i = i;
        it.q = hull_next(err, L, bits, blk_elems(block_elems, uniform, i), i, 0, &it.s);
        if (it.q >= 0) heap_push(h, &n, it);
    }
    while (n > 0) {
        heap_item it = heap_pop(h, &n);
        int64_t cost = blk_elems(block_elems, uniform, it.i) * (bits[it.q] - bits[level[it.i]]);
        if (cost > cap - used) break;
        loss += err[it.i * L + it.q] - err[it.i * L + level[it.i]];
        used += cost;
        level[it.i] = (uint8_t)it.q;
        rep->iterations++;
        heap_item nx; nx.i = it.i;
        nx.q = hull_next(err, L, bits, blk_elems(block_elems, uniform, it.i), it.i, it.q, &nx.s);
        if (nx.q >= 0) heap_push(h, &n, nx);
    }
    free(h);
    rep->accepted = rep->iterations;
    rep->used_bits = used; rep->proxy_loss_final = loss;
    fill_report(rep, level, N);
    return SBO_OK;
}

/* Algorithm 2 (scalable greedy search) with the static table as the loss:
 * warm start at the largest candidate <= B, batches of k = floor(gamma N) blocks,
 * expansion while the budget is slack, balanced exchange when it is active,
 * accept an exchange only if the proxy loss strictly falls, else halve k.        */
typedef struct { double key; int64_t i; } rank_item;
static int cmp_key_desc(const void* pa, const void* pb) {
    const rank_item* x = (const rank_item*)pa; const rank_item* y = (const rank_item*)pb;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
static int cmp_key_asc(const void* pa, const void* pb) {
    const rank_item* x = (const rank_item*)pa; const rank_item* y = (const rank_item*)pb;
    if (x->key < y->key) return -1;
    if (x->key > y->key) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
/* `trace` (optional, [trace_iters][N]): the level vector as it stands at the end of every
 * iteration of the while loop (accepted, rejected or expansion), for the first trace_iters
 * iterations.  Recording only: the arithmetic does not depend on it.                    */
static int allocate_scalebits_core(const double* err, int64_t N, const int64_t* block_elems,
                           int64_t uniform, const int* bits, int L, double budget,
                           double gamma0, double gammaT, uint8_t* level, sbo_alloc_report* rep,
                           uint8_t* trace, int64_t trace_iters) {
#define SBO_TRACE_ITERATION()                                                             \
    do {                                                                                  \
        if (trace && rep->iterations >= 1 && rep->iterations <= trace_iters)              \
            memcpy(trace + (size_t)(rep->iterations - 1) * (size_t)N, level, (size_t)N);  \
    } while (0)
    if (!check_bits(bits, L) || N <= 0) return SBO_ERR_INVALID;
    if (!(gamma0 > 0.0) || !(gammaT > 0.0) || gamma0 > 1.0 || gammaT > 1.0) return SBO_ERR_INVALID;
    memset(rep, 0, sizeof *rep);
    rep->min_margin = INFINITY;
    const int64_t cap = budget_cap(budget, block_elems, uniform, N);
    rep->cap_bits = cap;
    int l0 = -1;
    for (int l = 0; l < L; ++l) if ((double)bits[l] <= budget) l0 = l;   /* warm start */
    if (l0 < 0) return SBO_ERR_BUDGET;
    int64_t k = (int64_t)floor(gamma0 * (double)N); if (k < 1) k = 1;
    int64_t kT = (int64_t)floor(gammaT * (double)N); if (kT < 1) kT = 1;
    if (k < kT) k = kT;
    double loss = 0.0; int64_t used = 0;
    for (int64_t i = 0; i < N; ++i) {
        level[i] = (uint8_t)l0;
        loss += err[i * L + l0];
        used += blk_elems(block_elems, uniform, i) * bits[l0];
    }
    rep->proxy_loss_init = loss;
    rank_item* up = (rank_item*)malloc(sizeof(rank_item) * (size_t)N);
    rank_item* dn = (rank_item*)malloc(sizeof(rank_item) * (size_t)N);
    uint8_t* inU0 = (uint8_t*)malloc((size_t)N);
    int status = SBO_OK;
    while (k >= kT) {
        SBO_TRACE_ITERATION();                          /* the iteration that just ended */
        if (++rep->iterations > 4096) { status = SBO_ERR_NOCONVERGE; break; }
        /* refresh s_up / s_down at the current allocation */
        int64_t nup = 0;
        for (int64_t i = 0; i < N; ++i) {
            if (level[i] < L - 1) {
                double s = step_gain(err, L, bits, blk_elems(block_elems, uniform, i), i,
                                     level[i], level[i] + 1);
                if (s > 0.0) { up[nup].key = s; up[nup].i = i; ++nup; }
            }
        }
        qsort(up, (size_t)nup, sizeof(rank_item), cmp_key_desc);
        if (used < cap) {                               /* expansion stage */
            int64_t take = 0, cum = 0;
            for (int64_t p = 0; p < nup && p < k; ++p) {
                int64_t i = up[p].i;
                int64_t cost = blk_elems(block_elems, uniform, i) * (bits[level[i] + 1] - bits[level[i]]);
                if (used + cum + cost > cap) break;
                cum += cost; ++take;
            }
            if (take > 0) {
                for (int64_t p = 0; p < take; ++p) {
                    int64_t i = up[p].i;
                    loss += err[i * L + level[i] + 1] - err[i * L + level[i]];
                    level[i]++;
                }
                used += cum;
                rep->expansions++;
                continue;
            }
        }
        /* exchange stage */
        int64_t h = k / 2; if (h < 1) h = 1;
        memset(inU0, 0, (size_t)N);
        int64_t nU0 = nup < h ? nup : h;
        for (int64_t p = 0; p < nU0; ++p) inU0[up[p].i] = 1;
        int64_t ndn = 0;
        for (int64_t i = 0; i < N; ++i) {
            if (level[i] > 0 && !inU0[i]) {
                dn[ndn].key = step_gain(err, L, bits, blk_elems(block_elems, uniform, i), i,
                                        level[i] - 1, level[i]);
                dn[ndn].i = i; ++ndn;
            }
        }
        qsort(dn, (size_t)ndn, sizeof(rank_item), cmp_key_asc);
        int64_t nD = ndn < h ? ndn : h;
        int64_t freed = 0; double dD = 0.0;
        for (int64_t p = 0; p < nD; ++p) {
            int64_t i = dn[p].i;
            freed += blk_elems(block_elems, uniform, i) * (bits[level[i]] - bits[level[i] - 1]);
            dD += err[i * L + level[i] - 1] - err[i * L + level[i]];
        }
        int64_t nU = 0, costU = 0; double dU = 0.0;
        for (int64_t p = 0; p < nU0; ++p) {
            int64_t i = up[p].i;
            int64_t cost = blk_elems(block_elems, uniform, i) * (bits[level[i] + 1] - bits[level[i]]);
            if (costU + cost > freed + (cap - used)) break;
            costU += cost; ++nU;
            dU += err[i * L + level[i]] - err[i * L + level[i] + 1];
        }
        if (nU > 0 && nD > 0) {
            double mx = fabs(dU) > fabs(dD) ? fabs(dU) : fabs(dD);
            double margin = mx > 0.0 ? fabs(dU - dD) / mx : 0.0;
            if (margin < rep->min_margin) rep->min_margin = margin;
        }
        if (nU > 0 && nD > 0 && dU > dD) {
            for (int64_t p = 0; p < nU; ++p) level[up[p].i]++;
            for (int64_t p = 0; p < nD; ++p) level[dn[p].i]--;
            loss += dD - dU;
            used += costU - freed;
            rep->accepted++;
        } else {
            k /= 2;
            rep->rejected++;
        }
    }
    SBO_TRACE_ITERATION();
#undef SBO_TRACE_ITERATION
    free(up); free(dn); free(inU0);
    rep->used_bits = used; rep->proxy_loss_final = loss;
    fill_report(rep, level, N);
    return status;
}

int sbo_allocate_scalebits(const double* err, int64_t N, const int64_t* block_elems,
                           int64_t uniform, const int* bits, int L, double budget,
                           double gamma0, double gammaT, uint8_t* level, sbo_alloc_report* rep) {
    return allocate_scalebits_core(err, N, block_elems, uniform, bits, L, budget, gamma0, gammaT,
                                   level, rep, NULL, 0);
}

/* The same search, also returning the level vector after each of the first trace_iters
 * iterations (for checking a trajectory worked by hand from Algorithm 2's text).        */
int sbo_allocate_scalebits_trace(const double* err, int64_t N, const int64_t* block_elems,
                                 int64_t uniform, const int* bits, int L, double budget,
                                 double gamma0, double gammaT, uint8_t* level,
                                 sbo_alloc_report* rep, uint8_t* trace, int64_t trace_iters) {
    return allocate_scalebits_core(err, N, block_elems, uniform, bits, L, budget, gamma0, gammaT,
                                   level, rep, trace, trace_iters);
}

/* ---- first-order statistics of the current allocation (Appendix E.3) --------- */
/* The paper's own scores for Algorithm 2: with g = dL/dw evaluated at the current quantized
 * model and every block i quantized at ITS current bitwidth b = bits[level[i]],
 *   s_up[i]   = - sum over block i of G (W' - Q_b(W'))     (first-order loss decrease of moving
 *                                                            the block back to full precision;
 *                                                            the paper prints g^T (w - w^Q) and
 *                                                            ranks the LARGEST first, so the gain
 *                                                            is read with the minus sign)
 *   s_down[i] = 2^-b * sum over block i of |G * Q_b(W')|   (expected magnitude of the increase)
 *   s_l1[i]   = sum over block i of |G (W' - Q_b(W'))|     (the p = 1 element sensitivity of
 *                                                            Section 3.2, summed: the scale the
 *                                                            signed sum is compared at)
 * on the permuted layout, W' = W[rp][:, cp], G' = G[rp][:, cp].                              */
int sbo_first_order_scores(const uint16_t* W, const uint16_t* G, int64_t R, int64_t C, int64_t ldw,
                           int64_t ldg, const int32_t* row_perm, const int32_t* col_perm,
                           int br, int bc, int group, const int* bits, int L, const uint8_t* level,
                           double* s_up, double* s_down, double* s_l1) {
    if (!check_bits(bits, L)) return SBO_ERR_INVALID;
    if (br <= 0 || bc <= 0 || group <= 0 || R % br || C % bc || bc % group) return SBO_ERR_SHAPE;
    const int64_t nbr = R / br, nbc = C / bc;
    for (int64_t blk = 0; blk < nbr * nbc; ++blk)
        if (level[blk] >= L) return SBO_ERR_INVALID;
    #pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * group);
        double* vh = (double*)malloc(sizeof(double) * group);
        #pragma omp for schedule(dynamic, 1)
        for (int64_t blk = 0; blk < nbr * nbc; ++blk) {
            const int64_t bi = blk / nbc, bj = blk % nbc;
            const int b = bits[level[blk]];
            double up = 0.0, down = 0.0, l1 = 0.0;
            for (int rr = 0; rr < br; ++rr) {
                const int64_t r = bi * br + rr;
                const int64_t rs = row_perm ? row_perm[r] : r;
                for (int g0 = 0; g0 < bc; g0 += group) {
                    for (int k = 0; k < group; ++k) {
                        const int64_t j = bj * bc + g0 + k;
                        const int64_t js = col_perm ? col_perm[j] : j;
                        v[k] = sbo_bf16_to_f64(W[rs * ldw + js]);
                    }
                    sbo_quantize_group(v, group, b, NULL, vh, NULL, NULL);
                    for (int k = 0; k < group; ++k) {
                        const int64_t j = bj * bc + g0 + k;
                        const int64_t js = col_perm ? col_perm[j] : j;
                        const double g = sbo_bf16_to_f64(G[rs * ldg + js]);
                        const double t = g * (v[k] - vh[k]);
                        up -= t;
                        l1 += fabs(t);
                        down += fabs(g * vh[k]);
                    }
                }
            }
            s_up[blk] = up;
            s_down[blk] = ldexp(down, -b);
            if (s_l1) s_l1[blk] = l1;
        }
        free(v); free(vh);
    }
    return SBO_OK;
}

/* ---- reorder statistics, first-order form (Section 3.2, p = 1) --------------- */
/* The element sensitivity of Section 3.2 in the form the paper uses with gradients,
 * sigma_rj = |G_rj (W_rj - Q(W)_rj)|, on the ORIGINAL layout at ref_bits, aggregated per channel
 * with the l1 norm (Section 4.1): row_score[r] (+)= sum_j sigma_rj, col_score[j] (+)= sum_r.   */
int sbo_reorder_scores_first_order(const uint16_t* W, const uint16_t* G, int64_t R, int64_t C,
                                   int64_t ldw, int64_t ldg, int ref_bits, int group,
                                   double* row_score, double* col_score, int accumulate) {
    if (group <= 0 || C % group != 0 || ref_bits < 1 || ref_bits > 8) return SBO_ERR_SHAPE;
    if (!accumulate) {
        if (row_score) for (int64_t r = 0; r < R; ++r) row_score[r] = 0.0;
        if (col_score) for (int64_t j = 0; j < C; ++j) col_score[j] = 0.0;
    }
    double* v = (double*)malloc(sizeof(double) * group);
    double* vh = (double*)malloc(sizeof(double) * group);
    for (int64_t r = 0; r < R; ++r) {
        double rs = 0.0;
        for (int64_t j0 = 0; j0 < C; j0 += group) {
            for (int k = 0; k < group; ++k) v[k] = sbo_bf16_to_f64(W[r * ldw + j0 + k]);
            sbo_quantize_group(v, group, ref_bits, NULL, vh, NULL, NULL);
            for (int k = 0; k < group; ++k) {
                const double sigma = fabs(sbo_bf16_to_f64(G[r * ldg + j0 + k]) * (v[k] - vh[k]));
                rs += sigma;
                if (col_score) col_score[j0 + k] += sigma;
            }
        }
        if (row_score) row_score[r] += rs;
    }
    free(v); free(vh);
    return SBO_OK;
}

/* ---- one iteration of Algorithm 2 on caller-supplied scores ------------------- */
/* Lines 6-10 of Algorithm 2 with s_up / s_down given per block AT ITS CURRENT LEVEL (they change
 * with the model, so the caller refreshes them and decides on acceptance, line 11, itself).
 * Same readings as sbo_allocate_scalebits: one move = one level of the candidate list; ranking
 * keys per stored bit, s / ((b' - b) M_i), ties to the lower block; up-eligible: not at the
 * top level and s_up > 0; down-eligible: not at the bottom level; the expansion is truncated
 * to the longest prefix that fits the budget and, if nothing fits, the exchange runs instead;
 * the up set is chosen first and the down set excludes it; U is the longest prefix of the up
 * set whose cost fits the slack plus what D frees.  An exchange with an empty U or D moves
 * nothing.                                                                                    */
typedef struct {
    int64_t cap_bits, used_in, used_out;
    int32_t expansion;          /* 1: expansion step, 0: exchange step                          */
    int32_t moved;              /* 0: nothing fits / nothing eligible: level_out == level       */
    int64_t n_up, n_down;
    double sum_up, sum_down;    /* first-order change promised: -sum_up + sum_down              */
} sbo_step_report;

int sbo_exchange_step(const double* s_up, const double* s_down, const uint8_t* level, int64_t N,
                      const int64_t* block_elems, int64_t uniform, const int* bits, int L,
                      double budget, int64_t k, uint8_t* level_out, sbo_step_report* rep) {
    if (!check_bits(bits, L) || N <= 0 || k < 1) return SBO_ERR_INVALID;
    memset(rep, 0, sizeof *rep);
    const int64_t cap = budget_cap(budget, block_elems, uniform, N);
    int64_t used = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (level[i] >= L) return SBO_ERR_INVALID;
        used += blk_elems(block_elems, uniform, i) * bits[level[i]];
        level_out[i] = level[i];
    }
    rep->cap_bits = cap; rep->used_in = used; rep->used_out = used;
    rank_item* up = (rank_item*)malloc(sizeof(rank_item) * (size_t)N);
    rank_item* dn = (rank_item*)malloc(sizeof(rank_item) * (size_t)N);
    char* in_up = (char*)calloc((size_t)N, 1);
    int64_t nu = 0, nd = 0;
    for (int64_t i = 0; i < N; ++i) {
        const int l = level[i];
        const double M = (double)blk_elems(block_elems, uniform, i);
        if (l + 1 < L && s_up[i] > 0.0) {
            up[nu].key = s_up[i] / ((double)(bits[l + 1] - bits[l]) * M);
            up[nu].i = i; ++nu;
        }
    }
    qsort(up, (size_t)nu, sizeof(rank_item), cmp_key_desc);
    const int64_t slack = cap - used;
    if (used < cap) {                                   /* expansion stage */
        int64_t cum = 0, taken = 0;
        for (int64_t p = 0; p < nu && p < k; ++p) {
            const int64_t i = up[p].i; const int l = level[i];
            const int64_t cost = blk_elems(block_elems, uniform, i) * (bits[l + 1] - bits[l]);
            if (cum + cost > slack) break;
            cum += cost; ++taken;
            level_out[i] = (uint8_t)(l + 1);
            rep->sum_up += s_up[i];
        }
        if (taken > 0) {
            rep->expansion = 1; rep->moved = 1; rep->n_up = taken; rep->used_out = used + cum;
            free(up); free(dn); free(in_up);
            return SBO_OK;
        }
    }
    /* exchange stage */
    const int64_t h = k / 2 > 0 ? k / 2 : 1;
    const int64_t nu0 = nu < h ? nu : h;
    for (int64_t p = 0; p < nu0; ++p) in_up[up[p].i] = 1;
    for (int64_t i = 0; i < N; ++i) {
        const int l = level[i];
        if (l > 0 && !in_up[i]) {
            const double M = (double)blk_elems(block_elems, uniform, i);
            dn[nd].key = s_down[i] / ((double)(bits[l] - bits[l - 1]) * M);
            dn[nd].i = i; ++nd;
        }
    }
    qsort(dn, (size_t)nd, sizeof(rank_item), cmp_key_asc);
    const int64_t nd0 = nd < h ? nd : h;
    int64_t freed = 0;
    for (int64_t p = 0; p < nd0; ++p) {
        const int64_t i = dn[p].i; const int l = level[i];
        freed += blk_elems(block_elems, uniform, i) * (bits[l] - bits[l - 1]);
    }
    int64_t cum = 0, taken = 0;
    for (int64_t p = 0; p < nu0; ++p) {
        const int64_t i = up[p].i; const int l = level[i];
        const int64_t cost = blk_elems(block_elems, uniform, i) * (bits[l + 1] - bits[l]);
        if (cum + cost > slack + freed) break;
        cum += cost; ++taken;
    }
    if (taken > 0 && nd0 > 0) {
        for (int64_t p = 0; p < taken; ++p) {
            const int64_t i = up[p].i;
            level_out[i] = (uint8_t)(level[i] + 1);
            rep->sum_up += s_up[i];
        }
        for (int64_t p = 0; p < nd0; ++p) {
            const int64_t i = dn[p].i;
            level_out[i] = (uint8_t)(level[i] - 1);
            rep->sum_down += s_down[i];
        }
        rep->moved = 1; rep->n_up = taken; rep->n_down = nd0; rep->used_out = used + cum - freed;
    }
    free(up); free(dn); free(in_up);
    return SBO_OK;
}

/* ---- packing (Section 5.3: uniform bitwidth per tile) ----------------------- */
/* Per block (grid row-major), the codes of the block in block-row-major order,
 * code k in bits [k*b, (k+1)*b) of a little-endian stream of 32-bit words;
 * block_off_words = exclusive prefix sum of the block sizes in words;
 * meta[(r*(C/group) + gidx)] = ((float)scale, (float)lo) in permuted row-major
 * group order.                                                                  */
int sbo_pack_blocks(const uint16_t* W, int64_t R, int64_t C, int64_t ldw,
                    const int32_t* row_perm, const int32_t* col_perm,
                    int br, int bc, int group, const int* bits, int L, const uint8_t* level,
                    uint32_t* packed, int64_t capacity_words, int64_t* block_off_words,
                    float* meta) {
    if (!check_bits(bits, L)) return SBO_ERR_INVALID;
    if (br <= 0 || bc <= 0 || group <= 0 || R % br || C % bc || bc % group) return SBO_ERR_SHAPE;
    const int64_t nbr = R / br, nbc = C / bc, ngc = C / group;
    int64_t off = 0;
    for (int64_t blk = 0; blk < nbr * nbc; ++blk) {
        if (level[blk] >= L) return SBO_ERR_INVALID;
        block_off_words[blk] = off;
        int64_t nbits = (int64_t)br * bc * bits[level[blk]];
        if (nbits % 32) return SBO_ERR_SHAPE;
        off += nbits / 32;
    }
    block_off_words[nbr * nbc] = off;
    if (off > capacity_words) return SBO_ERR_SHAPE;
    memset(packed, 0, sizeof(uint32_t) * (size_t)off);
    double* v = (double*)malloc(sizeof(double) * group);
    int32_t* code = (int32_t*)malloc(sizeof(int32_t) * group);
    for (int64_t blk = 0; blk < nbr * nbc; ++blk) {
        const int64_t bi = blk / nbc, bj = blk % nbc;
        const int b = bits[level[blk]];
        uint32_t* out = packed + block_off_words[blk];
        for (int rr = 0; rr < br; ++rr) {
            const int64_t r = bi * br + rr;
            const int64_t rs = row_perm ? row_perm[r] : r;
            for (int g0 = 0; g0 < bc; g0 += group) {
                for (int k = 0; k < group; ++k) {
                    const int64_t j = bj * bc + g0 + k;
                    v[k] = sbo_bf16_to_f64(W[rs * ldw + (col_perm ? col_perm[j] : j)]);
                }
                double scale, lo;
                sbo_quantize_group(v, group, b, code, NULL, &scale, &lo);
                const int64_t gi = r * ngc + (bj * bc + g0) / group;
                meta[2 * gi] = (float)scale;
                meta[2 * gi + 1] = (float)lo;
                for (int k = 0; k < group; ++k) {
                    int64_t e = (int64_t)rr * bc + g0 + k;      /* element index in the block */
                    int64_t bit = e * b;
                    uint64_t val = ((uint64_t)(uint32_t)code[k]) << (bit % 32);
                    out[bit / 32] |= (uint32_t)val;
                    if ((bit % 32) + b > 32) out[bit / 32 + 1] |= (uint32_t)(val >> 32);
                }
            }
        }
    }
    free(v); free(code);
    return SBO_OK;
}

/* Fused dequantisation + matrix product on the packed format (Section 5.3, Table 4: the
 * mixed-precision kernel dequantises tile by tile, one bitwidth per tile, and multiplies):
 *     Y[t][r] = sum_c X[t][c] * What[r][c],   What[r][c] = lo[r][g(c)] + scale[r][g(c)] * q[r][c],
 * q read back from the bit stream sbo_pack_blocks wrote (code k of a block in bits
 * [k b, (k+1) b) of its little-endian word stream, block-row-major), scale and lo the fp32
 * metadata of (row, group).  Rows and columns are those of the packed (permuted) layout.
 * Plain definition in binary64: decode every code, form What, accumulate the dot products.
 * X: bf16 [T][C] (ldx), Y: binary64 [T][R]. */
int sbo_dequant_gemm(const uint16_t* X, int64_t T, int64_t ldx, const uint32_t* packed,
                     const int64_t* block_off_words, const float* meta, const uint8_t* level,
                     int64_t R, int64_t C, int br, int bc, int group, const int* bits, int L,
                     double* Y) {
    if (!check_bits(bits, L)) return SBO_ERR_INVALID;
    if (br <= 0 || bc <= 0 || group <= 0 || R % br || C % bc || bc % group) return SBO_ERR_SHAPE;
    const int64_t nbc = C / bc, ngc = C / group;
    double* what = (double*)malloc(sizeof(double) * (size_t)C);
    for (int64_t r = 0; r < R; ++r) {
        const int64_t bi = r / br;
        const int rr = (int)(r % br);
        for (int64_t j = 0; j < C; ++j) {
            const int64_t bj = j / bc;
            const int64_t blk = bi * nbc + bj;
            if (level[blk] >= L) { free(what); return SBO_ERR_INVALID; }
            const int b = bits[level[blk]];
            const uint32_t* in = packed + block_off_words[blk];
            const int64_t e = (int64_t)rr * bc + (j % bc);       /* element index in the block */
            const int64_t bit = e * b;
            uint64_t word = in[bit / 32];
            if ((bit % 32) + b > 32) word |= (uint64_t)in[bit / 32 + 1] << 32;
            const uint32_t q = (uint32_t)((word >> (bit % 32)) & ((1u << b) - 1u));
            const int64_t gi = r * ngc + j / group;
            what[j] = (double)meta[2 * gi + 1] + (double)meta[2 * gi] * (double)q;
        }
        for (int64_t t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int64_t j = 0; j < C; ++j) acc += sbo_bf16_to_f64(X[t * ldx + j]) * what[j];
            Y[t * R + r] = acc;
        }
    }
    free(what);
    return SBO_OK;
}

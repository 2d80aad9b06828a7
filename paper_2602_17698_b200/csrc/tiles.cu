// Weight-tile kernels: permuted gather, reorder statistics, block scores (the hot loop),
// rank-by-counting argsort, and the small grouped-query helpers.
//
// Quantizer (Section 5 "Implementation": round-to-nearest uniform, groups along the input
// axis; asymmetric min-max, min-anchored): per (row, group) lo = min, range = max - min,
// t = (v - lo) * qmax / range, q = rint(t), v - vhat = (v - lo) - q * range / qmax.
// The kernels keep a lane on FIXED columns while it walks the rows of a tile, so the
// column factor c_j multiplies the per-column accumulators once per tile instead of once
// per element, and every candidate bitwidth is evaluated from the same registers.
#include "common.cuh"

namespace {

constexpr int TILE_COLS = 128;
constexpr int CTA_THREADS = 256;
constexpr int CTA_WARPS = CTA_THREADS / 32;
constexpr float RNE_MAGIC = 12582912.f;        // 1.5 * 2^23: fma(x, s, MAGIC) - MAGIC = rint(x*s)
constexpr float MIN_RANGE = 7.52316385e-37f;   // 2^-120: below this a group counts as constant

struct BitsArg {
    float qmax[8];       // 2^b - 1
    float inv_qmax[8];   // 1 / (2^b - 1)
    int bits[8];
};

__device__ __forceinline__ uint32_t u32(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ __nv_bfloat162 b162(uint32_t v) { return *reinterpret_cast<__nv_bfloat162*>(&v); }

// min and max of a group: NW packed words per lane, `team` lanes (a power of two, aligned)
// per group.  Exact: bf16 min/max, the pair (min, -max) rides one register through the
// shuffles.
template <int NW>
__device__ __forceinline__ void group_minmax(const uint32_t (&w)[NW], int team, float& lo, float& hi) {
    __nv_bfloat162 mn = b162(w[0]), mx = mn;
#pragma unroll
    for (int k = 1; k < NW; ++k) {
        mn = __hmin2(mn, b162(w[k]));
        mx = __hmax2(mx, b162(w[k]));
    }
    const uint32_t mnu = u32(mn), mxu = u32(mx);
    const uint32_t a = u32(__hmin2(mn, b162(__byte_perm(mnu, mnu, 0x1032))));
    const uint32_t b = u32(__hmax2(mx, b162(__byte_perm(mxu, mxu, 0x1032)))) ^ 0x80008000u;
    uint32_t p = (a & 0x0000ffffu) | (b & 0xffff0000u);
    for (int o = team >> 1; o > 0; o >>= 1)
        p = u32(__hmin2(b162(p), b162(__shfl_xor_sync(0xffffffffu, p, o))));
    lo = bf16lo(p);
    hi = -bf16hi(p);
}

__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// ---- permuted gather: out[r][j] = W[rp[r]][cp[j]] ---------------------------------------
// One source row is staged in shared memory with coalesced 16-byte loads, then read in
// permuted order; 2-byte scattered reads never reach HBM.
__global__ void __launch_bounds__(CTA_THREADS)
gather_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int64_t C, int64_t ldw,
              const int32_t* __restrict__ rp, const int32_t* __restrict__ cp,
              __nv_bfloat16* __restrict__ out, int rows_per_cta) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned short* row = reinterpret_cast<unsigned short*>(smem_raw);
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    for (int rr = 0; rr < rows_per_cta; ++rr) {
        const int64_t r = r0 + rr;
        if (r >= R) break;
        const int64_t rs = rp ? rp[r] : r;
        const __nv_bfloat16* src = W + rs * ldw;
        for (int64_t j = (int64_t)threadIdx.x * 8; j < C; j += CTA_THREADS * 8)
            *reinterpret_cast<uint4*>(row + j) = ld_stream16(src + j);
        __syncthreads();
        unsigned short* dst = reinterpret_cast<unsigned short*>(out + r * C);
        for (int64_t j = (int64_t)threadIdx.x * 8; j < C; j += CTA_THREADS * 8) {
            uint32_t o[4];
            if (cp) {
                const int4 p0 = *reinterpret_cast<const int4*>(cp + j);
                const int4 p1 = *reinterpret_cast<const int4*>(cp + j + 4);
                o[0] = row[p0.x] | ((uint32_t)row[p0.y] << 16);
                o[1] = row[p0.z] | ((uint32_t)row[p0.w] << 16);
                o[2] = row[p1.x] | ((uint32_t)row[p1.y] << 16);
                o[3] = row[p1.z] | ((uint32_t)row[p1.w] << 16);
            } else {
                const uint4 v = *reinterpret_cast<const uint4*>(row + j);
                o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
            }
            *reinterpret_cast<uint4*>(dst + j) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        __syncthreads();
    }
}

// ---- shared inner step: one lane, CPL consecutive columns of one row ----------------------
template <int CPL>
__device__ __forceinline__ void load_cols(const __nv_bfloat16* p, bool ok, uint32_t (&w)[CPL / 2]) {
#pragma unroll
    for (int v = 0; v < CPL / 8; ++v) {
        uint4 x = ok ? ld_stream16(p + 8 * v) : make_uint4(0, 0, 0, 0);
        w[4 * v] = x.x; w[4 * v + 1] = x.y; w[4 * v + 2] = x.z; w[4 * v + 3] = x.w;
    }
}

// ---- block scores ------------------------------------------------------------------------
// CTA = 8 warps.  A lane owns CPL consecutive columns of a 128-column chunk; 128/CPL lanes
// cover a row of the chunk and a warp covers 32*CPL/128 rows per step.  grid.x = column
// tiles (one block when block_cols >= 128, else 128/block_cols blocks side by side),
// grid.y = block rows.
template <int L, int CPL, bool ROWW>
__global__ void __launch_bounds__(CTA_THREADS)
block_scores_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw,
                    const int32_t* __restrict__ load_row_perm,   // rows gathered at load time
                    const int32_t* __restrict__ c_perm,          // original column of permuted j
                    const int32_t* __restrict__ a_perm,          // original row of permuted r
                    const float* __restrict__ col_moment, const float* __restrict__ row_weight,
                    int br, int bc, int group, BitsArg ba, int64_t n_block_cols,
                    float* __restrict__ err, float* __restrict__ gain, SbDeviceState* dstate) {
    constexpr int LANE_COLS = TILE_COLS / CPL;      // lanes across a chunk row
    constexpr int ROW_SLOTS = 32 / LANE_COLS;       // rows per warp step
    constexpr int NW = CPL / 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cl = lane % LANE_COLS, slot = lane / LANE_COLS;
    const int team = group / CPL > 0 ? group / CPL : 1;
    const int chunks = bc >= TILE_COLS ? bc / TILE_COLS : 1;
    const int tile_w = bc >= TILE_COLS ? bc : TILE_COLS;
    const int64_t row0 = (int64_t)blockIdx.y * br;
    const int64_t colT = (int64_t)blockIdx.x * tile_w;

    float tot[L];
#pragma unroll
    for (int l = 0; l < L; ++l) tot[l] = 0.f;

    for (int ch = 0; ch < chunks; ++ch) {
        const int64_t col = colT + (int64_t)ch * TILE_COLS + cl * CPL;
        float acc[CPL][L];
#pragma unroll
        for (int k = 0; k < CPL; ++k)
#pragma unroll
            for (int l = 0; l < L; ++l) acc[k][l] = 0.f;

        for (int rr = warp * ROW_SLOTS + slot; rr < br; rr += CTA_WARPS * ROW_SLOTS) {
            const int64_t r = row0 + rr;
            const int64_t rs = load_row_perm ? load_row_perm[r] : r;
            uint32_t w[NW];
            load_cols<CPL>(W + rs * ldw + col, true, w);
            float lo, hi;
            group_minmax<NW>(w, team, lo, hi);
            const float range = hi - lo;
            const bool live = range >= MIN_RANGE;
            const float rinv = live ? rcp_approx(range) : 0.f;
            float ar = 1.f;
            if (ROWW) ar = row_weight[a_perm ? a_perm[r] : r];
            float vm[CPL];
#pragma unroll
            for (int k = 0; k < NW; ++k) {
                vm[2 * k] = bf16lo(w[k]) - lo;
                vm[2 * k + 1] = bf16hi(w[k]) - lo;
            }
#pragma unroll
            for (int l = 0; l < L; ++l) {
                const float inv = ba.qmax[l] * rinv;
                const float nscale = live ? -(range * ba.inv_qmax[l]) : 0.f;
                // With many levels q * scale carries the fp32 rounding of the step times q,
                // a bias shared by the whole group: from 6 bits on the step is kept as a
                // two-float sum (the residual range - scale * qmax is exact in one FMA).
                const bool fine = ba.bits[l] >= 6;
                const float nscale_lo = fine ? -(fmaf(nscale, ba.qmax[l], range) * ba.inv_qmax[l]) : 0.f;
#pragma unroll
                for (int k = 0; k < CPL; ++k) {
                    const float q = fmaf(vm[k], inv, RNE_MAGIC) - RNE_MAGIC;
                    float e = fmaf(q, nscale, vm[k]);
                    if (fine) e = fmaf(q, nscale_lo, e);
                    if (ROWW) acc[k][l] = fmaf(e * ar, e, acc[k][l]);
                    else acc[k][l] = fmaf(e, e, acc[k][l]);
                }
            }
        }
        // column factors once per chunk
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const int64_t j = col + k;
            const float cw = col_moment[c_perm ? c_perm[j] : j];
#pragma unroll
            for (int l = 0; l < L; ++l) tot[l] = fmaf(cw, acc[k][l], tot[l]);
        }
    }

    // reduce: lanes of the same block (sub-block when bc < 128), then warps, fixed order
    const int lanes_per_sub = bc >= TILE_COLS ? LANE_COLS : bc / CPL;    // lanes across one block
    const int nsub = bc >= TILE_COLS ? 1 : TILE_COLS / bc;
#pragma unroll
    for (int l = 0; l < L; ++l) {
        float v = tot[l];
        for (int o = lanes_per_sub >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        for (int o = LANE_COLS; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        tot[l] = v;
    }
    __shared__ float red[CTA_WARPS][4][8];
    if (slot == 0 && (cl % lanes_per_sub) == 0) {
        const int sb = cl / lanes_per_sub;
#pragma unroll
        for (int l = 0; l < L; ++l) red[warp][sb][l] = tot[l];
    }
    __syncthreads();
    if (threadIdx.x < nsub) {
        const int sb = threadIdx.x;
        const int64_t blk = (int64_t)blockIdx.y * n_block_cols + (int64_t)blockIdx.x * nsub + sb;
        float e[L];
        bool finite = true;
#pragma unroll
        for (int l = 0; l < L; ++l) {
            float s = 0.f;
#pragma unroll
            for (int wv = 0; wv < CTA_WARPS; ++wv) s += red[wv][sb][l];
            e[l] = s;
            err[blk * L + l] = s;
            finite = finite && isfinite(s);
        }
        if (!finite) sb_latch(dstate, SB_ERR_NONFINITE, SBK_SCORES);
        if (gain) {
            const float M = (float)br * (float)bc;
#pragma unroll
            for (int l = 0; l + 1 < L; ++l)
                gain[blk * (L - 1) + l] = (e[l] - e[l + 1]) / ((float)(ba.bits[l + 1] - ba.bits[l]) * M);
        }
    }
}

// ---- reorder statistics --------------------------------------------------------------------
// 128 x 128 tiles of the ORIGINAL layout, one candidate (ref_bits).  Writes per-tile partial
// row sums rowpart[tile_col][r] and column sums colpart[tile_row][j]; a second kernel adds
// them up in a fixed order (no floating-point atomics: run-to-run deterministic).
template <bool ROWW>
__global__ void __launch_bounds__(CTA_THREADS)
reorder_stats_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int64_t C, int64_t ldw,
                     const float* __restrict__ col_moment, const float* __restrict__ row_weight,
                     int group, float qmax, float inv_qmax,
                     float* __restrict__ rowpart, float* __restrict__ colpart) {
    constexpr int CPL = 16, NW = 8, LANE_COLS = 8, ROW_SLOTS = 4, TILE_ROWS = 128;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cl = lane % LANE_COLS, slot = lane / LANE_COLS;
    const int team = group / CPL > 0 ? group / CPL : 1;
    const int64_t col = (int64_t)blockIdx.x * TILE_COLS + cl * CPL;
    const bool col_ok = col < C;
    const int64_t row0 = (int64_t)blockIdx.y * TILE_ROWS;
    float cw[CPL], acc[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
        cw[k] = col_ok ? col_moment[col + k] : 0.f;
        acc[k] = 0.f;
    }
    for (int rr = warp * ROW_SLOTS + slot; rr < TILE_ROWS; rr += CTA_WARPS * ROW_SLOTS) {
        const int64_t r = row0 + rr;
        const bool ok = col_ok && r < R;
        uint32_t w[NW];
        load_cols<CPL>(W + (ok ? r * ldw + col : 0), ok, w);
        float lo, hi;
        group_minmax<NW>(w, team, lo, hi);
        const float range = hi - lo;
        const bool live = range >= MIN_RANGE;
        const float inv = live ? qmax * rcp_approx(range) : 0.f;
        const float nscale = live ? -(range * inv_qmax) : 0.f;
        const float nscale_lo = -(fmaf(nscale, qmax, range) * inv_qmax);   // two-float step
        float ar = 1.f;
        if (ROWW) ar = (r < R) ? row_weight[r] : 0.f;
        float rs = 0.f;
#pragma unroll
        for (int k = 0; k < NW; ++k) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float vm = (h ? bf16hi(w[k]) : bf16lo(w[k])) - lo;
                const float q = fmaf(vm, inv, RNE_MAGIC) - RNE_MAGIC;
                const float e = fmaf(q, nscale_lo, fmaf(q, nscale, vm));
                const float e2 = ROWW ? e * e * ar : e * e;
                acc[2 * k + h] += e2;
                rs = fmaf(cw[2 * k + h], e2, rs);
            }
        }
#pragma unroll
        for (int o = LANE_COLS >> 1; o > 0; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
        if (rowpart && cl == 0 && r < R) rowpart[(int64_t)blockIdx.x * R + r] = rs;
    }
    if (!colpart) return;
    __shared__ float red[CTA_WARPS * ROW_SLOTS][TILE_COLS + 4];
#pragma unroll
    for (int k = 0; k < CPL; ++k) red[warp * ROW_SLOTS + slot][cl * CPL + k] = acc[k] * cw[k];
    __syncthreads();
    if (threadIdx.x < TILE_COLS) {
        const int64_t j = (int64_t)blockIdx.x * TILE_COLS + threadIdx.x;
        if (j < C) {
            float s = 0.f;
#pragma unroll
            for (int p = 0; p < CTA_WARPS * ROW_SLOTS; ++p) s += red[p][threadIdx.x];
            colpart[(int64_t)blockIdx.y * C + j] = s;
        }
    }
}

__global__ void sum_partials_kernel(const float* __restrict__ part, int nparts, int64_t n,
                                    int accumulate, float* __restrict__ out, SbDeviceState* dstate) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int p = 0; p < nparts; ++p) s += part[(int64_t)p * n + i];
    if (!isfinite(s)) sb_latch(dstate, SB_ERR_NONFINITE, SBK_STATS);
    out[i] = accumulate ? out[i] + s : s;
}

// ---- argsort by counting: rank_i = #{j in segment : s_j > s_i or (s_j == s_i and j < i)} ----
__device__ __forceinline__ uint32_t order_key(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__global__ void rank_count_kernel(const float* __restrict__ score, int64_t K, int64_t seg,
                                  int64_t span, int* __restrict__ rank) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const int64_t s0 = i / seg * seg;
    const int64_t j0 = s0 + (int64_t)blockIdx.y * span;
    const int64_t j1 = min(s0 + seg, j0 + span);
    const uint32_t ki = order_key(score[i]);
    int cnt = 0;
    for (int64_t j = j0; j < j1; ++j) {
        const uint32_t kj = order_key(__ldg(score + j));
        cnt += (kj > ki) || (kj == ki && j < i);
    }
    if (cnt) atomicAdd(rank + i, cnt);
}
__global__ void rank_scatter_kernel(const int* __restrict__ rank, int64_t K, int64_t seg,
                                    int32_t* __restrict__ perm) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    perm[i / seg * seg + rank[i]] = (int32_t)i;
}

__global__ void fold_scores_kernel(float* dst, const float* __restrict__ src, int64_t n_dst,
                                   int reps, int64_t seg) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_dst) return;
    const int64_t h = i / seg, d = i % seg;
    float s = dst[i];
    for (int u = 0; u < reps; ++u) s += src[(h * reps + u) * seg + d];
    dst[i] = s;
}
__global__ void expand_perm_kernel(int32_t* out, const int32_t* __restrict__ perm, int64_t n_src,
                                   int reps, int64_t seg) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_src) return;
    const int64_t h = i / seg, d = i % seg;
    const int64_t local = perm[i] - h * seg;
    for (int u = 0; u < reps; ++u) out[(h * reps + u) * seg + d] = (int32_t)((h * reps + u) * seg + local);
}

BitsArg make_bits(const int* bits, int n) {
    BitsArg ba{};
    for (int l = 0; l < 8; ++l) {
        const int b = l < n ? bits[l] : 1;
        ba.bits[l] = b;
        ba.qmax[l] = (float)((1 << b) - 1);
        ba.inv_qmax[l] = 1.0f / (float)((1 << b) - 1);
    }
    return ba;
}

bool valid_group(int g) { return g == 16 || g == 32 || g == 64 || g == 128; }

sb_status argsort_axis(sb_ctx* ctx, const float* score, int64_t K, int64_t seg, int32_t* perm, int* rank) {
    SB_CUDA(ctx, cudaMemsetAsync(rank, 0, sizeof(int) * K, ctx->stream));
    int splits = (int)((seg + 2047) / 2048);
    if (splits > 64) splits = 64;
    const int64_t span = (seg + splits - 1) / splits;
    dim3 grid((unsigned)((K + 255) / 256), splits);
    rank_count_kernel<<<grid, 256, 0, ctx->stream>>>(score, K, seg, span, rank);
    SB_LAUNCHED(ctx);
    rank_scatter_kernel<<<(unsigned)((K + 255) / 256), 256, 0, ctx->stream>>>(rank, K, seg, perm);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

template <int L, int CPL>
void launch_scores(sb_ctx* ctx, dim3 grid, bool roww, const __nv_bfloat16* W, int64_t ldw,
                   const int32_t* lrp, const int32_t* cperm, const int32_t* aperm, const float* cm,
                   const float* rw, int br, int bc, int group, const BitsArg& ba, int64_t nbc,
                   float* err, float* gain) {
    if (roww)
        block_scores_kernel<L, CPL, true><<<grid, CTA_THREADS, 0, ctx->stream>>>(
            W, ldw, lrp, cperm, aperm, cm, rw, br, bc, group, ba, nbc, err, gain, ctx->dstate);
    else
        block_scores_kernel<L, CPL, false><<<grid, CTA_THREADS, 0, ctx->stream>>>(
            W, ldw, lrp, cperm, aperm, cm, rw, br, bc, group, ba, nbc, err, gain, ctx->dstate);
}

}  // namespace

// used by pack.cu as well
sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out) {
    const size_t smem = (size_t)C * 2;
    if (smem > 200 * 1024) return sb_fail(ctx, SB_ERR_SHAPE, "gather: rows longer than 102400 columns");
    static bool attr_set = false;
    if (!attr_set) {
        SB_CUDA(ctx, cudaFuncSetAttribute(gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          200 * 1024));
        attr_set = true;
    }
    int rows_per_cta = 4;
    const unsigned grid = (unsigned)((R + rows_per_cta - 1) / rows_per_cta);
    gather_kernel<<<grid, CTA_THREADS, smem, ctx->stream>>>(
        static_cast<const __nv_bfloat16*>(W), R, C, ldw, rp, cp, static_cast<__nv_bfloat16*>(out),
        rows_per_cta);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

extern "C" {

sb_status sb_reorder_channels(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                              const float* col_moment, const float* row_weight, int ref_bits,
                              int group, float* row_score, float* col_score, int accumulate,
                              int64_t row_segment, int64_t col_segment, int32_t* row_perm,
                              int32_t* col_perm) {
    if (!ctx) return SB_ERR_INVALID;
    if (R <= 0 || C <= 0) return sb_fail(ctx, SB_ERR_INVALID, "reorder: empty matrix");
    const bool sort_rows = row_segment > 0 && row_perm, sort_cols = col_segment > 0 && col_perm;
    if (sort_rows && (!row_score || R % row_segment)) return sb_fail(ctx, SB_ERR_SHAPE, "reorder: row segment");
    if (sort_cols && (!col_score || C % col_segment)) return sb_fail(ctx, SB_ERR_SHAPE, "reorder: column segment");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    if (W) {
        if (!col_moment) return sb_fail(ctx, SB_ERR_INVALID, "reorder: col_moment is NULL");
        if (ref_bits < 1 || ref_bits > 8) return sb_fail(ctx, SB_ERR_INVALID, "reorder: ref_bits");
        if (!valid_group(group) || C % group || C % 16 || ldw % 8 || ldw < C ||
            (reinterpret_cast<uintptr_t>(W) & 15))
            return sb_fail(ctx, SB_ERR_SHAPE, "reorder: group in {16,32,64,128} must divide C; ldw %% 8; 16-byte base");
    }
    const int tiles_r = (int)((R + 127) / 128), tiles_c = (int)((C + 127) / 128);
    const int64_t maxK = R > C ? R : C;
    void* arena;
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)tiles_c * R * 4, (size_t)tiles_r * C * 4,
                                                 (size_t)maxK * 4}), &arena);
    if (st != SB_OK) return st;
    Carver cv(arena);
    float* rowpart = cv.take<float>((size_t)tiles_c * R);
    float* colpart = cv.take<float>((size_t)tiles_r * C);
    int* rank = cv.take<int>((size_t)maxK);
    if (W && (row_score || col_score)) {
        const float qmax = (float)((1 << ref_bits) - 1);
        dim3 grid(tiles_c, tiles_r);
        auto* Wb = static_cast<const __nv_bfloat16*>(W);
        if (row_weight)
            reorder_stats_kernel<true><<<grid, CTA_THREADS, 0, ctx->stream>>>(
                Wb, R, C, ldw, col_moment, row_weight, group, qmax, 1.0f / qmax,
                row_score ? rowpart : nullptr, col_score ? colpart : nullptr);
        else
            reorder_stats_kernel<false><<<grid, CTA_THREADS, 0, ctx->stream>>>(
                Wb, R, C, ldw, col_moment, row_weight, group, qmax, 1.0f / qmax,
                row_score ? rowpart : nullptr, col_score ? colpart : nullptr);
        SB_LAUNCHED(ctx);
        if (row_score) {
            sum_partials_kernel<<<(unsigned)((R + 255) / 256), 256, 0, ctx->stream>>>(
                rowpart, tiles_c, R, accumulate & SB_ACC_ROW, row_score, ctx->dstate);
            SB_LAUNCHED(ctx);
        }
        if (col_score) {
            sum_partials_kernel<<<(unsigned)((C + 255) / 256), 256, 0, ctx->stream>>>(
                colpart, tiles_r, C, accumulate & SB_ACC_COL, col_score, ctx->dstate);
            SB_LAUNCHED(ctx);
        }
    }
    if (sort_rows) { st = argsort_axis(ctx, row_score, R, row_segment, row_perm, rank); if (st) return st; }
    if (sort_cols) { st = argsort_axis(ctx, col_score, C, col_segment, col_perm, rank); if (st) return st; }
    return SB_OK;
}

sb_status sb_fold_segment_scores(sb_ctx* ctx, float* dst, const float* src, int64_t n_dst, int reps,
                                 int64_t seg) {
    if (!ctx) return SB_ERR_INVALID;
    if (!dst || !src || n_dst <= 0 || reps < 1 || seg < 1 || n_dst % seg)
        return sb_fail(ctx, SB_ERR_INVALID, "fold: bad arguments");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    fold_scores_kernel<<<(unsigned)((n_dst + 255) / 256), 256, 0, ctx->stream>>>(dst, src, n_dst, reps, seg);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

sb_status sb_expand_segment_perm(sb_ctx* ctx, int32_t* out, const int32_t* perm, int64_t n_src,
                                 int reps, int64_t seg) {
    if (!ctx) return SB_ERR_INVALID;
    if (!out || !perm || n_src <= 0 || reps < 1 || seg < 1 || n_src % seg)
        return sb_fail(ctx, SB_ERR_INVALID, "expand: bad arguments");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    expand_perm_kernel<<<(unsigned)((n_src + 255) / 256), 256, 0, ctx->stream>>>(out, perm, n_src, reps, seg);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

sb_status sb_block_scores(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                          const int32_t* row_perm, const int32_t* col_perm, const float* col_moment,
                          const float* row_weight, int br, int bc, int group, const int* bits,
                          int n_bits, float* err, float* gain, void* W_perm_out) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !col_moment || !err || R <= 0 || C <= 0) return sb_fail(ctx, SB_ERR_INVALID, "scores: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "scores: bits must be ascending in 1..8");
    if (br <= 0 || bc <= 0 || br % 4 || R % br || C % bc || !valid_group(group) || bc % group ||
        !(bc == 32 || bc == 64 || bc % 128 == 0) || ldw % 8 || ldw < C ||
        (reinterpret_cast<uintptr_t>(W) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "scores: block %dx%d group %d does not tile %lldx%lld", br, bc,
                       group, (long long)R, (long long)C);
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(W);
    int64_t ld = ldw;
    const int32_t* load_rp = row_perm;
    if (col_perm || W_perm_out) {
        void* dst = W_perm_out;
        if (!dst) {
            sb_status st = sb_scratch(ctx, (size_t)R * C * 2 + 256, &dst);
            if (st != SB_OK) return st;
        }
        sb_status st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, dst);
        if (st != SB_OK) return st;
        src = static_cast<const __nv_bfloat16*>(dst);
        ld = C;
        load_rp = nullptr;
    }
    const BitsArg ba = make_bits(bits, n_bits);
    const int tile_w = bc >= 128 ? bc : 128;
    if (C % tile_w) return sb_fail(ctx, SB_ERR_SHAPE, "scores: C must be a multiple of 128");
    dim3 grid((unsigned)(C / tile_w), (unsigned)(R / br));
    const int64_t nbc = C / bc;
    const bool roww = row_weight != nullptr;
#define SB_SCORES(Lv, CPLv)                                                                       \
    launch_scores<Lv, CPLv>(ctx, grid, roww, src, ld, load_rp, col_perm, row_perm, col_moment,     \
                            row_weight, br, bc, group, ba, nbc, err, gain)
    switch (n_bits) {
        case 1: SB_SCORES(1, 16); break;
        case 2: SB_SCORES(2, 16); break;
        case 3: SB_SCORES(3, 16); break;
        case 4: SB_SCORES(4, 16); break;
        case 5: SB_SCORES(5, 8); break;
        case 6: SB_SCORES(6, 8); break;
        case 7: SB_SCORES(7, 8); break;
        default: SB_SCORES(8, 8); break;
    }
#undef SB_SCORES
    SB_LAUNCHED(ctx);
    return SB_OK;
}

}  // extern "C"

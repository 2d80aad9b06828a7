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
#include "quant_common.cuh"

namespace {

constexpr int CTA_THREADS = 256;
constexpr int CTA_WARPS = CTA_THREADS / 32;

// ---- permuted gather: out[r][j] = W[rp[r]][cp[j]] ---------------------------------------
// A source row is staged in shared memory with coalesced asynchronous 16-byte copies (a ring of
// three rows: two are in flight while one is written out, one barrier per row), then read in
// permuted order: 2-byte scattered reads never reach HBM.
constexpr int GA_STAGES = 3;
__global__ void __launch_bounds__(CTA_THREADS)
gather_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int C, int64_t ldw,
              const int32_t* __restrict__ rp, const int32_t* __restrict__ cp,
              __nv_bfloat16* __restrict__ out, int rows_per_cta, SbDeviceState* ds) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const unsigned row_bytes = (unsigned)C * 2u;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int nrows = (int)min((int64_t)rows_per_cta, R - r0);
    const int j0 = (int)threadIdx.x * 8;
    auto stage = [&](int rr, int st) {
        if (rr < nrows) {
            const int64_t r = r0 + rr;
            int64_t rs = rp ? (int64_t)rp[r] : r;
            if (!SB_IN_BOUNDS(ds, SBK_GATHER, rs, R)) rs = 0;          // a bad permutation entry reads row 0
            const __nv_bfloat16* src = W + rs * ldw;
            unsigned char* dst = smem_raw + (unsigned)st * row_bytes;
            for (int j = j0; j < C; j += CTA_THREADS * 8) cp_async16(dst + 2 * j, src + j);
        }
        cp_async_commit();                      // one group per row, empty past the end
    };
    stage(0, 0);
    stage(1, 1);
    int st = 0;
    for (int rr = 0; rr < nrows; ++rr, st = st + 1 == GA_STAGES ? 0 : st + 1) {
        cp_async_wait<1>();                     // row rr has landed (row rr + 1 may be in flight)
        __syncthreads();                        // ... for every thread; row rr - 1 is consumed
        stage(rr + 2, st >= 1 ? st - 1 : GA_STAGES - 1);
        const unsigned short* row = reinterpret_cast<const unsigned short*>(smem_raw + (unsigned)st * row_bytes);
        unsigned short* dst = reinterpret_cast<unsigned short*>(out + (r0 + rr) * (int64_t)C);
        for (int j = j0; j < C; j += CTA_THREADS * 8) {
            uint4 o;
            if (cp) {
                int4 p0 = __ldg(reinterpret_cast<const int4*>(cp + j));
                int4 p1 = __ldg(reinterpret_cast<const int4*>(cp + j + 4));
#ifdef SB_CHECKED
                {
                    int* pv[8] = {&p0.x, &p0.y, &p0.z, &p0.w, &p1.x, &p1.y, &p1.z, &p1.w};
                    for (int k = 0; k < 8; ++k) if (!SB_IN_BOUNDS(ds, SBK_GATHER, *pv[k], C)) *pv[k] = 0;
                }
#endif
                o.x = row[p0.x] | ((uint32_t)row[p0.y] << 16);
                o.y = row[p0.z] | ((uint32_t)row[p0.w] << 16);
                o.z = row[p1.x] | ((uint32_t)row[p1.y] << 16);
                o.w = row[p1.z] | ((uint32_t)row[p1.w] << 16);
            } else {
                o = *reinterpret_cast<const uint4*>(row + j);
            }
            *reinterpret_cast<uint4*>(dst + j) = o;
        }
    }
    cp_async_wait<0>();
}

// The same with the column permutation held in registers: a thread writes the same output
// columns in every row, so it reads its source columns once (as byte offsets, two per
// register) instead of once per row.  NIT * 2048 >= C, C < 32768.
template <int NIT>
__global__ void __launch_bounds__(CTA_THREADS)
gather_cols_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int C, int64_t ldw,
                   const int32_t* __restrict__ rp, const int32_t* __restrict__ cp,
                   __nv_bfloat16* __restrict__ out, int rows_per_cta, SbDeviceState* ds) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const unsigned row_bytes = (unsigned)C * 2u;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int nrows = (int)min((int64_t)rows_per_cta, R - r0);
    const int j0 = (int)threadIdx.x * 8;
    uint32_t off2[NIT][4];
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int j = j0 + it * (CTA_THREADS * 8);
        int4 p0 = make_int4(0, 0, 0, 0), p1 = p0;
        if (j < C) {
            p0 = __ldg(reinterpret_cast<const int4*>(cp + j));
            p1 = __ldg(reinterpret_cast<const int4*>(cp + j + 4));
#ifdef SB_CHECKED
            int* pv[8] = {&p0.x, &p0.y, &p0.z, &p0.w, &p1.x, &p1.y, &p1.z, &p1.w};
            for (int k = 0; k < 8; ++k) if (!SB_IN_BOUNDS(ds, SBK_GATHER, *pv[k], C)) *pv[k] = 0;
#endif
        }
        off2[it][0] = (uint32_t)(2 * p0.x) | ((uint32_t)(2 * p0.y) << 16);
        off2[it][1] = (uint32_t)(2 * p0.z) | ((uint32_t)(2 * p0.w) << 16);
        off2[it][2] = (uint32_t)(2 * p1.x) | ((uint32_t)(2 * p1.y) << 16);
        off2[it][3] = (uint32_t)(2 * p1.z) | ((uint32_t)(2 * p1.w) << 16);
    }
    auto stage = [&](int rr, int st) {
        if (rr < nrows) {
            const int64_t r = r0 + rr;
            int64_t rs = rp ? (int64_t)rp[r] : r;
            if (!SB_IN_BOUNDS(ds, SBK_GATHER, rs, R)) rs = 0;          // a bad permutation entry reads row 0
            const __nv_bfloat16* src = W + rs * ldw;
            unsigned char* dst = smem_raw + (unsigned)st * row_bytes;
            for (int j = j0; j < C; j += CTA_THREADS * 8) cp_async16(dst + 2 * j, src + j);
        }
        cp_async_commit();
    };
    stage(0, 0);
    stage(1, 1);
    int st = 0;
    for (int rr = 0; rr < nrows; ++rr, st = st + 1 == GA_STAGES ? 0 : st + 1) {
        cp_async_wait<1>();
        __syncthreads();
        stage(rr + 2, st >= 1 ? st - 1 : GA_STAGES - 1);
        const unsigned char* row = smem_raw + (unsigned)st * row_bytes;
        unsigned short* dst = reinterpret_cast<unsigned short*>(out + (r0 + rr) * (int64_t)C);
        auto pair = [&](uint32_t o2) -> uint32_t {
            const uint32_t a = *reinterpret_cast<const unsigned short*>(row + (o2 & 0xffffu));
            const uint32_t b = *reinterpret_cast<const unsigned short*>(row + (o2 >> 16));
            return a | (b << 16);
        };
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            const int j = j0 + it * (CTA_THREADS * 8);
            if (j < C) {
                uint4 o;
                o.x = pair(off2[it][0]); o.y = pair(off2[it][1]);
                o.z = pair(off2[it][2]); o.w = pair(off2[it][3]);
                *reinterpret_cast<uint4*>(dst + j) = o;
            }
        }
    }
    cp_async_wait<0>();
}
// ---- shared inner step: one lane, CPL consecutive columns of one row ----------------------
template <int CPL>
__device__ __forceinline__ void load_cols(const __nv_bfloat16* p, bool ok, uint32_t (&w)[CPL / 2]) {
#pragma unroll
    for (int v = 0; v < CPL / 8; ++v) {
        // plain read-only loads: a lane's two 16-byte pieces share 32-byte sectors with its
        // neighbours', so the second load of a row should hit L1
        uint4 x = ok ? __ldg(reinterpret_cast<const uint4*>(p + 8 * v)) : make_uint4(0, 0, 0, 0);
        w[4 * v] = x.x; w[4 * v + 1] = x.y; w[4 * v + 2] = x.z; w[4 * v + 3] = x.w;
    }
}

// ---- reorder statistics, first-order form --------------------------------------------------
// (The second-moment form runs on the score kernel's slab walk: scores.cu.)
// Element sensitivity |G_rj (W_rj - Q(W)_rj)| (Section 3.2 with p = 1) from a caller's gradient G,
// summed per channel (l1 aggregation, Section 4.1).  128 x 128 tiles of the ORIGINAL layout, one
// candidate (ref_bits).  Every tile writes its partial row sums rowpart[tile_col][r] and column
// sums colpart[tile_row][j]; the last tile of a tile row (tile column) to finish adds the partials
// of that row strip (column strip) in tile order -- a fixed order whichever CTA does it, and no
// floating-point atomics, so reruns are bit-identical -- and adds them to / stores them in the
// score vectors.  A tile is `tile_rows` (a multiple of 32) x 128; the host picks tile_rows so that
// the tiles fill whole rounds of the CTA slots of the GPU.
template <bool FINE>
__global__ void __launch_bounds__(CTA_THREADS)
reorder_stats_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int64_t C, int64_t ldw, int tile_rows,
                     const __nv_bfloat16* __restrict__ G, int64_t ldg,
                     int group, float qmax, float inv_qmax,
                     float* __restrict__ rowpart, float* __restrict__ colpart,
                     float* __restrict__ row_score, float* __restrict__ col_score, int accumulate,
                     unsigned* __restrict__ done_row, unsigned* __restrict__ done_col,
                     SbDeviceState* dstate) {
    constexpr int CPL = 16, NW = 8, LANE_COLS = 8, ROW_SLOTS = 4;
    const int ITERS = tile_rows / (CTA_WARPS * ROW_SLOTS);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cl = lane % LANE_COLS, slot = lane / LANE_COLS;
    const int team = group / CPL > 0 ? group / CPL : 1;
    const int64_t col = (int64_t)blockIdx.x * TILE_COLS + cl * CPL;
    const bool col_ok = col < C;
    const int64_t row0 = (int64_t)blockIdx.y * tile_rows;
    const f32x2 magic2 = pk2(RNE_MAGIC, RNE_MAGIC), nmagic2 = pk2(-RNE_MAGIC, -RNE_MAGIC);
    f32x2 acc[NW];
#pragma unroll
    for (int k = 0; k < NW; ++k) acc[k] = 0ull;
    // the next step's 16-byte loads are in flight while this step is evaluated
    uint32_t wn[NW], gn[NW];
    {
        const int64_t r = row0 + warp * ROW_SLOTS + slot;
        const bool ok = col_ok && r < R;
        load_cols<CPL>(W + (ok ? r * ldw + col : 0), ok, wn);
        load_cols<CPL>(G + (ok ? r * ldg + col : 0), ok, gn);
    }
#pragma unroll 2
    for (int it = 0; it < ITERS; ++it) {
        const int rr = it * (CTA_WARPS * ROW_SLOTS) + warp * ROW_SLOTS + slot;
        const int64_t r = row0 + rr;
        uint32_t w[NW], gw[NW];
#pragma unroll
        for (int k = 0; k < NW; ++k) { w[k] = wn[k]; gw[k] = gn[k]; }
        if (it + 1 < ITERS) {
            const int64_t rn = r + CTA_WARPS * ROW_SLOTS;
            const bool okn = col_ok && rn < R;
            load_cols<CPL>(W + (okn ? rn * ldw + col : 0), okn, wn);
            load_cols<CPL>(G + (okn ? rn * ldg + col : 0), okn, gn);
        }
        float lo, hi;
        group_minmax<NW>(w, team, lo, hi);
        const float range = hi - lo;
        const bool live = range >= MIN_RANGE;
        const float inv = live ? qmax * rcp_approx(range) : 0.f;
        const float nscale = live ? -(range * inv_qmax) : 0.f;
        const f32x2 inv2 = pk2(inv, inv), ns2 = pk2(nscale, nscale), nlo2 = pk2(-lo, -lo);
        f32x2 nslo2 = 0ull;
        if (FINE) {                                     // two-float step from 6 bits on
            const float nscale_lo = -(fmaf(nscale, qmax, range) * inv_qmax);
            nslo2 = pk2(nscale_lo, nscale_lo);
        }
        f32x2 rs2 = 0ull;
#pragma unroll
        for (int k = 0; k < NW; ++k) {
            const f32x2 vm = add2(pk2(bf16lo(w[k]), bf16hi(w[k])), nlo2);
            const f32x2 qq = add2(fma2(vm, inv2, magic2), nmagic2);
            f32x2 e = fma2(qq, ns2, vm);
            if (FINE) e = fma2(qq, nslo2, e);
            const f32x2 ge = mul2(pk2(bf16lo(gw[k]), bf16hi(gw[k])), e);
            const f32x2 e2 = ge & 0x7fffffff7fffffffull;        // |g e| on both halves
            acc[k] = add2(acc[k], e2);
            rs2 = add2(rs2, e2);
        }
        float r0f, r1f;
        upk2(rs2, r0f, r1f);
        float rs = r0f + r1f;
#pragma unroll
        for (int o = LANE_COLS >> 1; o > 0; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
        if (rowpart && cl == 0 && r < R) rowpart[(int64_t)blockIdx.x * R + r] = rs;
    }
    __shared__ float red[CTA_WARPS * ROW_SLOTS][TILE_COLS + 4];
    if (colpart) {
#pragma unroll
        for (int k = 0; k < NW; ++k) {
            float a0, a1;
            upk2(acc[k], a0, a1);
            red[warp * ROW_SLOTS + slot][cl * CPL + 2 * k] = a0;
            red[warp * ROW_SLOTS + slot][cl * CPL + 2 * k + 1] = a1;
        }
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
    // last tile of this tile row / tile column: add the strip's partials in tile order
    __shared__ bool last_row, last_col;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        last_row = rowpart && atomicAdd(done_row + blockIdx.y, 1u) == gridDim.x - 1;
        last_col = colpart && atomicAdd(done_col + blockIdx.x, 1u) == gridDim.y - 1;
    }
    __syncthreads();
    if (!last_row && !last_col) return;
    __threadfence();
    if (last_row) {
        for (int rr = threadIdx.x; rr < tile_rows; rr += CTA_THREADS) {
            const int64_t r = row0 + rr;
            if (r < R) {
                float s = 0.f;
                for (unsigned t = 0; t < gridDim.x; ++t) s += __ldcg(rowpart + (int64_t)t * R + r);
                if (!isfinite(s)) sb_latch(dstate, SB_ERR_NONFINITE, SBK_STATS);
                row_score[r] = (accumulate & SB_ACC_ROW) ? row_score[r] + s : s;
            }
        }
        if (threadIdx.x == 0) done_row[blockIdx.y] = 0u;
    }
    if (last_col && threadIdx.x >= CTA_THREADS - TILE_COLS) {
        const int t0 = threadIdx.x - (CTA_THREADS - TILE_COLS);
        const int64_t j = (int64_t)blockIdx.x * TILE_COLS + t0;
        if (j < C) {
            float s = 0.f;
            for (unsigned t = 0; t < gridDim.y; ++t) s += __ldcg(colpart + (int64_t)t * C + j);
            if (!isfinite(s)) sb_latch(dstate, SB_ERR_NONFINITE, SBK_STATS);
            col_score[j] = (accumulate & SB_ACC_COL) ? col_score[j] + s : s;
        }
        if (t0 == 0) done_col[blockIdx.x] = 0u;
    }
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
#pragma unroll 8
    for (int64_t j = j0; j < j1; ++j) {
        const uint32_t kj = order_key(__ldg(score + j));     // same j across the warp: broadcast
        cnt += (kj > ki) || (kj == ki && j < i);
    }
    if (cnt) atomicAdd(rank + i, cnt);
}
// the same count with the compared keys staged in shared memory: a CTA's 256 channels lie in one
// segment (segment % 256 == 0), blockIdx.y picks a run of 256 compared channels of that segment
__global__ void __launch_bounds__(256)
rank_count_tile_kernel(const float* __restrict__ score, int64_t K, int64_t seg, int* __restrict__ rank) {
    __shared__ uint32_t sk[256];
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t s0 = (int64_t)blockIdx.x * 256 / seg * seg;
    const int64_t j0 = s0 + (int64_t)blockIdx.y * 256;
    sk[threadIdx.x] = order_key(score[j0 + threadIdx.x]);
    __syncthreads();
    const uint32_t ki = order_key(score[i]);
    // j < i decides ties: all-or-nothing for a tile except the one that contains i
    const int64_t d = i - j0;                      // compared channels with index below i: j - j0 < d
    int cnt = 0;
    if (d <= 0) {
#pragma unroll 16
        for (int j = 0; j < 256; ++j) cnt += sk[j] > ki;
    } else if (d >= 256) {
#pragma unroll 16
        for (int j = 0; j < 256; ++j) cnt += sk[j] >= ki;
    } else {
#pragma unroll 16
        for (int j = 0; j < 256; ++j) cnt += (sk[j] > ki) || (sk[j] == ki && j < (int)d);
    }
    if (cnt) atomicAdd(rank + i, cnt);
}
__global__ void rank_scatter_kernel(const int* __restrict__ rank, int64_t K, int64_t seg,
                                    int32_t* __restrict__ perm) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    perm[i / seg * seg + rank[i]] = (int32_t)i;
}

// dst[i] = (dst[i] +) src[0][i] + src[1][i] + ... in that order: the score vectors of the matrices
// of a coupled channel set, each written by a call of its own (possibly on a stream of its own),
// added in the order the one-stream accumulation would have taken.
constexpr int SB_SUM_MAX_SRC = 8;
struct SumSources { const float* p[SB_SUM_MAX_SRC]; };
__global__ void sum_scores_kernel(float* __restrict__ dst, SumSources ss, int n_src, int64_t n, int accumulate) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float v[SB_SUM_MAX_SRC];
#pragma unroll
    for (int k = 0; k < SB_SUM_MAX_SRC; ++k) v[k] = k < n_src ? __ldg(ss.p[k] + i) : 0.f;
    float s = accumulate ? __fadd_rn(dst[i], v[0]) : v[0];
#pragma unroll
    for (int k = 1; k < SB_SUM_MAX_SRC; ++k) if (k < n_src) s = __fadd_rn(s, v[k]);
    dst[i] = s;
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

sb_status argsort_axis(sb_ctx* ctx, const float* score, int64_t K, int64_t seg, int32_t* perm, int* rank) {
    SB_CUDA(ctx, cudaMemsetAsync(rank, 0, sizeof(int) * K, ctx->stream));
    if (seg % 256 == 0) {
        dim3 grid((unsigned)(K / 256), (unsigned)(seg / 256));
        rank_count_tile_kernel<<<grid, 256, 0, ctx->stream>>>(score, K, seg, rank);
        SB_LAUNCHED(ctx);
        rank_scatter_kernel<<<(unsigned)((K + 255) / 256), 256, 0, ctx->stream>>>(rank, K, seg, perm);
        SB_LAUNCHED(ctx);
        return SB_OK;
    }
    // short comparison loops (<= 256 per thread): the counting is latency-bound otherwise
    int splits = (int)((seg + 255) / 256);
    if (splits > 1024) splits = 1024;
    const int64_t span = (seg + splits - 1) / splits;
    dim3 grid((unsigned)((K + 255) / 256), splits);
    rank_count_kernel<<<grid, 256, 0, ctx->stream>>>(score, K, seg, span, rank);
    SB_LAUNCHED(ctx);
    rank_scatter_kernel<<<(unsigned)((K + 255) / 256), 256, 0, ctx->stream>>>(rank, K, seg, perm);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

}  // namespace

// used by pack.cu as well
sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out) {
    const size_t smem = (size_t)C * 2 * GA_STAGES;  // a ring of row buffers
    if (smem > 200 * 1024) return sb_fail(ctx, SB_ERR_SHAPE, "gather: rows longer than 34133 columns");
    SB_FUNC_ATTR(ctx, gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    int rows_per_cta = 8;
    const unsigned grid = (unsigned)((R + rows_per_cta - 1) / rows_per_cta);
    auto* Wb = static_cast<const __nv_bfloat16*>(W);
    auto* ob = static_cast<__nv_bfloat16*>(out);
#define SB_GATHER_COLS(NIT)                                                                          \
    do {                                                                                             \
        SB_FUNC_ATTR(ctx, gather_cols_kernel<NIT>, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                     200 * 1024);                                                                    \
        gather_cols_kernel<NIT><<<grid, CTA_THREADS, smem, ctx->stream>>>(Wb, R, (int)C, ldw, rp, cp, ob, \
                                                                          rows_per_cta, ctx->dstate); \
    } while (0)
    if (cp && C <= 4096) SB_GATHER_COLS(2);
    else if (cp && C <= 8192) SB_GATHER_COLS(4);
    else if (cp && C <= 16384) SB_GATHER_COLS(8);
    else gather_kernel<<<grid, CTA_THREADS, smem, ctx->stream>>>(Wb, R, (int)C, ldw, rp, cp, ob, rows_per_cta, ctx->dstate);
#undef SB_GATHER_COLS
    SB_LAUNCHED(ctx);
    return SB_OK;
}

// the second-moment form runs on the slab walk of the score kernel (scores.cu)
size_t sb_stats_col_rec_floats(int64_t C, int sm_count);
size_t sb_stats_rowpart_floats(int64_t R, int64_t C);
sb_status sb_reorder_stats_slab(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                const float* col_moment, const float* row_weight, int ref_bits, int group,
                                float* row_score, float* col_score, int accumulate, float* col_rec, float* rowpart);

// both forms of the reorder statistics (G == NULL: second-moment form) and the sorts
static sb_status reorder_impl(sb_ctx* ctx, const void* W, const void* G, int64_t R, int64_t C, int64_t ldw,
                              int64_t ldg, const float* col_moment, const float* row_weight, int ref_bits,
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
        if (!G && !col_moment) return sb_fail(ctx, SB_ERR_INVALID, "reorder: col_moment is NULL");
        if (G && (ldg % 8 || ldg < C || (reinterpret_cast<uintptr_t>(G) & 15)))
            return sb_fail(ctx, SB_ERR_SHAPE, "reorder: gradient needs ldg %% 8 == 0, ldg >= C, 16-byte base");
        if (ref_bits < 1 || ref_bits > 8) return sb_fail(ctx, SB_ERR_INVALID, "reorder: ref_bits");
        if (!valid_group(group) || C % group || C % 16 || ldw % 8 || ldw < C ||
            (reinterpret_cast<uintptr_t>(W) & 15))
            return sb_fail(ctx, SB_ERR_SHAPE, "reorder: group in {16,32,64,128} must divide C; ldw %% 8; 16-byte base");
    }
    const int tiles_c = (int)((C + 127) / 128);
    // Tile height: the CTAs run in rounds of `slots` (three or four fit an SM), so the time is about
    // rounds x (tile_rows + a prologue / epilogue worth some 64 rows); take the height (a multiple of
    // 32 rows) that minimises it.  A height that leaves a few tiles for an extra round costs a
    // whole round: 512 rows on 14336 x 4096 made 896 tiles for 444 slots, three rounds instead of two.
    // the instance that will run, for its occupancy
    const bool fine = ref_bits >= 6;
    const void* kern = fine ? (const void*)reorder_stats_kernel<true> : (const void*)reorder_stats_kernel<false>;
    int occ = 0;
    SB_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, CTA_THREADS, 0));
    if (occ < 1) occ = 1;
    const long long slots = (long long)occ * ctx->sm_count;
    int tile_rows = 128;
    {
        long long best = -1;
        for (int h = 32; h <= 2048; h += 32) {
            const long long n = (long long)((R + h - 1) / h) * tiles_c;
            const long long rounds = (n + slots - 1) / slots;
            const long long cost = rounds * (h + 64);
            if (best < 0 || cost < best) { best = cost; tile_rows = h; }
        }
    }
    const int tiles_r = (int)((R + tile_rows - 1) / tile_rows);
    const int64_t maxK = R > C ? R : C;
    void* arena;
    const size_t slab_rec = sb_stats_col_rec_floats(C, ctx->sm_count), slab_rows = sb_stats_rowpart_floats(R, C);
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)tiles_c * R * 4, (size_t)tiles_r * C * 4,
                                                 (size_t)maxK * 4, slab_rec * 4, slab_rows * 4}), &arena);
    if (st != SB_OK) return st;
    Carver cv(arena);
    float* rowpart = cv.take<float>((size_t)tiles_c * R);
    float* colpart = cv.take<float>((size_t)tiles_r * C);
    int* rank = cv.take<int>((size_t)maxK);
    float* slab_col_rec = cv.take<float>(slab_rec);
    float* slab_rowpart = cv.take<float>(slab_rows);
    if (W && !G && (row_score || col_score)) {
        st = sb_reorder_stats_slab(ctx, W, R, C, ldw, col_moment, row_weight, ref_bits, group, row_score, col_score,
                                   accumulate, slab_col_rec, slab_rowpart);
        if (st != SB_OK) return st;
    } else if (W && (row_score || col_score)) {
        const float qmax = (float)((1 << ref_bits) - 1);
        if (tiles_r > SB_STATS_TILES || tiles_c > SB_STATS_TILES)
            return sb_fail(ctx, SB_ERR_SHAPE, "reorder: more than %d tiles on an axis", SB_STATS_TILES);
        dim3 grid(tiles_c, tiles_r);
        auto* Wb = static_cast<const __nv_bfloat16*>(W);
        float* rpart = row_score ? rowpart : nullptr;
        float* cpart = col_score ? colpart : nullptr;
        unsigned* done_row = ctx->stats_done;
        unsigned* done_col = ctx->stats_done + SB_STATS_TILES;
        auto* Gb = static_cast<const __nv_bfloat16*>(G);
        if (fine)
            reorder_stats_kernel<true><<<grid, CTA_THREADS, 0, ctx->stream>>>(
                Wb, R, C, ldw, tile_rows, Gb, ldg, group, qmax, 1.0f / qmax, rpart, cpart, row_score, col_score,
                accumulate, done_row, done_col, ctx->dstate);
        else
            reorder_stats_kernel<false><<<grid, CTA_THREADS, 0, ctx->stream>>>(
                Wb, R, C, ldw, tile_rows, Gb, ldg, group, qmax, 1.0f / qmax, rpart, cpart, row_score, col_score,
                accumulate, done_row, done_col, ctx->dstate);
        SB_LAUNCHED(ctx);
    }
    if (sort_rows) { st = argsort_axis(ctx, row_score, R, row_segment, row_perm, rank); if (st) return st; }
    if (sort_cols) { st = argsort_axis(ctx, col_score, C, col_segment, col_perm, rank); if (st) return st; }
    return SB_OK;
}

extern "C" {

sb_status sb_reorder_channels(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                              const float* col_moment, const float* row_weight, int ref_bits,
                              int group, float* row_score, float* col_score, int accumulate,
                              int64_t row_segment, int64_t col_segment, int32_t* row_perm,
                              int32_t* col_perm) {
    return reorder_impl(ctx, W, nullptr, R, C, ldw, 0, col_moment, row_weight, ref_bits, group, row_score,
                        col_score, accumulate, row_segment, col_segment, row_perm, col_perm);
}

sb_status sb_reorder_channels_first_order(sb_ctx* ctx, const void* W, const void* G, int64_t R, int64_t C,
                                          int64_t ldw, int64_t ldg, int ref_bits, int group,
                                          float* row_score, float* col_score, int accumulate,
                                          int64_t row_segment, int64_t col_segment, int32_t* row_perm,
                                          int32_t* col_perm) {
    if (ctx && W && !G) return sb_fail(ctx, SB_ERR_INVALID, "reorder (first order): G is NULL");
    return reorder_impl(ctx, W, G, R, C, ldw, ldg, nullptr, nullptr, ref_bits, group, row_score, col_score,
                        accumulate, row_segment, col_segment, row_perm, col_perm);
}

sb_status sb_permute_matrix(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                            const int32_t* row_perm, const int32_t* col_perm, void* out) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !out || R <= 0 || C <= 0) return sb_fail(ctx, SB_ERR_INVALID, "permute: null or empty");
    if (C % 8 || ldw % 8 || ldw < C || (reinterpret_cast<uintptr_t>(W) & 15) || (reinterpret_cast<uintptr_t>(out) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "permute: C, ldw must be multiples of 8, both matrices 16-byte aligned");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    return sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, out);
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

sb_status sb_sum_scores(sb_ctx* ctx, float* dst, const float* const* src, int n_src, int64_t n, int accumulate) {
    if (!ctx) return SB_ERR_INVALID;
    if (!dst || !src || n <= 0 || n_src < 1 || n_src > SB_SUM_MAX_SRC)
        return sb_fail(ctx, SB_ERR_INVALID, "sum: bad arguments (1 .. %d sources)", SB_SUM_MAX_SRC);
    SumSources ss{};
    for (int k = 0; k < n_src; ++k) {
        if (!src[k]) return sb_fail(ctx, SB_ERR_INVALID, "sum: source %d is NULL", k);
        ss.p[k] = src[k];
    }
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    sum_scores_kernel<<<(unsigned)((n + 255) / 256), 256, 0, ctx->stream>>>(dst, ss, n_src, n, accumulate);
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

}  // extern "C"

// First-order mode (Appendix E.3 "choice of sensitivity statistics"): the paper's own scores
// for Algorithm 2 from a caller-supplied gradient G = dL/dw at the current quantized model,
//   s_up[i]   = - sum_block G (W' - Q_b(W'))         b = the block's CURRENT bitwidth
//   s_down[i] = 2^-b sum_block |G Q_b(W')|
//   s_l1[i]   = sum_block |G (W' - Q_b(W'))|          (p = 1 element sensitivities, summed)
// and one iteration of Algorithm 2 (lines 6-10) on such per-block scores: two sorts, three
// prefix sums and a threshold.  The caller evaluates the loss and decides on acceptance.
#include "lookback.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int FO_THREADS = 128;
constexpr int FO_WARPS = FO_THREADS / 32;
constexpr double FO_MAGIC64 = 6755399441055744.0;   // 1.5 * 2^52: low word of (t + MAGIC) = rint(t)
constexpr unsigned long long KEY_NONE = ~0ull;  // sorts last in either order

struct FoBits { int bits[8]; };

// CTA = one block row x one tile of max(block_cols, 128) columns.  A lane owns 16 consecutive
// columns of a 128-column chunk (two 16-byte loads each of W and G), a warp covers 4 rows per
// step.
__global__ void __launch_bounds__(FO_THREADS)
first_order_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, const __nv_bfloat16* __restrict__ G,
                   int64_t ldg, int br, int bc, int group, FoBits fb, int n_bits,
                   const unsigned char* __restrict__ level, int64_t n_block_cols,
                   float* __restrict__ s_up, float* __restrict__ s_down, float* __restrict__ s_l1,
                   SbDeviceState* ds) {
    __shared__ float red[FO_WARPS][4][3];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cl = lane & 7, slot = lane >> 3;
    const int tile_w = bc >= 128 ? bc : 128;
    const int chunks = tile_w / 128;
    const int piece = bc < 128 ? bc : 128;               // columns of one block inside a chunk
    const int lpp = piece >> 4;                           // lanes per piece
    const int npieces = 128 / piece;
    const int pc = cl / lpp;
    const int64_t bi = blockIdx.y;
    const int64_t bj = bc >= 128 ? (int64_t)blockIdx.x : (int64_t)blockIdx.x * npieces + pc;
    const int64_t blk = bi * n_block_cols + bj;
    int lv = level[blk];
    if (lv >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_SCORES); lv = n_bits - 1; }
    const int b = fb.bits[lv];
    const float qmax = (float)((1 << b) - 1), inv_qmax = 1.0f / qmax;
    const int team = group >> 4;
    float up = 0.f, dn = 0.f, l1 = 0.f;
    for (int ch = 0; ch < chunks; ++ch) {
        const int64_t col = (int64_t)blockIdx.x * tile_w + ch * 128 + cl * 16;
        for (int rr = warp * 4 + slot; rr < br; rr += FO_WARPS * 4) {      // br % 4 == 0
            const int64_t r = bi * br + rr;
            const uint4* pw = reinterpret_cast<const uint4*>(W + r * ldw + col);
            const uint4* pg = reinterpret_cast<const uint4*>(G + r * ldg + col);
            const uint4 w0 = __ldg(pw), w1 = __ldg(pw + 1), g0 = __ldg(pg), g1 = __ldg(pg + 1);
            const uint32_t wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
            const uint32_t gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            float lo, hi;
            group_minmax<8>(wv, team, lo, hi);
            // The signed sum is discontinuous where a code flips, and exact rounding ties are
            // common for bf16 weights on these grids: the codes follow the binary64 sequence
            //   inv = qmax / range; q = rint((v - lo) * inv)
            // literally (as the pack kernel does); the residual v - (lo + q * range / qmax) is then
            // taken in fp32 with the grid step as a two-float sum.
            const double dlo = (double)lo;
            const double range64 = __dsub_rn((double)hi, dlo);            // exact
            const float range = (float)range64;
            const bool live = range64 != 0.0;
            const double inv64 = live ? __ddiv_rn((double)qmax, range64) : 0.0;
            const float ns = live ? -(range * inv_qmax) : 0.f;
            const float ns_lo = live ? -(fmaf(ns, qmax, range) * inv_qmax) : 0.f;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float v = (k & 1) ? bf16hi(wv[k >> 1]) : bf16lo(wv[k >> 1]);
                const float g = (k & 1) ? bf16hi(gv[k >> 1]) : bf16lo(gv[k >> 1]);
                const double t = __dmul_rn(__dsub_rn((double)v, dlo), inv64);
                const unsigned qi = (unsigned)__double2loint(__dadd_rn(t, FO_MAGIC64));   // rint(t), 0..255
                const float q = __uint_as_float(0x4B000000u | qi) - 8388608.f;            // exact int -> float
                const float vm = v - lo;
                const float e = fmaf(q, ns_lo, fmaf(q, ns, vm));          // v - Q(v)
                const float ge = g * e;
                up -= ge;
                l1 += fabsf(ge);
                dn += fabsf(g * (v - e));
            }
        }
    }
    // lanes of the same block, then the four row slots, then the warps: fixed order
    for (int o = lpp >> 1; o > 0; o >>= 1) {
        up += __shfl_xor_sync(0xffffffffu, up, o);
        dn += __shfl_xor_sync(0xffffffffu, dn, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
    }
#pragma unroll
    for (int o = 8; o < 32; o <<= 1) {
        up += __shfl_xor_sync(0xffffffffu, up, o);
        dn += __shfl_xor_sync(0xffffffffu, dn, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
    }
    if (slot == 0 && (cl % lpp) == 0) { red[warp][pc][0] = up; red[warp][pc][1] = dn; red[warp][pc][2] = l1; }
    __syncthreads();
    if (threadIdx.x < npieces) {
        float a = 0.f, d = 0.f, s = 0.f;
#pragma unroll
        for (int wq = 0; wq < FO_WARPS; ++wq) { a += red[wq][threadIdx.x][0]; d += red[wq][threadIdx.x][1]; s += red[wq][threadIdx.x][2]; }
        const int64_t ob = bi * n_block_cols + (bc >= 128 ? (int64_t)blockIdx.x : (int64_t)blockIdx.x * npieces + threadIdx.x);
        int lvo = level[ob];
        if (lvo >= n_bits) lvo = n_bits - 1;
        if (!isfinite(a) || !isfinite(d)) sb_latch(ds, SB_ERR_NONFINITE, SBK_SCORES);
        s_up[ob] = a;
        s_down[ob] = d / (float)(1 << fb.bits[lvo]);
        if (s_l1) s_l1[ob] = s;
    }
}

// ---- one iteration of Algorithm 2 on given scores ---------------------------------------------
struct StepState {
    unsigned long long used;         // sum M_i b_i of the incoming levels
    long long cap, k, h;
    long long n_up, n_down, used_out;
    int expansion, moved;
    double sum_up, sum_down;
};

struct StepArgs {
    const float* s_up; const float* s_down; const unsigned char* level; long long N;
    const long long* block_elems; long long uniform; int L; int bits[8];
    StepState* st;
    SbDeviceState* ds;          // status word (bounds checks of the checked build)
};

__device__ __forceinline__ unsigned long long fo_order_key64(double d) {
    const unsigned long long u = (unsigned long long)__double_as_longlong(d);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
__device__ __forceinline__ long long fo_elems(const StepArgs& a, long long i) {
    return a.block_elems ? a.block_elems[i] : a.uniform;
}

// ranking keys per stored bit, in binary64 from the fp32 scores; ineligible blocks sort last
__global__ void step_keys_fo_kernel(StepArgs a, unsigned long long* kup, unsigned* vup,
                                    unsigned long long* kdn, unsigned* vdn) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long u = 0;
    if (i < a.N) {
        const int l = a.level[i];
        const long long M = fo_elems(a, i);
        const float su = a.s_up[i];
        unsigned long long ku = KEY_NONE, kd = KEY_NONE;
        if (l + 1 < a.L && su > 0.f)
            ku = ~fo_order_key64(__ddiv_rn((double)su, __dmul_rn((double)(a.bits[l + 1] - a.bits[l]), (double)M)));
        if (l > 0 && l < a.L)
            kd = fo_order_key64(__ddiv_rn((double)a.s_down[i], __dmul_rn((double)(a.bits[l] - a.bits[l - 1]), (double)M)));
        if (kd == KEY_NONE && l > 0 && l < a.L) kd = KEY_NONE - 1;      // an eligible key never equals NONE
        kup[i] = ku; vup[i] = (unsigned)i;
        kdn[i] = kd; vdn[i] = (unsigned)i;
        u = (unsigned long long)(M * a.bits[l < a.L ? l : a.L - 1]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
    if ((threadIdx.x & 31) == 0 && u) atomicAdd(&a.st->used, u);    // integer: order-independent
}

// cost of the p-th up-candidate if it is among the first `lim` (0 otherwise)
__global__ void step_upcost_kernel(StepArgs a, const unsigned long long* __restrict__ kup,
                                   const unsigned* __restrict__ vup, long long lim,
                                   unsigned long long* __restrict__ cost) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= a.N) return;
    unsigned long long c = 0;
    if (p < lim && kup[p] != KEY_NONE) {
        const long long i = vup[p];
        const int l = a.level[i];
        c = (unsigned long long)(fo_elems(a, i) * (a.bits[l + 1] - a.bits[l]));
    }
    cost[p] = c;
}
__global__ void step_mark_up_kernel(const unsigned long long* __restrict__ kup, const unsigned* __restrict__ vup,
                                    long long N, long long h, unsigned char* __restrict__ in_up) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < N && p < h && kup[p] != KEY_NONE) in_up[vup[p]] = 1;
}
__global__ void step_dnflag_kernel(const unsigned long long* __restrict__ kdn, const unsigned* __restrict__ vdn,
                                   long long N, const unsigned char* __restrict__ in_up,
                                   unsigned* __restrict__ flag) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < N) flag[p] = (kdn[p] != KEY_NONE && !in_up[vdn[p]]) ? 1u : 0u;
}
__global__ void step_dncost_kernel(StepArgs a, const unsigned* __restrict__ vdn, const unsigned* __restrict__ flag,
                                   const unsigned* __restrict__ rank, long long h,
                                   unsigned long long* __restrict__ cost) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= a.N) return;
    unsigned long long c = 0;
    if (flag[p] && (long long)rank[p] < h) {
        const long long i = vdn[p];
        const int l = a.level[i];
        c = (unsigned long long)(fo_elems(a, i) * (a.bits[l] - a.bits[l - 1]));
    }
    cost[p] = c;
}

// number of leading entries p < lim whose inclusive cumulative cost cum[p + 1] is <= bound
// (cum is the exclusive scan with the total in cum[N]; costs are positive for p < lim)
__device__ long long fo_prefix_fit(const unsigned long long* cum, long long lim, long long bound) {
    if (bound < 0) return 0;
    long long lo = 0, hi = lim;                 // answer in [0, lim]
    while (lo < hi) {
        const long long mid = (lo + hi + 1) / 2;
        if ((long long)cum[mid] <= bound) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// one thread: the step's few scalars (binary searches over the scanned arrays)
__global__ void step_decide_kernel(StepArgs a, const unsigned long long* __restrict__ kup,
                                   const unsigned long long* __restrict__ cumup,
                                   const unsigned* __restrict__ flag, const unsigned* __restrict__ dnrank,
                                   const unsigned long long* __restrict__ cumdn) {
    StepState* st = a.st;
    const long long N = a.N, k = st->k, h = st->h;
    // eligible up-candidates: the prefix of the sorted list before the first NONE
    long long lo = 0, hi = N;
    while (lo < hi) {
        const long long mid = (lo + hi) / 2;
        if (kup[mid] == KEY_NONE) hi = mid; else lo = mid + 1;
    }
    const long long n_elig = lo;
    const long long used = (long long)st->used, slack = st->cap - used;
    st->expansion = 0; st->moved = 0; st->n_up = 0; st->n_down = 0; st->used_out = used;
    if (used < st->cap) {
        const long long lim = n_elig < k ? n_elig : k;
        const long long n = fo_prefix_fit(cumup, lim, slack);
        if (n > 0) {
            st->expansion = 1; st->moved = 1; st->n_up = n;
            st->used_out = used + (long long)cumup[n];
            return;
        }
    }
    const long long limh = n_elig < h ? n_elig : h;
    const long long n_flag = (long long)dnrank[N - 1] + (long long)flag[N - 1];
    const long long nD = n_flag < h ? n_flag : h;
    const long long freed = (long long)cumdn[N];
    const long long nU = fo_prefix_fit(cumup, limh, slack + freed);
    if (nU > 0 && nD > 0) {
        st->moved = 1; st->n_up = nU; st->n_down = nD;
        st->used_out = used + (long long)cumup[nU] - freed;
    }
}

// the moves, and the sums of the moved blocks' scores (per-CTA partials, added in CTA order)
constexpr int AP_THREADS = 256;
__global__ void __launch_bounds__(AP_THREADS)
step_apply_kernel(StepArgs a, const unsigned* __restrict__ vup, const unsigned* __restrict__ vdn,
                  const unsigned* __restrict__ flag, const unsigned* __restrict__ dnrank,
                  unsigned char* __restrict__ level_out, double* __restrict__ part) {
    __shared__ double sh[2][AP_THREADS / 32];
    const StepState st = *a.st;
    const long long p = (long long)blockIdx.x * AP_THREADS + threadIdx.x;
    double su = 0.0, sd = 0.0;
    if (st.moved && p < a.N) {
        if (p < st.n_up) {
            const long long i = vup[p];
            if (SB_IN_BOUNDS(a.ds, SBK_ALLOC, i, a.N)) {
                level_out[i] = (unsigned char)(a.level[i] + 1);
                su = (double)a.s_up[i];
            }
        }
        if (!st.expansion && flag[p] && (long long)dnrank[p] < st.h) {
            const long long i = vdn[p];
            if (SB_IN_BOUNDS(a.ds, SBK_ALLOC, i, a.N)) {
                level_out[i] = (unsigned char)(a.level[i] - 1);
                sd = (double)a.s_down[i];
            }
        }
    }
    su = warp_sum(su); sd = warp_sum(sd);
    if ((threadIdx.x & 31) == 0) { sh[0][threadIdx.x >> 5] = su; sh[1][threadIdx.x >> 5] = sd; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double x = 0.0, y = 0.0;
        for (int wq = 0; wq < AP_THREADS / 32; ++wq) { x += sh[0][wq]; y += sh[1][wq]; }
        part[2 * blockIdx.x] = x; part[2 * blockIdx.x + 1] = y;
    }
}
__global__ void step_finish_kernel(StepArgs a, const double* __restrict__ part, int nparts) {
    double x = 0.0, y = 0.0;
    for (int q = 0; q < nparts; ++q) { x += part[2 * q]; y += part[2 * q + 1]; }
    a.st->sum_up = x; a.st->sum_down = y;
}

}  // namespace

extern "C" {

sb_status sb_first_order_scores(sb_ctx* ctx, const void* W, const void* G, int64_t R, int64_t C,
                                int64_t ldw, int64_t ldg, const int32_t* row_perm, const int32_t* col_perm,
                                int br, int bc, int group, const int* bits, int n_bits, const uint8_t* level,
                                float* s_up, float* s_down, float* s_l1) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !G || !level || !s_up || !s_down || R <= 0 || C <= 0)
        return sb_fail(ctx, SB_ERR_INVALID, "first-order scores: null or empty");
    if (!sb_check_bits(bits, n_bits))
        return sb_fail(ctx, SB_ERR_INVALID, "first-order scores: bits must be ascending in 1..8");
    const bool g_ok = group == 16 || group == 32 || group == 64 || group == 128;
    if (br <= 0 || bc <= 0 || br % 4 || R % br || C % bc || !g_ok || bc % group || C % 128 ||
        !(bc == 32 || bc == 64 || bc % 128 == 0) || ldw % 8 || ldw < C || ldg % 8 || ldg < C ||
        (reinterpret_cast<uintptr_t>(W) & 15) || (reinterpret_cast<uintptr_t>(G) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "first-order scores: block %dx%d group %d does not tile %lldx%lld",
                       br, bc, group, (long long)R, (long long)C);
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const __nv_bfloat16* w = static_cast<const __nv_bfloat16*>(W);
    const __nv_bfloat16* g = static_cast<const __nv_bfloat16*>(G);
    int64_t lw = ldw, lg = ldg;
    if (row_perm || col_perm) {          // the permuted layout of both matrices, in scratch
        void* arena;
        const size_t bytes = (size_t)R * C * 2;
        sb_status st = sb_scratch(ctx, Carver::need({bytes, bytes}), &arena);
        if (st != SB_OK) return st;
        Carver cv(arena);
        void* wp = cv.take<unsigned char>(bytes);
        void* gp = cv.take<unsigned char>(bytes);
        st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, wp);
        if (st != SB_OK) return st;
        st = sb_gather_bf16(ctx, G, R, C, ldg, row_perm, col_perm, gp);
        if (st != SB_OK) return st;
        w = static_cast<const __nv_bfloat16*>(wp); g = static_cast<const __nv_bfloat16*>(gp);
        lw = lg = C;
    }
    FoBits fb{};
    for (int l = 0; l < 8; ++l) fb.bits[l] = l < n_bits ? bits[l] : bits[n_bits - 1];
    const int tile_w = bc >= 128 ? bc : 128;
    dim3 grid((unsigned)(C / tile_w), (unsigned)(R / br));
    first_order_kernel<<<grid, FO_THREADS, 0, ctx->stream>>>(w, lw, g, lg, br, bc, group, fb, n_bits, level,
                                                            C / bc, s_up, s_down, s_l1, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

sb_status sb_exchange_step(sb_ctx* ctx, const float* s_up, const float* s_down, const uint8_t* level,
                           int64_t N, const int64_t* block_elems, int64_t uniform_block_elems,
                           const int* bits, int n_bits, double budget, int64_t k, uint8_t* level_out,
                           sb_step_report* report) {
    if (!ctx) return SB_ERR_INVALID;
    if (!s_up || !s_down || !level || !level_out || !report || N <= 0 || k < 1)
        return sb_fail(ctx, SB_ERR_INVALID, "exchange step: null, empty or k < 1");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "exchange step: bits must be ascending in 1..8");
    if (!block_elems && uniform_block_elems <= 0) return sb_fail(ctx, SB_ERR_INVALID, "exchange step: block size");
    if (N >= (1ll << 32)) return sb_fail(ctx, SB_ERR_SHAPE, "exchange step: N must fit 32 bits");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(report, 0, sizeof *report);

    const size_t ns = (size_t)N + 1;
    const size_t sort_bytes = sb_radix_sort_scratch_bytes(N);
    const int nparts = (int)((N + AP_THREADS - 1) / AP_THREADS);
    void* arena;
    sb_status stt = sb_scratch(ctx, Carver::need({sizeof(StepState), ns * 8, ns * 8, ns * 8, ns * 4, ns * 4,
                                                   ns * 4, ns * 8, ns * 8, ns * 4, ns * 4, (size_t)N,
                                                   (size_t)nparts * 16, sort_bytes, ns * 8}), &arena);
    if (stt != SB_OK) return stt;
    Carver cv(arena);
    StepState* dst = cv.take<StepState>(1);
    unsigned long long* kup = cv.take<unsigned long long>(ns);
    unsigned long long* kdn = cv.take<unsigned long long>(ns);
    unsigned long long* ktmp = cv.take<unsigned long long>(ns);
    unsigned* vup = cv.take<unsigned>(ns);
    unsigned* vdn = cv.take<unsigned>(ns);
    unsigned* vtmp = cv.take<unsigned>(ns);
    unsigned long long* cumup = cv.take<unsigned long long>(ns);
    unsigned long long* cumdn = cv.take<unsigned long long>(ns);
    unsigned* flag = cv.take<unsigned>(ns);
    unsigned* dnrank = cv.take<unsigned>(ns);
    unsigned char* in_up = cv.take<unsigned char>((size_t)N);
    double* part = cv.take<double>((size_t)nparts * 2);
    void* sort_scratch = cv.take<unsigned char>(sort_bytes);
    unsigned long long* cost = cv.take<unsigned long long>(ns);

    long long total_elems = 0;
    StepState* hst = static_cast<StepState*>(ctx->pinned);
    if (block_elems) {
        stt = sb_scan_exclusive_u64(ctx, reinterpret_cast<const unsigned long long*>(block_elems), cost, N);
        if (stt != SB_OK) return stt;
        SB_CUDA(ctx, cudaMemcpyAsync(hst, cost + N, 8, cudaMemcpyDeviceToHost, ctx->stream));
        SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        total_elems = *reinterpret_cast<long long*>(hst);
    } else {
        total_elems = (long long)N * uniform_block_elems;
    }
    StepState init{};
    init.cap = (long long)floor(budget * (double)total_elems);
    init.k = k;
    init.h = k / 2 > 0 ? k / 2 : 1;
    memcpy(hst, &init, sizeof init);
    SB_CUDA(ctx, cudaMemcpyAsync(dst, hst, sizeof init, cudaMemcpyHostToDevice, ctx->stream));

    StepArgs a{};
    a.s_up = s_up; a.s_down = s_down; a.level = level; a.N = N;
    a.block_elems = reinterpret_cast<const long long*>(block_elems); a.uniform = uniform_block_elems;
    a.L = n_bits;
    for (int l = 0; l < 8; ++l) a.bits[l] = l < n_bits ? bits[l] : 0;
    a.st = dst; a.ds = ctx->dstate;
    const unsigned g = (unsigned)((N + 255) / 256);
    step_keys_fo_kernel<<<g, 256, 0, ctx->stream>>>(a, kup, vup, kdn, vdn);
    SB_LAUNCHED(ctx);
    stt = sb_radix_sort_u64(ctx, kup, ktmp, vup, vtmp, N, sort_scratch);
    if (stt != SB_OK) return stt;
    stt = sb_radix_sort_u64(ctx, kdn, ktmp, vdn, vtmp, N, sort_scratch);
    if (stt != SB_OK) return stt;
    // costs of the first k up-candidates and their prefix sums (the first h are a prefix of them)
    step_upcost_kernel<<<g, 256, 0, ctx->stream>>>(a, kup, vup, k, cost);
    SB_LAUNCHED(ctx);
    stt = sb_scan_exclusive_u64(ctx, cost, cumup, N);
    if (stt != SB_OK) return stt;
    // the down set: the first h down-eligible blocks that are not among the first h up-candidates
    SB_CUDA(ctx, cudaMemsetAsync(in_up, 0, (size_t)N, ctx->stream));
    step_mark_up_kernel<<<g, 256, 0, ctx->stream>>>(kup, vup, N, init.h, in_up);
    SB_LAUNCHED(ctx);
    step_dnflag_kernel<<<g, 256, 0, ctx->stream>>>(kdn, vdn, N, in_up, flag);
    SB_LAUNCHED(ctx);
    stt = sb_scan_exclusive_u32(ctx, flag, dnrank, N);
    if (stt != SB_OK) return stt;
    step_dncost_kernel<<<g, 256, 0, ctx->stream>>>(a, vdn, flag, dnrank, init.h, cost);
    SB_LAUNCHED(ctx);
    stt = sb_scan_exclusive_u64(ctx, cost, cumdn, N);
    if (stt != SB_OK) return stt;
    step_decide_kernel<<<1, 1, 0, ctx->stream>>>(a, kup, cumup, flag, dnrank, cumdn);
    SB_LAUNCHED(ctx);
    if (level_out != level)
        SB_CUDA(ctx, cudaMemcpyAsync(level_out, level, (size_t)N, cudaMemcpyDeviceToDevice, ctx->stream));
    step_apply_kernel<<<(unsigned)nparts, AP_THREADS, 0, ctx->stream>>>(a, vup, vdn, flag, dnrank, level_out, part);
    SB_LAUNCHED(ctx);
    step_finish_kernel<<<1, 1, 0, ctx->stream>>>(a, part, nparts);
    SB_LAUNCHED(ctx);
    SB_CUDA(ctx, cudaMemcpyAsync(hst, dst, sizeof(StepState), cudaMemcpyDeviceToHost, ctx->stream));
    SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    const StepState fin = *hst;
    report->cap_bits = fin.cap; report->used_in = (int64_t)fin.used; report->used_out = fin.used_out;
    report->expansion = fin.expansion; report->moved = fin.moved;
    report->n_up = fin.n_up; report->n_down = fin.n_down;
    report->sum_up = fin.sum_up; report->sum_down = fin.sum_down;
    return sb_sync(ctx);
}

}  // extern "C"

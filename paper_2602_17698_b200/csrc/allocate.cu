// Global bit allocation on the separable proxy loss L(level) = sum_i err[i][level_i].
//
// Algorithm 2 re-ranks all blocks by the gain of their next step up (down) in every
// iteration.  With a static table those gains are the fixed numbers
//     g(i, l) = (err[i][l] - err[i][l+1]) / ((b_{l+1} - b_l) M_i),
// so all N (L-1) steps are sorted ONCE (by the binary64 key, ties to the lower block), and
// the ranking of an iteration is the sub-sequence of that list whose step starts (ends) at
// the block's current level.  "Top k by s_up, truncated to the budget" then is one
// device-wide prefix sum of (count, cost) over the flagged entries -- a single look-back
// scan per direction and iteration instead of a sort.  Algorithm 1 (greedy along each
// block's convex hull) is one sort, one scan of the step costs and a threshold.
#include "lookback.cuh"

namespace {

constexpr int AT = 256;             // threads of the scan-select kernels
constexpr int AI = 8;               // entries per thread
constexpr int ATILE = AT * AI;
constexpr int BT = 256;             // threads of the per-block kernels

struct AllocState {
    long long cap, used;
    double loss, loss_init;
    long long k, kT;
    int iter, accepted, rejected, expansions;
    int done, status;
    // per-iteration accumulators (cleared by the update step)
    int expand_ok;                  // the best up-step fits the slack: expansion stage
    int accept;
    unsigned nU, nD;
    unsigned long long freed, costU;
    double dU, dD;
    unsigned done_down, done_decide, done_apply, done_eval;   // last-CTA tickets
    long long hist[8];
};

struct AllocArgs {
    const float* err; const long long* block_elems; long long uniform;
    long long N; int L; int bits[8];
    unsigned char* level;
    AllocState* st;
    unsigned* uprank; unsigned* upstamp; unsigned long long* upcum;   // per block
    unsigned* dnstamp; unsigned* ustamp;                               // per block
    double* part;                                                      // partial sums
};

__device__ __forceinline__ unsigned long long order_key64(double d) {
    const unsigned long long u = (unsigned long long)__double_as_longlong(d);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
__device__ __forceinline__ long long elems_of(const AllocArgs& a, long long i) {
    return a.block_elems ? a.block_elems[i] : a.uniform;
}
__device__ __forceinline__ double gain64(const AllocArgs& a, long long i, int from, int to) {
    const double num = __dsub_rn((double)a.err[i * a.L + from], (double)a.err[i * a.L + to]);
    const double den = __dmul_rn((double)(a.bits[to] - a.bits[from]), (double)elems_of(a, i));
    return __ddiv_rn(num, den);
}

// deterministic CTA sum of one double per thread (fixed tree), result in thread 0
template <int NT>
__device__ __forceinline__ double cta_sum(double v) {
    __shared__ double sh[NT / 32];
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < NT / 32; ++w) s += sh[w];
    __syncthreads();
    return s;
}

// true in exactly one CTA: the last one to get here.  All writes and atomics of every CTA
// made before the call are visible to it afterwards.
__device__ __forceinline__ bool cta_is_last(unsigned* counter) {
    __shared__ bool last_sh;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_sh = atomicAdd(counter, 1u) == gridDim.x - 1;
    __syncthreads();
    const bool last = last_sh;
    if (last) __threadfence();
    return last;
}

// ---- set-up -----------------------------------------------------------------------------
// keys of all steps e = i (L-1) + l; up list sorts descending (key = ~order), down ascending
__global__ void step_keys_kernel(AllocArgs a, unsigned long long* kup, unsigned long long* kdn,
                                 unsigned* vup, unsigned* vdn) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n = a.N * (a.L - 1);
    if (e >= n) return;
    const long long i = e / (a.L - 1);
    const int l = (int)(e % (a.L - 1));
    const unsigned long long o = order_key64(gain64(a, i, l, l + 1));
    kup[e] = ~o; kdn[e] = o;
    vup[e] = (unsigned)e; vdn[e] = (unsigned)e;
}

// level = l0 everywhere; loss / used partial sums; also clears the per-block stamps
__global__ void __launch_bounds__(BT) init_levels_kernel(AllocArgs a, int l0, int clear) {
    const long long i = (long long)blockIdx.x * BT + threadIdx.x;
    double e = 0.0;
    long long u = 0;
    if (i < a.N) {
        a.level[i] = (unsigned char)l0;
        e = (double)a.err[i * a.L + l0];
        u = elems_of(a, i) * a.bits[l0];
        if (clear) { a.upstamp[i] = 0; a.dnstamp[i] = 0; a.ustamp[i] = 0; }
    }
    const double s = cta_sum<BT>(e);
    if (threadIdx.x == 0) a.part[blockIdx.x] = s;
    // integer sums are order-independent: plain atomics
    unsigned long long uu = (unsigned long long)u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) uu += __shfl_xor_sync(0xffffffffu, uu, o);
    if ((threadIdx.x & 31) == 0 && uu) atomicAdd((unsigned long long*)&a.st->used, uu);
}
__global__ void init_finish_kernel(AllocArgs a, int nparts) {
    double s = 0.0;
    for (int p = 0; p < nparts; ++p) s += a.part[p];
    a.st->loss = s;
    a.st->loss_init = s;
}

// ---- one iteration of Algorithm 2 ---------------------------------------------------------
// Step 1: walk the up list; entries whose step starts at the block's level and gains > 0 are
// candidates.  Candidate number p (0-based) with p < k records its rank and the cumulative
// cost of candidates 0..p.
__global__ void __launch_bounds__(AT)
select_up_kernel(AllocArgs a, const unsigned* __restrict__ list, long long n, LookbackBuf lb,
                 unsigned epoch, SbDeviceState* ds) {
    const unsigned tile = lookback_tile_id(ds);
    const AllocState s = *a.st;
    if (s.done) return;   // every tile sees the same state: nobody waits on anybody
    const long long base = (long long)tile * ATILE + (long long)threadIdx.x * AI;
    unsigned blk[AI]; unsigned long long cost[AI]; bool flag[AI];
    CntCost sum{0ull, 0u, 0u};
#pragma unroll
    for (int j = 0; j < AI; ++j) {
        flag[j] = false; cost[j] = 0; blk[j] = 0;
        if (base + j < n) {
            const unsigned e = list[base + j];
            const long long i = e / (unsigned)(a.L - 1);
            const int l = (int)(e % (unsigned)(a.L - 1));
            if (a.level[i] == l && a.err[i * a.L + l] > a.err[i * a.L + l + 1]) {
                flag[j] = true;
                blk[j] = (unsigned)i;
                cost[j] = (unsigned long long)(elems_of(a, i) * (a.bits[l + 1] - a.bits[l]));
                sum.cnt += 1; sum.cost += cost[j];
            }
        }
    }
    CntCost tile_total;
    CntCost ex = block_exclusive_scan<CntCost, AT>(sum, tile_total);
    const CntCost prefix = lookback_prefix<CntCost>(tile_total, tile, lb, epoch, ds);
    CntCost run = t_add(prefix, ex);
    if ((long long)run.cnt >= s.k) return;
#pragma unroll
    for (int j = 0; j < AI; ++j) {
        if (!flag[j]) continue;
        const unsigned p = run.cnt;
        run.cnt += 1; run.cost += cost[j];
        if ((long long)p < s.k) {
            a.uprank[blk[j]] = p;
            a.upcum[blk[j]] = run.cost;
            a.upstamp[blk[j]] = (unsigned)s.iter + 1u;
            if (p == 0 && s.used < s.cap && (long long)cost[j] <= s.cap - s.used) a.st->expand_ok = 1;
        }
    }
}

// Step 2 (exchange stage only): walk the down list; entries whose step ends at the block's
// level, outside the first h up-candidates, are down-candidates; the first h of them form D.
__global__ void __launch_bounds__(AT)
select_down_kernel(AllocArgs a, const unsigned* __restrict__ list, long long n, LookbackBuf lb,
                   unsigned epoch, SbDeviceState* ds) {
    const unsigned tile = lookback_tile_id(ds);
    const AllocState s = *a.st;
    if (s.done || s.expand_ok) return;   // uniform over the grid (set before this launch)
    const long long h = s.k / 2 > 0 ? s.k / 2 : 1;
    const unsigned stamp = (unsigned)s.iter + 1u;
    const long long base = (long long)tile * ATILE + (long long)threadIdx.x * AI;
    unsigned blk[AI]; unsigned long long cost[AI]; double de[AI]; bool flag[AI];
    CntCost sum{0ull, 0u, 0u};
#pragma unroll
    for (int j = 0; j < AI; ++j) {
        flag[j] = false; cost[j] = 0; blk[j] = 0; de[j] = 0.0;
        if (base + j < n) {
            const unsigned e = list[base + j];
            const long long i = e / (unsigned)(a.L - 1);
            const int l = (int)(e % (unsigned)(a.L - 1));
            const bool in_u0 = a.upstamp[i] == stamp && (long long)a.uprank[i] < h;
            if (a.level[i] == l + 1 && !in_u0) {
                flag[j] = true;
                blk[j] = (unsigned)i;
                cost[j] = (unsigned long long)(elems_of(a, i) * (a.bits[l + 1] - a.bits[l]));
                de[j] = __dsub_rn((double)a.err[i * a.L + l], (double)a.err[i * a.L + l + 1]);
                sum.cnt += 1; sum.cost += cost[j];
            }
        }
    }
    CntCost tile_total;
    CntCost ex = block_exclusive_scan<CntCost, AT>(sum, tile_total);
    const CntCost prefix = lookback_prefix<CntCost>(tile_total, tile, lb, epoch, ds);
    CntCost run = t_add(prefix, ex);
    double dsum = 0.0; unsigned long long fsum = 0; unsigned cnt = 0;
#pragma unroll
    for (int j = 0; j < AI; ++j) {
        if (!flag[j]) continue;
        const unsigned p = run.cnt;
        run.cnt += 1;
        if ((long long)p < h) {
            a.dnstamp[blk[j]] = stamp;
            dsum += de[j]; fsum += cost[j]; cnt += 1;
        }
    }
    const double tsum = cta_sum<AT>(dsum);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        fsum += __shfl_xor_sync(0xffffffffu, fsum, o);
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    }
    if ((threadIdx.x & 31) == 0 && cnt) {
        atomicAdd(&a.st->freed, fsum);
        atomicAdd(&a.st->nD, cnt);
    }
    if (threadIdx.x == 0) a.part[tile] = tsum;
    if (cta_is_last(&a.st->done_down) && threadIdx.x == 0) {
        double t = 0.0;
        for (unsigned p = 0; p < gridDim.x; ++p) t += ((volatile double*)a.part)[p];
        a.st->dD = t;
    }
}

// Step 3: the up-set U.  Expansion: candidates 0..k-1 whose cumulative cost fits the slack.
// Exchange: candidates 0..h-1 whose cumulative cost fits slack + what D frees.  The last CTA
// adds the partial gains in a fixed order and takes the accept decision.
__global__ void __launch_bounds__(BT) decide_kernel(AllocArgs a, double* part) {
    const AllocState s = *a.st;
    if (s.done) return;
    const long long i = (long long)blockIdx.x * BT + threadIdx.x;
    const unsigned stamp = (unsigned)s.iter + 1u;
    const bool expand = s.expand_ok != 0;
    const long long h = s.k / 2 > 0 ? s.k / 2 : 1;
    const long long lim_rank = expand ? s.k : h;
    const long long lim_cost = (s.cap - s.used) + (expand ? 0ll : (long long)s.freed);
    double de = 0.0; unsigned long long c = 0; unsigned cnt = 0;
    if (i < a.N && a.upstamp[i] == stamp && (long long)a.uprank[i] < lim_rank &&
        (long long)a.upcum[i] <= lim_cost) {
        const int l = a.level[i];
        a.ustamp[i] = stamp;
        de = __dsub_rn((double)a.err[i * a.L + l], (double)a.err[i * a.L + l + 1]);
        c = (unsigned long long)(elems_of(a, i) * (a.bits[l + 1] - a.bits[l]));
        cnt = 1;
    }
    const double tsum = cta_sum<BT>(de);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        c += __shfl_xor_sync(0xffffffffu, c, o);
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    }
    if ((threadIdx.x & 31) == 0 && cnt) {
        atomicAdd(&a.st->costU, c);
        atomicAdd(&a.st->nU, cnt);
    }
    if (threadIdx.x == 0) part[blockIdx.x] = tsum;
    if (cta_is_last(&a.st->done_decide) && threadIdx.x == 0) {
        double t = 0.0;
        for (unsigned p = 0; p < gridDim.x; ++p) t += ((volatile double*)part)[p];
        a.st->dU = t;
        const unsigned nU = *(volatile unsigned*)&a.st->nU, nD = *(volatile unsigned*)&a.st->nD;
        const double dD = *(volatile double*)&a.st->dD;
        a.st->accept = expand ? (nU > 0) : (nU > 0 && nD > 0 && t > dD);
    }
}

// Step 4: apply the move, then (last CTA) advance the loop state.
__global__ void __launch_bounds__(BT) apply_kernel(AllocArgs a) {
    const AllocState s = *a.st;
    if (s.done) return;
    const long long i = (long long)blockIdx.x * BT + threadIdx.x;
    const unsigned stamp = (unsigned)s.iter + 1u;
    const bool expand = s.expand_ok != 0;
    if (i < a.N && s.accept) {
        if (a.ustamp[i] == stamp) a.level[i] += 1;
        else if (!expand && a.dnstamp[i] == stamp) a.level[i] -= 1;
    }
    if (cta_is_last(&a.st->done_apply) && threadIdx.x == 0) {
        AllocState* st = a.st;
        if (expand && s.accept) {
            st->used = s.used + (long long)s.costU;
            st->loss = s.loss - s.dU;
            st->expansions = s.expansions + 1;
        } else if (s.accept) {
            st->used = s.used + (long long)s.costU - (long long)s.freed;
            st->loss = s.loss + (s.dD - s.dU);
            st->accepted = s.accepted + 1;
        } else {
            st->k = s.k / 2;
            st->rejected = s.rejected + 1;
        }
        st->iter = s.iter + 1;
        if (st->k < s.kT) st->done = 1;
        else if (st->iter >= 4096) { st->done = 1; st->status = SB_ERR_NOCONVERGE; }
        st->expand_ok = 0; st->accept = 0; st->nU = 0; st->nD = 0; st->freed = 0; st->costU = 0;
        st->dU = 0.0; st->dD = 0.0;
        st->done_down = 0; st->done_decide = 0; st->done_apply = 0;
        __threadfence();
    }
}

// ---- Algorithm 1 ---------------------------------------------------------------------------
// Hull steps of block i from level 0: the next vertex is the level of strictly lower error with
// the steepest slope (exact ties: the farthest).  Entry e = i (L-1) + (q-1) describes the step
// INTO level q; non-vertices sort last with cost 0.
__global__ void hull_steps_kernel(AllocArgs a, unsigned long long* keys, unsigned* vals,
                                  unsigned long long* stepcost) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.N) return;
    const int L = a.L;
    for (int q = 1; q < L; ++q) {
        const long long e = i * (L - 1) + (q - 1);
        keys[e] = ~0ull; vals[e] = (unsigned)e; stepcost[e] = 0ull;
    }
    int p = 0;
    double prev = 0.0; bool have_prev = false;
    while (p < L - 1) {
        int best = -1; double bs = 0.0;
        for (int q = p + 1; q < L; ++q) {
            if (!(a.err[i * L + q] < a.err[i * L + p])) continue;
            const double sl = gain64(a, i, p, q);
            if (best < 0 || sl >= bs) { best = q; bs = sl; }
        }
        if (best < 0) break;
        // keys never rise along a block, so the global order keeps a block's steps in sequence
        if (have_prev && bs > prev) bs = prev;
        const long long e = i * (L - 1) + (best - 1);
        keys[e] = ~order_key64(bs);
        stepcost[e] = (unsigned long long)(elems_of(a, i) * (a.bits[best] - a.bits[p]));
        prev = bs; have_prev = true;
        p = best;
    }
}
__global__ void gather_cost_kernel(const unsigned* __restrict__ list, const unsigned long long* __restrict__ stepcost,
                                   long long n, unsigned long long* out) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < n) out[p] = stepcost[list[p]];
}
// selected = valid step whose inclusive cumulative cost fits the slack; level = highest target
__global__ void greedy_apply_kernel(AllocArgs a, const unsigned* __restrict__ list,
                                    const unsigned long long* __restrict__ cost_sorted,
                                    const unsigned long long* __restrict__ excl, long long n,
                                    int* level32, int* steps) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    const unsigned long long c = cost_sorted[p];
    if (c == 0) return;
    const long long slack = a.st->cap - a.st->used;
    if ((long long)(excl[p] + c) > slack) return;
    const unsigned e = list[p];
    const long long i = e / (unsigned)(a.L - 1);
    const int q = (int)(e % (unsigned)(a.L - 1)) + 1;
    atomicMax(level32 + i, q);
    atomicAdd(steps, 1);
}
__global__ void level_from32_kernel(AllocArgs a, const int* level32) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < a.N) a.level[i] = (unsigned char)level32[i];
}

// loss, used bits and level histogram of the final allocation
__global__ void __launch_bounds__(BT) eval_kernel(AllocArgs a, double* part, int set_loss) {
    const long long i = (long long)blockIdx.x * BT + threadIdx.x;
    double e = 0.0; unsigned long long u = 0;
    __shared__ unsigned hist[8];
    if (threadIdx.x < 8) hist[threadIdx.x] = 0;
    __syncthreads();
    if (i < a.N) {
        const int l = a.level[i];
        e = (double)a.err[i * a.L + l];
        u = (unsigned long long)(elems_of(a, i) * a.bits[l]);
        atomicAdd(&hist[l & 7], 1u);
    }
    const double s = cta_sum<BT>(e);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
    if ((threadIdx.x & 31) == 0 && u && set_loss) atomicAdd((unsigned long long*)&a.st->used, u);
    __syncthreads();
    if (threadIdx.x < 8 && hist[threadIdx.x]) atomicAdd((unsigned long long*)&a.st->hist[threadIdx.x], (unsigned long long)hist[threadIdx.x]);
    if (threadIdx.x == 0) part[blockIdx.x] = s;
    if (cta_is_last(&a.st->done_eval) && threadIdx.x == 0 && set_loss) {
        double t = 0.0;
        for (unsigned p = 0; p < gridDim.x; ++p) t += ((volatile double*)part)[p];
        a.st->loss = t;
    }
}

}  // namespace

extern "C" sb_status sb_allocate_bits(sb_ctx* ctx, const float* err, int64_t N,
                                      const int64_t* block_elems, int64_t uniform_block_elems,
                                      const int* bits, int n_bits, double budget, int mode,
                                      double gamma0, double gammaT, uint8_t* level,
                                      sb_alloc_report* report) {
    if (!ctx) return SB_ERR_INVALID;
    if (!err || !level || !report || N <= 0) return sb_fail(ctx, SB_ERR_INVALID, "allocate: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "allocate: bits must be ascending in 1..8");
    if (!block_elems && uniform_block_elems <= 0) return sb_fail(ctx, SB_ERR_INVALID, "allocate: block size");
    if (mode != SB_ALLOC_SCALEBITS && mode != SB_ALLOC_GREEDY) return sb_fail(ctx, SB_ERR_INVALID, "allocate: mode");
    if (mode == SB_ALLOC_SCALEBITS &&
        (!(gamma0 > 0.0) || !(gammaT > 0.0) || gamma0 > 1.0 || gammaT > 1.0))
        return sb_fail(ctx, SB_ERR_INVALID, "allocate: gamma0, gammaT must lie in (0, 1]");
    const int L = n_bits;
    const long long nsteps = (long long)N * (L - 1);
    if (nsteps >= (1ll << 32)) return sb_fail(ctx, SB_ERR_SHAPE, "allocate: N * (n_bits - 1) must fit 32 bits");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    memset(report, 0, sizeof *report);

    // total weights -> cap.  Uniform blocks: closed form; else a device sum via the scan.
    const int nblkB = (int)((N + BT - 1) / BT);
    const long long ntiles = (nsteps + ATILE - 1) / ATILE;
    const size_t nparts = (size_t)(nblkB > ntiles ? nblkB : ntiles) + 8;
    const size_t sort_bytes = sb_radix_sort_scratch_bytes(nsteps > 0 ? nsteps : 1);
    const size_t ns = (size_t)(nsteps > 0 ? nsteps : 1) + 1;
    void* arena;
    sb_status stt = sb_scratch(ctx, Carver::need({sizeof(AllocState), ns * 8, ns * 8, ns * 8, ns * 8,
                                                   ns * 4, ns * 4, ns * 4, ns * 4,
                                                   (size_t)N * 4, (size_t)N * 4, (size_t)N * 8,
                                                   (size_t)N * 4, (size_t)N * 4, nparts * 8,
                                                   nparts * 8, sort_bytes, (size_t)(N + 1) * 8}), &arena);
    if (stt != SB_OK) return stt;
    Carver cv(arena);
    AllocState* dst = cv.take<AllocState>(1);
    unsigned long long* kA = cv.take<unsigned long long>(ns);
    unsigned long long* kB = cv.take<unsigned long long>(ns);
    unsigned long long* kC = cv.take<unsigned long long>(ns);
    unsigned long long* kD = cv.take<unsigned long long>(ns);
    unsigned* vA = cv.take<unsigned>(ns);
    unsigned* vB = cv.take<unsigned>(ns);
    unsigned* vC = cv.take<unsigned>(ns);
    unsigned* vD = cv.take<unsigned>(ns);
    unsigned* uprank = cv.take<unsigned>((size_t)N);
    unsigned* upstamp = cv.take<unsigned>((size_t)N);
    unsigned long long* upcum = cv.take<unsigned long long>((size_t)N);
    unsigned* dnstamp = cv.take<unsigned>((size_t)N);
    unsigned* ustamp = cv.take<unsigned>((size_t)N);
    double* part = cv.take<double>(nparts);
    double* part2 = cv.take<double>(nparts);
    void* sort_scratch = cv.take<unsigned char>(sort_bytes);
    unsigned long long* totals = cv.take<unsigned long long>((size_t)N + 1);

    long long total_elems = 0;
    AllocState* hst = static_cast<AllocState*>(ctx->pinned);
    if (block_elems) {
        stt = sb_scan_exclusive_u64(ctx, reinterpret_cast<const unsigned long long*>(block_elems), totals, N);
        if (stt != SB_OK) return stt;
        SB_CUDA(ctx, cudaMemcpyAsync(hst, totals + N, 8, cudaMemcpyDeviceToHost, ctx->stream));
        SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        total_elems = *reinterpret_cast<long long*>(hst);
    } else {
        total_elems = (long long)N * uniform_block_elems;
    }
    const long long cap = (long long)floor(budget * (double)total_elems);
    report->cap_bits = cap;

    AllocArgs a{};
    a.err = err; a.block_elems = reinterpret_cast<const long long*>(block_elems);
    a.uniform = uniform_block_elems; a.N = N; a.L = L;
    for (int l = 0; l < 8; ++l) a.bits[l] = l < L ? bits[l] : 0;
    a.level = level; a.st = dst;
    a.uprank = uprank; a.upstamp = upstamp; a.upcum = upcum; a.dnstamp = dnstamp; a.ustamp = ustamp;
    a.part = part;

    int l0 = 0;
    AllocState init{};
    init.cap = cap;
    if (mode == SB_ALLOC_SCALEBITS) {
        l0 = -1;
        for (int l = 0; l < L; ++l) if ((double)bits[l] <= budget) l0 = l;
        if (l0 < 0) return sb_fail(ctx, SB_ERR_BUDGET, "allocate: budget %.4f below the smallest candidate %d", budget, bits[0]);
        long long k = (long long)floor(gamma0 * (double)N); if (k < 1) k = 1;
        long long kT = (long long)floor(gammaT * (double)N); if (kT < 1) kT = 1;
        if (k < kT) k = kT;
        init.k = k; init.kT = kT;
    }
    memcpy(hst, &init, sizeof init);
    SB_CUDA(ctx, cudaMemcpyAsync(dst, hst, sizeof init, cudaMemcpyHostToDevice, ctx->stream));
    init_levels_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, l0, 1);
    SB_LAUNCHED(ctx);
    init_finish_kernel<<<1, 1, 0, ctx->stream>>>(a, nblkB);
    SB_LAUNCHED(ctx);

    auto read_state = [&](AllocState* out) -> sb_status {
        SB_CUDA(ctx, cudaMemcpyAsync(hst, dst, sizeof(AllocState), cudaMemcpyDeviceToHost, ctx->stream));
        SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        *out = *hst;
        return SB_OK;
    };

    AllocState fin{};
    if (mode == SB_ALLOC_GREEDY) {
        // the lowest candidate must fit
        stt = read_state(&fin);
        if (stt != SB_OK) return stt;
        report->proxy_loss_init = fin.loss_init;
        report->used_bits = fin.used;
        if (fin.used > cap) return sb_fail(ctx, SB_ERR_BUDGET, "allocate: budget below the smallest candidate");
        if (nsteps > 0) {
            int* level32 = reinterpret_cast<int*>(uprank);
            int* steps = reinterpret_cast<int*>(upstamp);
            SB_CUDA(ctx, cudaMemsetAsync(level32, 0, sizeof(int) * N, ctx->stream));
            SB_CUDA(ctx, cudaMemsetAsync(steps, 0, sizeof(int), ctx->stream));
            hull_steps_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, kA, vA, kC);
            SB_LAUNCHED(ctx);
            stt = sb_radix_sort_u64(ctx, kA, kB, vA, vB, nsteps, sort_scratch);
            if (stt != SB_OK) return stt;
            const unsigned g = (unsigned)((nsteps + 255) / 256);
            gather_cost_kernel<<<g, 256, 0, ctx->stream>>>(vA, kC, nsteps, kB);
            SB_LAUNCHED(ctx);
            stt = sb_scan_exclusive_u64(ctx, kB, kD, nsteps);   // kD needs nsteps + 1 entries
            if (stt != SB_OK) return stt;
            greedy_apply_kernel<<<g, 256, 0, ctx->stream>>>(a, vA, kB, kD, nsteps, level32, steps);
            SB_LAUNCHED(ctx);
            level_from32_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, level32);
            SB_LAUNCHED(ctx);
            SB_CUDA(ctx, cudaMemcpyAsync(reinterpret_cast<int*>(hst) + 512, steps, sizeof(int),
                                         cudaMemcpyDeviceToHost, ctx->stream));
        }
        // recompute used / loss / histogram from the final levels
        SB_CUDA(ctx, cudaMemsetAsync(&dst->used, 0, sizeof(long long), ctx->stream));
        eval_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, part2, 1);
        SB_LAUNCHED(ctx);
        stt = read_state(&fin);
        if (stt != SB_OK) return stt;
        report->iterations = nsteps > 0 ? reinterpret_cast<int*>(hst)[512] : 0;
        report->accepted = report->iterations;
    } else {
        report->proxy_loss_init = 0.0;
        if (nsteps > 0) {
            const unsigned g = (unsigned)((nsteps + 255) / 256);
            step_keys_kernel<<<g, 256, 0, ctx->stream>>>(a, kA, kC, vA, vC);
            SB_LAUNCHED(ctx);
            stt = sb_radix_sort_u64(ctx, kA, kB, vA, vB, nsteps, sort_scratch);
            if (stt != SB_OK) return stt;
            stt = sb_radix_sort_u64(ctx, kC, kD, vC, vD, nsteps, sort_scratch);
            if (stt != SB_OK) return stt;
            bool done = false;
            int chunk = 8;
            while (!done) {
                for (int it = 0; it < chunk; ++it) {
                    unsigned epoch; sb_status s2;
                    LookbackBuf lb = sb_lookback(ctx, (unsigned)ntiles, &epoch, &s2);
                    if (s2 != SB_OK) return s2;
                    select_up_kernel<<<(unsigned)ntiles, AT, 0, ctx->stream>>>(a, vA, nsteps, lb, epoch, ctx->dstate);
                    SB_LAUNCHED(ctx);
                    lb = sb_lookback(ctx, (unsigned)ntiles, &epoch, &s2);
                    if (s2 != SB_OK) return s2;
                    select_down_kernel<<<(unsigned)ntiles, AT, 0, ctx->stream>>>(a, vC, nsteps, lb, epoch, ctx->dstate);
                    SB_LAUNCHED(ctx);
                    decide_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, part2);
                    SB_LAUNCHED(ctx);
                    apply_kernel<<<nblkB, BT, 0, ctx->stream>>>(a);
                    SB_LAUNCHED(ctx);
                }
                stt = read_state(&fin);
                if (stt != SB_OK) return stt;
                done = fin.done != 0;
            }
        }
        // single candidate (or finished): histogram of the final levels
        eval_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, part2, 0);
        SB_LAUNCHED(ctx);
        stt = read_state(&fin);
        if (stt != SB_OK) return stt;
        report->proxy_loss_init = fin.loss_init;
    }
    report->used_bits = fin.used;
    report->proxy_loss_final = fin.loss;
    if (mode == SB_ALLOC_SCALEBITS) {
        report->iterations = fin.iter;
        report->accepted = fin.accepted;
        report->rejected = fin.rejected;
        report->expansions = fin.expansions;
    }
    for (int l = 0; l < 8; ++l) report->level_hist[l] = fin.hist[l];
    // device status (look-back timeouts, non-finite inputs latched earlier)
    sb_status dev = sb_sync(ctx);
    if (dev != SB_OK) return dev;
    if (fin.status != 0) return sb_fail(ctx, (sb_status)fin.status, "allocate: iteration cap reached");
    return SB_OK;
}

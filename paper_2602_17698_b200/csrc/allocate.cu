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
#include <cooperative_groups.h>

#include "lookback.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int AT = 256;             // threads of the scan-select kernels
constexpr int AI = 8;               // entries per thread
constexpr int ATILE = AT * AI;
constexpr int BT = 256;             // threads of the per-block kernels
constexpr int LT_WARPS_MAX = 32;
constexpr int LOOP_MAX_CTAS = 4096;
constexpr int GL_THREADS = 256;     // grid (cooperative) form of the loop kernel
constexpr int CL_THREADS = 512, CL_CTAS = 16;   // cluster form
constexpr int LC = 4;               // list entries a thread has in flight at a time
constexpr unsigned ENT_NONE = 0xffffffffu;      // list entry that is never a candidate

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
    long long used_init;            // bits of the warm start (greedy: of the lowest candidate)
};

struct AllocArgs {
    const float* err; const long long* block_elems; long long uniform;
    long long N; int L; int bits[8];
    unsigned char* level;
    AllocState* st;
    // per block: (stamp << 32 | rank) of its up-candidate, the cumulative cost and the error
    // difference of that candidate, and the move marked for the apply step (stamp << 1 | down)
    unsigned long long* upsr; unsigned long long* upcum; double* upde; unsigned* mark;
    double* part;                                                      // partial sums
    SbDeviceState* ds;                                                 // status word (bounds checks of the checked build)
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

// The same sums (fixed tree, so every CTA that adds the same values gets the same bits) for two
// doubles per thread, result in EVERY thread, one CTA barrier: the buffer alternates with `flip`,
// and a buffer is written again only after the barrier of the call in between.
template <int NT>
__device__ __forceinline__ void cta_sum2_all(double& u, double& d, unsigned& flip) {
    __shared__ double sh[2][2][NT / 32];
    u = warp_sum(u); d = warp_sum(d);
    if ((threadIdx.x & 31) == 0) { sh[flip][0][threadIdx.x >> 5] = u; sh[flip][1][threadIdx.x >> 5] = d; }
    __syncthreads();
    double su = 0.0, sd = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) { su += sh[flip][0][w]; sd += sh[flip][1][w]; }
    u = su; d = sd;
    flip ^= 1u;
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
// keys of all steps e = i (L-1) + l; the up list sorts by gain descending (key = ~order)
__global__ void step_keys_kernel(AllocArgs a, unsigned long long* kup, unsigned* vup) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n = a.N * (a.L - 1);
    if (e >= n) return;
    const long long i = e / (a.L - 1);
    const int l = (int)(e % (a.L - 1));
    const unsigned long long o = order_key64(gain64(a, i, l, l + 1));
    kup[e] = ~o;
    vup[e] = (unsigned)e;
}

// The down list (gain ascending, ties to the lower step id) is the up list (gain descending,
// ties to the lower step id) read backwards, except that runs of equal keys keep their order.
__global__ void tie_heads_kernel(const unsigned long long* __restrict__ keys, long long n,
                                 unsigned* __restrict__ head) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < n) head[p] = (p == 0 || keys[p] != keys[p - 1]) ? 1u : 0u;
}
__global__ void run_starts_kernel(const unsigned* __restrict__ head, const unsigned* __restrict__ excl,
                                  long long n, unsigned* __restrict__ start) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    if (head[p]) start[excl[p]] = (unsigned)p;                    // run id = excl[p]
    if (p == n - 1) start[excl[p] + head[p]] = (unsigned)n;       // one past the last run
}
// Both lists in the form the loop reads: entry = block << 3 | from-level, plus the error
// difference of the step.  Up-steps that do not lower the error are never candidates.
__global__ void entry_info_kernel(AllocArgs a, const unsigned* __restrict__ up_list,
                                  const unsigned* __restrict__ head, const unsigned* __restrict__ excl,
                                  const unsigned* __restrict__ start, long long n,
                                  unsigned* __restrict__ up_ent, double* __restrict__ up_de,
                                  unsigned* __restrict__ dn_ent, double* __restrict__ dn_de) {
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    const unsigned e = up_list[p], Lm1 = (unsigned)(a.L - 1);
    const unsigned i = e / Lm1, l = e - i * Lm1;
    const float e0 = a.err[(long long)i * a.L + l], e1 = a.err[(long long)i * a.L + l + 1];
    const double de = __dsub_rn((double)e0, (double)e1);
    const unsigned ent = (i << 3) | l;
    up_ent[p] = e0 > e1 ? ent : ENT_NONE;
    up_de[p] = de;
    const unsigned r = excl[p] + head[p] - 1u;
    const long long ra = start[r], rb = start[r + 1];
    const long long q = (n - rb) + (p - ra);
    dn_ent[q] = ent;
    dn_de[q] = de;
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
        if (clear) { a.upsr[i] = 0ull; a.mark[i] = 0u; }
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
    a.st->used_init = a.st->used;
}
// The loop state before the first kernel reads it, computed where it is used so that the call
// needs no host round trip: cap = floor(budget * total weights), k = floor(gamma0 N) and
// kT = floor(gammaT N), both at least 1 (the same binary64 operations the host would do).
__global__ void init_state_kernel(AllocState* st, const unsigned long long* total_dev, long long total_host,
                                  double budget, double gamma0, double gammaT, long long N, int scalebits) {
    AllocState z{};
    const long long total = total_dev ? (long long)*total_dev : total_host;
    z.cap = (long long)floor(budget * (double)total);
    if (scalebits) {
        long long k = (long long)floor(gamma0 * (double)N); if (k < 1) k = 1;
        long long kT = (long long)floor(gammaT * (double)N); if (kT < 1) kT = 1;
        if (k < kT) k = kT;
        z.k = k; z.kT = kT;
    }
    *st = z;
}
// The report in the caller's device memory; conditions the loop found are latched for sb_sync.
__global__ void report_kernel(AllocArgs a, const int* greedy_steps, int greedy, sb_alloc_report* rep) {
    const AllocState s = *a.st;
    sb_alloc_report r{};
    r.cap_bits = s.cap;
    r.used_bits = s.used;
    r.proxy_loss_init = s.loss_init;
    r.proxy_loss_final = s.loss;
    if (greedy) {
        r.iterations = greedy_steps ? *greedy_steps : 0;
        r.accepted = r.iterations;
        if (s.used_init > s.cap) sb_latch(a.ds, SB_ERR_BUDGET, SBK_ALLOC);   // the lowest candidate must fit
    } else {
        r.iterations = s.iter; r.accepted = s.accepted; r.rejected = s.rejected; r.expansions = s.expansions;
        if (s.status != 0) sb_latch(a.ds, s.status, SBK_ALLOC);              // iteration cap reached
    }
    for (int l = 0; l < 8; ++l) r.level_hist[l] = s.hist[l];
    *rep = r;
}

// ---- the Algorithm 2 loop, one persistent kernel ----------------------------------------------
// All iterations run inside one launch; the phases of an iteration are separated by barriers over
// all CTAs (every CTA is resident: one thread-block cluster, or a cooperative launch).  CTA c owns
// a contiguous slice of both sorted lists.  A "select" is two passes over the slice: (1) count the
// candidates and add up their costs, publish the CTA total; (2) after the barrier, the exclusive
// prefix over the lower CTAs gives every candidate its global rank and cumulative cost.  The loop
// state (k, used, loss, counters) is replicated: every CTA derives it from the same published
// totals, added in the same order, so no CTA has to wait for a single writer.
//   expansion iteration: up-count | up-rank + U | apply            (3 barriers)
//   exchange  iteration: up-count | up-rank | down-count | down-rank + D | U | apply   (6)
// The lists are static: entry p carries (block << 3 | from-level) and the error difference of its
// step, so a pass costs one dependent load (the block's current level), issued for LC entries at a
// time.  Data written by other CTAs during the kernel is read through L2 (__ldcg): L1 is not
// coherent across SMs inside one launch.
struct LoopWork {
    CntCost* up_tot; long long* up_first; CntCost* dn_tot;
    double* dD; unsigned long long* freed; unsigned* nD;
    double* dU; unsigned long long* costU; unsigned* nU;
};

__device__ __forceinline__ CntCost ldcg_cc(const CntCost* p) {
    const ulonglong2 v = __ldcg(reinterpret_cast<const ulonglong2*>(p));
    CntCost c; c.cost = v.x; c.cnt = (unsigned)v.y; c.pad = 0u;
    return c;
}

// Reduction of K 64-bit values per thread over the CTA, result in every thread, fixed order.
// OPS holds two bits per slot: 0 = sum, 1 = min, 2 = max.  One barrier per call: the buffer
// alternates, and any later call's barrier separates a buffer's readers from its next writers.
template <int OP>
__device__ __forceinline__ unsigned long long red_op(unsigned long long x, unsigned long long y) {
    if constexpr (OP == 0) return x + y;
    else if constexpr (OP == 1) return x < y ? x : y;
    else return x > y ? x : y;
}
template <int NT, int K, int OPS, int S = 0>
__device__ __forceinline__ void allreduce_slot(unsigned long long (&v)[K], unsigned long long (*sh)[K]) {
    if constexpr (S < K) {
        constexpr int OP = (OPS >> (2 * S)) & 3;
        unsigned long long r = sh[0][S];
#pragma unroll
        for (int wq = 1; wq < NT / 32; ++wq) r = red_op<OP>(r, sh[wq][S]);
        v[S] = r;
        allreduce_slot<NT, K, OPS, S + 1>(v, sh);
    }
}
template <int NT, int K, int OPS, int S = 0>
__device__ __forceinline__ void warpreduce_slot(unsigned long long (&v)[K]) {
    if constexpr (S < K) {
        constexpr int OP = (OPS >> (2 * S)) & 3;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v[S] = red_op<OP>(v[S], __shfl_xor_sync(0xffffffffu, v[S], o));
        warpreduce_slot<NT, K, OPS, S + 1>(v);
    }
}
template <int NT, int K, int OPS>
__device__ __forceinline__ void cta_allreduce(unsigned long long (&v)[K], unsigned& flip) {
    __shared__ unsigned long long sh[2][NT / 32][K];
    warpreduce_slot<NT, K, OPS>(v);
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int s = 0; s < K; ++s) sh[flip][threadIdx.x >> 5][s] = v[s];
    }
    __syncthreads();
    allreduce_slot<NT, K, OPS>(v, sh[flip]);
    flip ^= 1u;
}

template <int LT, bool CLUSTER>
__global__ void __launch_bounds__(LT)
scalebits_loop_kernel(AllocArgs a, const unsigned* __restrict__ up_ent, const double* __restrict__ up_de,
                      const unsigned* __restrict__ dn_ent, const double* __restrict__ dn_de,
                      long long ne, LoopWork w) {
    // CLUSTER: the whole grid is one thread-block cluster and the phase barrier is the hardware
    // cluster barrier; otherwise a cooperative launch and the grid-wide barrier
    auto phase_barrier = [&]() {
        if (CLUSTER) cg::this_cluster().sync();
        else cg::this_grid().sync();
    };
    const int G = gridDim.x, c = blockIdx.x, tid = threadIdx.x;
    const long long per_cta = (ne + G - 1) / G;
    const long long ipt = (per_cta + LT - 1) / LT;                    // entries per thread
    const long long cta_hi = min(ne, (long long)(c + 1) * per_cta);
    const long long t_lo = min(cta_hi, (long long)c * per_cta + (long long)tid * ipt);
    const long long t_hi = min(cta_hi, t_lo + ipt);

    const AllocState s0 = *a.st;                    // written before the launch
    const long long cap = s0.cap, kT = s0.kT;
    long long k = s0.k, used = s0.used;
    double loss = s0.loss;
    int iter = 0, accepted = 0, rejected = 0, expansions = 0, status = 0;
    unsigned flip = 0, flip2 = 0;

    // bit difference of the step l -> l + 1 in nibble l (a table in registers, not in local memory)
    unsigned dbits = 0;
#pragma unroll
    for (int l = 0; l < 7; ++l) dbits |= (unsigned)(a.bits[l + 1] > a.bits[l] ? a.bits[l + 1] - a.bits[l] : 0) << (4 * l);
    const long long* const block_elems = a.block_elems;
    const long long uniform = a.uniform;
    auto cost_of = [&](unsigned e) -> unsigned long long {
        const long long m = block_elems ? block_elems[e >> 3] : uniform;
        return (unsigned long long)(m * (long long)((dbits >> (4u * (e & 7u))) & 15u));
    };
    // visit(p, e) for this thread's up-candidates in list order, until it returns false
    auto for_up = [&](auto&& visit) {
        for (long long base = t_lo; base < t_hi; base += LC) {
            unsigned e[LC]; int lv[LC];
#pragma unroll
            for (int j = 0; j < LC; ++j) e[j] = base + j < t_hi ? __ldg(up_ent + base + j) : ENT_NONE;
#pragma unroll
            for (int j = 0; j < LC; ++j) lv[j] = e[j] != ENT_NONE ? (int)__ldcg(a.level + (e[j] >> 3)) : -1;
#pragma unroll
            for (int j = 0; j < LC; ++j)
                if (lv[j] == (int)(e[j] & 7u)) { if (!visit(base + j, e[j])) return; }
        }
    };
    // down-candidates: the step ends at the block's level and the block is not among the first
    // h up-candidates of this iteration
    auto for_dn = [&](unsigned stamp, long long h, auto&& visit) {
        for (long long base = t_lo; base < t_hi; base += LC) {
            unsigned e[LC]; int lv[LC]; unsigned long long sr[LC];
#pragma unroll
            for (int j = 0; j < LC; ++j) e[j] = base + j < t_hi ? __ldg(dn_ent + base + j) : ENT_NONE;
#pragma unroll
            for (int j = 0; j < LC; ++j) {
                lv[j] = -1; sr[j] = 0ull;
                if (e[j] != ENT_NONE) {
                    lv[j] = (int)__ldcg(a.level + (e[j] >> 3));
                    sr[j] = __ldcg(a.upsr + (e[j] >> 3));
                }
            }
#pragma unroll
            for (int j = 0; j < LC; ++j) {
                if (lv[j] != (int)(e[j] & 7u) + 1) continue;
                if ((unsigned)(sr[j] >> 32) == stamp && (long long)(unsigned)sr[j] < h) continue;
                if (!visit(base + j, e[j])) return;
            }
        }
    };

    while (k >= kT) {
        if (iter >= 4096) { status = SB_ERR_NOCONVERGE; break; }
        const unsigned stamp = (unsigned)iter + 1u;
        const long long slack = cap - used;
        const long long h = k / 2 > 0 ? k / 2 : 1;

        // ---- up-count ---------------------------------------------------------------------------
        CntCost mine{0ull, 0u, 0u};
        long long my_first = -1;
        for_up([&](long long, unsigned e) {
            const unsigned long long cost = cost_of(e);
            if (mine.cnt == 0) my_first = (long long)cost;
            mine.cnt += 1; mine.cost += cost;
            return true;
        });
        CntCost cta_tot;
        const CntCost ex = block_exclusive_scan<CntCost, LT>(mine, cta_tot);
        if (ex.cnt == 0 && mine.cnt > 0) w.up_first[c] = my_first;      // the CTA's first candidate
        if (tid == 0) {
            w.up_tot[c] = cta_tot;
            if (cta_tot.cnt == 0) w.up_first[c] = -1;
        }
        phase_barrier();

        // ---- prefix over the lower CTAs, cost of the globally first candidate ------------------
        unsigned long long pre[3] = {0ull, 0ull, 0x7fffffffull};      // cost, count, first CTA with one
        for (int j = tid; j < G; j += LT) {
            const CntCost t = ldcg_cc(w.up_tot + j);
            if (j < c) { pre[0] += t.cost; pre[1] += t.cnt; }
            if (t.cnt > 0 && (unsigned long long)j < pre[2]) pre[2] = (unsigned long long)j;
        }
        cta_allreduce<LT, 3, 0 | (0 << 2) | (1 << 4)>(pre, flip);
        const long long first_cost = pre[2] != 0x7fffffffull ? __ldcg(w.up_first + pre[2]) : -1;
        const bool expand = used < cap && first_cost >= 0 && first_cost <= slack;
        const long long lim_rank = expand ? k : h;

        // ---- up-rank (and, in an expansion, the set U itself) -----------------------------------
        // U is a prefix of the ranked candidates, so its cost is the largest cumulative cost in it
        double dU_mine = 0.0; unsigned long long costU_mine = 0; unsigned nU_mine = 0;
        if (mine.cnt > 0 && (long long)pre[1] + ex.cnt < lim_rank) {
            unsigned long long run_cost = pre[0] + ex.cost;
            long long run_cnt = (long long)pre[1] + ex.cnt;
            for_up([&](long long p, unsigned e) {
                const long long i = (long long)(e >> 3);
                const double de = __ldg(up_de + p);
                run_cost += cost_of(e);
                a.upsr[i] = ((unsigned long long)stamp << 32) | (unsigned long long)(unsigned)run_cnt;
                a.upcum[i] = run_cost;
                a.upde[i] = de;
                if (expand && (long long)run_cost <= slack) {
                    a.mark[i] = stamp << 1;
                    dU_mine += de; costU_mine = run_cost; nU_mine += 1;
                }
                run_cnt += 1;
                return run_cnt < lim_rank;
            });
        }
        if (expand) {
            const double d = cta_sum<LT>(dU_mine);
            unsigned long long r2[2] = {costU_mine, nU_mine};
            cta_allreduce<LT, 2, 2 | (0 << 2)>(r2, flip);
            if (tid == 0) { w.dU[c] = d; w.costU[c] = r2[0]; w.nU[c] = (unsigned)r2[1]; }
        }
        phase_barrier();

        if (!expand) {
            // ---- down-count ----------------------------------------------------------------------
            CntCost dm{0ull, 0u, 0u};
            for_dn(stamp, h, [&](long long, unsigned e) { dm.cnt += 1; dm.cost += cost_of(e); return true; });
            CntCost dn_cta;
            const CntCost dex = block_exclusive_scan<CntCost, LT>(dm, dn_cta);
            if (tid == 0) w.dn_tot[c] = dn_cta;
            phase_barrier();
            unsigned long long dpre[1] = {0ull};
            for (int j = tid; j < c; j += LT) dpre[0] += ldcg_cc(w.dn_tot + j).cnt;
            cta_allreduce<LT, 1, 0>(dpre, flip);
            // ---- down-rank: the first h candidates form D -----------------------------------------
            double dD_mine = 0.0; unsigned long long freed_mine = 0; unsigned nD_mine = 0;
            if (dm.cnt > 0 && (long long)dpre[0] + dex.cnt < h) {
                long long run_cnt = (long long)dpre[0] + dex.cnt;
                for_dn(stamp, h, [&](long long p, unsigned e) {
                    a.mark[e >> 3] = (stamp << 1) | 1u;
                    dD_mine += __ldg(dn_de + p); freed_mine += cost_of(e); nD_mine += 1;
                    run_cnt += 1;
                    return run_cnt < h;
                });
            }
            {
                const double d = cta_sum<LT>(dD_mine);
                unsigned long long r2[2] = {freed_mine, nD_mine};
                cta_allreduce<LT, 2, 0>(r2, flip);
                if (tid == 0) { w.dD[c] = d; w.freed[c] = r2[0]; w.nD[c] = (unsigned)r2[1]; }
            }
            phase_barrier();
            // ---- U: up-candidates 0..h-1 whose cumulative cost fits slack + what D frees ------------
            unsigned long long fr[1] = {0ull};
            for (int j = tid; j < G; j += LT) fr[0] += __ldcg(w.freed + j);
            cta_allreduce<LT, 1, 0>(fr, flip);
            const long long lim_cost = slack + (long long)fr[0];
            for (long long i = (long long)c * LT + tid; i < a.N; i += (long long)G * LT) {
                const unsigned long long sr = __ldcg(a.upsr + i), cum = __ldcg(a.upcum + i);
                const double de = __ldcg(a.upde + i);
                if ((unsigned)(sr >> 32) == stamp && (long long)(unsigned)sr < h && (long long)cum <= lim_cost) {
                    a.mark[i] = stamp << 1;
                    dU_mine += de; nU_mine += 1;
                    if (cum > costU_mine) costU_mine = cum;
                }
            }
            const double d = cta_sum<LT>(dU_mine);
            unsigned long long r2[2] = {costU_mine, nU_mine};
            cta_allreduce<LT, 2, 2 | (0 << 2)>(r2, flip);
            if (tid == 0) { w.dU[c] = d; w.costU[c] = r2[0]; w.nU[c] = (unsigned)r2[1]; }
            phase_barrier();
        }

        // ---- totals (same order in every CTA), decision, apply, replicated state update -----------
        // every thread fetches the totals of its CTAs at once (one L2 round trip, not one per CTA);
        // the sums over CTAs follow a fixed tree
        double dU = 0.0, dD = 0.0;
        unsigned long long tot[4] = {0ull, 0ull, 0ull, 0ull};       // costU (max), nU, freed, nD
        for (int j = tid; j < G; j += LT) {
            dU += __ldcg(w.dU + j);
            if (!expand) dD += __ldcg(w.dD + j);
            const unsigned long long cu = __ldcg(w.costU + j);
            if (cu > tot[0]) tot[0] = cu;
            tot[1] += __ldcg(w.nU + j);
            if (!expand) { tot[2] += __ldcg(w.freed + j); tot[3] += __ldcg(w.nD + j); }
        }
        cta_allreduce<LT, 4, 2 | (0 << 2) | (0 << 4) | (0 << 6)>(tot, flip);
        const unsigned long long costU = tot[0], freed = tot[2];
        const unsigned nU = (unsigned)tot[1], nD = (unsigned)tot[3];
        cta_sum2_all<LT>(dU, dD, flip2);
        const bool accept = expand ? (nU > 0) : (nU > 0 && nD > 0 && dU > dD);
        if (accept) {
            for (long long i = (long long)c * LT + tid; i < a.N; i += (long long)G * LT) {
                const unsigned m = __ldcg(a.mark + i);
                if ((m >> 1) == stamp)
                    a.level[i] = (unsigned char)((int)__ldcg(a.level + i) + ((m & 1u) ? -1 : 1));
            }
        }
        if (expand && accept) { used += (long long)costU; loss -= dU; expansions += 1; }
        else if (accept) { used += (long long)costU - (long long)freed; loss += dD - dU; accepted += 1; }
        else { k /= 2; rejected += 1; }
        iter += 1;
        phase_barrier();                                  // the new levels are visible to the next up-count
    }
    if (c == 0 && tid == 0) {
        AllocState* st = a.st;
        st->k = k; st->used = used; st->loss = loss; st->iter = iter; st->accepted = accepted;
        st->rejected = rejected; st->expansions = expansions; st->done = 1; st->status = status;
    }
}

// The same loop for lists of at most 32 entries per thread (every layer-sized and model-sized
// table on a full grid): a thread remembers its candidates of an iteration as bit masks, so the
// rank, the membership of U / D and the apply step walk those bits instead of re-reading the
// blocks' levels, and nothing per block but the up-rank stamp (read by the down pass) is stored.
// Dependent L2 round trips per expansion iteration: 3 instead of 8.
template <int LT, bool CLUSTER>
__global__ void __launch_bounds__(LT)
scalebits_loop_masked_kernel(AllocArgs a, const unsigned* __restrict__ up_ent, const double* __restrict__ up_de,
                             const unsigned* __restrict__ dn_ent, const double* __restrict__ dn_de,
                             long long ne, LoopWork w) {
    auto phase_barrier = [&]() {
        if (CLUSTER) cg::this_cluster().sync();
        else cg::this_grid().sync();
    };
    constexpr int MLC = 8;             // list entries in flight per thread: one round for the layer-sized lists
    const int G = gridDim.x, c = blockIdx.x, tid = threadIdx.x;
    const long long per_cta = (ne + G - 1) / G;
    const long long ipt = (per_cta + LT - 1) / LT;                    // entries per thread, <= 32
    const long long cta_hi = min(ne, (long long)(c + 1) * per_cta);
    const long long t_lo = min(cta_hi, (long long)c * per_cta + (long long)tid * ipt);
    const long long t_hi = min(cta_hi, t_lo + ipt);
    const int n_mine = (int)(t_hi - t_lo);

    const AllocState s0 = *a.st;                    // written before the launch
    const long long cap = s0.cap, kT = s0.kT;
    long long k = s0.k, used = s0.used;
    double loss = s0.loss;
    int iter = 0, accepted = 0, rejected = 0, expansions = 0, status = 0;
    unsigned flip = 0, flip2 = 0;

    unsigned dbits = 0;
#pragma unroll
    for (int l = 0; l < 7; ++l) dbits |= (unsigned)(a.bits[l + 1] > a.bits[l] ? a.bits[l + 1] - a.bits[l] : 0) << (4 * l);
    const long long* const block_elems = a.block_elems;
    const long long uniform = a.uniform;
    auto cost_of = [&](unsigned e) -> unsigned long long {
        const long long m = block_elems ? block_elems[e >> 3] : uniform;
        return (unsigned long long)(m * (long long)((dbits >> (4u * (e & 7u))) & 15u));
    };
    constexpr unsigned long long FIRST_NONE = ~0ull;

    while (k >= kT) {
        if (iter >= 4096) { status = SB_ERR_NOCONVERGE; break; }
        const unsigned stamp = (unsigned)iter + 1u;
        const long long slack = cap - used;
        const long long h = k / 2 > 0 ? k / 2 : 1;

        // ---- up-count: candidate mask, count, cost ----------------------------------------------
        unsigned cm = 0;
        CntCost mine{0ull, 0u, 0u};
        unsigned long long my_first = 0;
        for (int b0 = 0; b0 < n_mine; b0 += MLC) {
            unsigned e[MLC]; int lv[MLC];
#pragma unroll
            for (int j = 0; j < MLC; ++j) e[j] = b0 + j < n_mine ? __ldg(up_ent + t_lo + b0 + j) : ENT_NONE;
#pragma unroll
            for (int j = 0; j < MLC; ++j) lv[j] = e[j] != ENT_NONE ? (int)__ldcg(a.level + (e[j] >> 3)) : -1;
#pragma unroll
            for (int j = 0; j < MLC; ++j) {
                if (lv[j] == (int)(e[j] & 7u)) {
                    const unsigned long long cost = cost_of(e[j]);
                    if (mine.cnt == 0) my_first = cost;
                    mine.cnt += 1; mine.cost += cost;
                    cm |= 1u << (b0 + j);
                }
            }
        }
        CntCost cta_tot;
        const CntCost ex = block_exclusive_scan<CntCost, LT>(mine, cta_tot);
        if (ex.cnt == 0 && mine.cnt > 0) w.up_first[c] = (long long)my_first;   // the CTA's first candidate
        if (tid == 0) {
            w.up_tot[c] = cta_tot;
            if (cta_tot.cnt == 0) w.up_first[c] = -1;
        }
        phase_barrier();

        // ---- prefix over the lower CTAs; cost of the globally first candidate (key = CTA, cost) --
        unsigned long long pre[3] = {0ull, 0ull, FIRST_NONE};
        for (int j = tid; j < G; j += LT) {
            const CntCost t = ldcg_cc(w.up_tot + j);
            const long long fc = __ldcg(w.up_first + j);
            if (j < c) { pre[0] += t.cost; pre[1] += t.cnt; }
            if (t.cnt > 0) {
                const unsigned long long key = ((unsigned long long)j << 48) | ((unsigned long long)fc & 0xffffffffffffull);
                if (key < pre[2]) pre[2] = key;
            }
        }
        cta_allreduce<LT, 3, 0 | (0 << 2) | (1 << 4)>(pre, flip);
        const long long first_cost = pre[2] != FIRST_NONE ? (long long)(pre[2] & 0xffffffffffffull) : -1;
        const bool expand = used < cap && first_cost >= 0 && first_cost <= slack;
        const long long lim_rank = expand ? k : h;
        const unsigned long long base_cost = pre[0] + ex.cost;
        const long long base_cnt = (long long)pre[1] + ex.cnt;

        // ---- up-rank: in an expansion the set U itself, else the stamps the down pass excludes ----
        // U is a prefix of the ranked candidates, so its cost is the largest cumulative cost in it
        double dU_mine = 0.0; unsigned long long costU_mine = 0; unsigned nU_mine = 0;
        unsigned um = 0;
        if (cm && base_cnt < lim_rank) {
            unsigned long long run_cost = base_cost;
            long long run_cnt = base_cnt;
            for (unsigned m = cm; m && run_cnt < lim_rank; m &= m - 1) {
                const int j = __ffs(m) - 1;
                const unsigned e = __ldg(up_ent + t_lo + j);
                run_cost += cost_of(e);
                if (expand) {
                    if ((long long)run_cost <= slack) {
                        um |= 1u << j;
                        dU_mine += __ldg(up_de + t_lo + j); costU_mine = run_cost; nU_mine += 1;
                    }
                } else {
                    a.upsr[e >> 3] = ((unsigned long long)stamp << 32) | (unsigned long long)(unsigned)run_cnt;
                }
                run_cnt += 1;
            }
        }
        if (expand) {
            // an expansion is accepted whenever U is not empty, and U is known here: the owner of a
            // list entry writes the block's new level now, so the barrier below also publishes the
            // levels and the iteration needs no third one
            for (unsigned m = um; m; m &= m - 1) {
                const unsigned e = __ldg(up_ent + t_lo + (__ffs(m) - 1));
                if (SB_IN_BOUNDS(a.ds, SBK_ALLOC, e >> 3, a.N)) a.level[e >> 3] = (unsigned char)((e & 7u) + 1u);
            }
            const double d = cta_sum<LT>(dU_mine);
            unsigned long long r2[2] = {costU_mine, nU_mine};
            cta_allreduce<LT, 2, 2 | (0 << 2)>(r2, flip);
            if (tid == 0) { w.dU[c] = d; w.costU[c] = r2[0]; w.nU[c] = (unsigned)r2[1]; }
        }
        phase_barrier();

        unsigned dsel = 0;
        if (!expand) {
            // ---- down-count: the step ends at the block's level, the block is not in the up set ----
            unsigned dcm = 0;
            CntCost dm{0ull, 0u, 0u};
            for (int b0 = 0; b0 < n_mine; b0 += MLC) {
                unsigned e[MLC]; int lv[MLC]; unsigned long long sr[MLC];
#pragma unroll
                for (int j = 0; j < MLC; ++j) e[j] = b0 + j < n_mine ? __ldg(dn_ent + t_lo + b0 + j) : ENT_NONE;
#pragma unroll
                for (int j = 0; j < MLC; ++j) {
                    lv[j] = -1; sr[j] = 0ull;
                    if (e[j] != ENT_NONE) {
                        lv[j] = (int)__ldcg(a.level + (e[j] >> 3));
                        sr[j] = __ldcg(a.upsr + (e[j] >> 3));
                    }
                }
#pragma unroll
                for (int j = 0; j < MLC; ++j) {
                    if (lv[j] != (int)(e[j] & 7u) + 1) continue;
                    if ((unsigned)(sr[j] >> 32) == stamp && (long long)(unsigned)sr[j] < h) continue;
                    dm.cnt += 1; dm.cost += cost_of(e[j]);
                    dcm |= 1u << (b0 + j);
                }
            }
            CntCost dn_cta;
            const CntCost dex = block_exclusive_scan<CntCost, LT>(dm, dn_cta);
            if (tid == 0) w.dn_tot[c] = dn_cta;
            phase_barrier();
            unsigned long long dpre[1] = {0ull};
            for (int j = tid; j < c; j += LT) dpre[0] += ldcg_cc(w.dn_tot + j).cnt;
            cta_allreduce<LT, 1, 0>(dpre, flip);
            // ---- down-rank: the first h candidates form D -----------------------------------------
            double dD_mine = 0.0; unsigned long long freed_mine = 0; unsigned nD_mine = 0;
            long long run_cnt = (long long)dpre[0] + dex.cnt;
            for (unsigned m = dcm; m && run_cnt < h; m &= m - 1, ++run_cnt) {
                const int j = __ffs(m) - 1;
                const unsigned e = __ldg(dn_ent + t_lo + j);
                dsel |= 1u << j;
                dD_mine += __ldg(dn_de + t_lo + j); freed_mine += cost_of(e); nD_mine += 1;
            }
            {
                const double d = cta_sum<LT>(dD_mine);
                unsigned long long r2[2] = {freed_mine, nD_mine};
                cta_allreduce<LT, 2, 0>(r2, flip);
                if (tid == 0) { w.dD[c] = d; w.freed[c] = r2[0]; w.nD[c] = (unsigned)r2[1]; }
            }
            phase_barrier();
            // ---- U: up-candidates 0..h-1 whose cumulative cost fits slack + what D frees ------------
            unsigned long long fr[1] = {0ull};
            for (int j = tid; j < G; j += LT) fr[0] += __ldcg(w.freed + j);
            cta_allreduce<LT, 1, 0>(fr, flip);
            const long long lim_cost = slack + (long long)fr[0];
            if (cm && base_cnt < h) {
                unsigned long long run_cost = base_cost;
                long long rank = base_cnt;
                for (unsigned m = cm; m && rank < h; m &= m - 1, ++rank) {
                    const int j = __ffs(m) - 1;
                    run_cost += cost_of(__ldg(up_ent + t_lo + j));
                    if ((long long)run_cost > lim_cost) break;      // cumulative costs only grow
                    um |= 1u << j;
                    dU_mine += __ldg(up_de + t_lo + j); costU_mine = run_cost; nU_mine += 1;
                }
            }
            const double d = cta_sum<LT>(dU_mine);
            unsigned long long r2[2] = {costU_mine, nU_mine};
            cta_allreduce<LT, 2, 2 | (0 << 2)>(r2, flip);
            if (tid == 0) { w.dU[c] = d; w.costU[c] = r2[0]; w.nU[c] = (unsigned)r2[1]; }
            phase_barrier();
        }

        // ---- totals (same order in every CTA), decision, apply, replicated state update -----------
        // every thread fetches the totals of its CTAs at once (one L2 round trip, not one per CTA);
        // the sums over CTAs follow a fixed tree
        double dU = 0.0, dD = 0.0;
        unsigned long long tot[4] = {0ull, 0ull, 0ull, 0ull};       // costU (max), nU, freed, nD
        for (int j = tid; j < G; j += LT) {
            dU += __ldcg(w.dU + j);
            if (!expand) dD += __ldcg(w.dD + j);
            const unsigned long long cu = __ldcg(w.costU + j);
            if (cu > tot[0]) tot[0] = cu;
            tot[1] += __ldcg(w.nU + j);
            if (!expand) { tot[2] += __ldcg(w.freed + j); tot[3] += __ldcg(w.nD + j); }
        }
        cta_allreduce<LT, 4, 2 | (0 << 2) | (0 << 4) | (0 << 6)>(tot, flip);
        const unsigned long long costU = tot[0], freed = tot[2];
        const unsigned nU = (unsigned)tot[1], nD = (unsigned)tot[3];
        cta_sum2_all<LT>(dU, dD, flip2);
        const bool accept = expand ? (nU > 0) : (nU > 0 && nD > 0 && dU > dD);
        if (accept && !expand) {
            // the owner of a list entry knows the block and its new level: no loads
            for (unsigned m = um; m; m &= m - 1) {
                const unsigned e = __ldg(up_ent + t_lo + (__ffs(m) - 1));
                if (SB_IN_BOUNDS(a.ds, SBK_ALLOC, e >> 3, a.N)) a.level[e >> 3] = (unsigned char)((e & 7u) + 1u);
            }
            for (unsigned m = dsel; m; m &= m - 1) {
                const unsigned e = __ldg(dn_ent + t_lo + (__ffs(m) - 1));
                if (SB_IN_BOUNDS(a.ds, SBK_ALLOC, e >> 3, a.N)) a.level[e >> 3] = (unsigned char)(e & 7u);
            }
        }
        if (expand && accept) { used += (long long)costU; loss -= dU; expansions += 1; }
        else if (accept) { used += (long long)costU - (long long)freed; loss += dD - dU; accepted += 1; }
        else { k /= 2; rejected += 1; }
        iter += 1;
        if (!expand) phase_barrier();                     // the new levels are visible to the next up-count
    }
    if (c == 0 && tid == 0) {
        AllocState* st = a.st;
        st->k = k; st->used = used; st->loss = loss; st->iter = iter; st->accepted = accepted;
        st->rejected = rejected; st->expansions = expansions; st->done = 1; st->status = status;
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
    if (!SB_IN_BOUNDS(a.ds, SBK_ALLOC, i, a.N)) return;
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

// Everything of an allocation call in stream order, no host round trip (so the call can be part
// of a captured CUDA graph); the report goes to device memory.
static sb_status allocate_enqueue(sb_ctx* ctx, const float* err, int64_t N,
                                  const int64_t* block_elems, int64_t uniform_block_elems,
                                  const int* bits, int n_bits, double budget, int mode,
                                  double gamma0, double gammaT, uint8_t* level,
                                  sb_alloc_report* report_dev, bool own_report) {
    if (!ctx) return SB_ERR_INVALID;
    if (!err || !level || (!report_dev && !own_report) || N <= 0) return sb_fail(ctx, SB_ERR_INVALID, "allocate: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "allocate: bits must be ascending in 1..8");
    if (!block_elems && uniform_block_elems <= 0) return sb_fail(ctx, SB_ERR_INVALID, "allocate: block size");
    if (mode != SB_ALLOC_SCALEBITS && mode != SB_ALLOC_GREEDY) return sb_fail(ctx, SB_ERR_INVALID, "allocate: mode");
    if (mode == SB_ALLOC_SCALEBITS &&
        (!(gamma0 > 0.0) || !(gammaT > 0.0) || gamma0 > 1.0 || gammaT > 1.0))
        return sb_fail(ctx, SB_ERR_INVALID, "allocate: gamma0, gammaT must lie in (0, 1]");
    const int L = n_bits;
    const long long nsteps = (long long)N * (L - 1);
    if (nsteps >= (1ll << 32) || N >= (1ll << 29) - 1)
        return sb_fail(ctx, SB_ERR_SHAPE, "allocate: N must be below 2^29 and N * (n_bits - 1) below 2^32");
    int l0 = 0;
    if (mode == SB_ALLOC_SCALEBITS) {
        l0 = -1;
        for (int l = 0; l < L; ++l) if ((double)bits[l] <= budget) l0 = l;
        if (l0 < 0) return sb_fail(ctx, SB_ERR_BUDGET, "allocate: budget %.4f below the smallest candidate %d", budget, bits[0]);
    }
    SB_CUDA(ctx, cudaSetDevice(ctx->device));

    const int nblkB = (int)((N + BT - 1) / BT);
    const long long ntiles = (nsteps + ATILE - 1) / ATILE;
    const size_t nparts = (size_t)(nblkB > ntiles ? nblkB : ntiles) + 8;
    const size_t sort_bytes = sb_radix_sort_scratch_bytes(nsteps > 0 ? nsteps : 1);
    const size_t ns = (size_t)(nsteps > 0 ? nsteps : 1) + 1;
    void* arena;
    sb_status stt = sb_scratch(ctx, Carver::need({sizeof(AllocState), ns * 8, ns * 8, ns * 8, ns * 8,
                                                   ns * 4, ns * 4, ns * 4, ns * 4,
                                                   (size_t)N * 8, (size_t)N * 8, (size_t)N * 8,
                                                   (size_t)N * 4, nparts * 8,
                                                   nparts * 8, sort_bytes, (size_t)(N + 1) * 8,
                                                   (size_t)LOOP_MAX_CTAS * 128, sizeof(sb_alloc_report)}), &arena);
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
    unsigned long long* upsr = cv.take<unsigned long long>((size_t)N);
    unsigned long long* upcum = cv.take<unsigned long long>((size_t)N);
    double* upde = cv.take<double>((size_t)N);
    unsigned* mark = cv.take<unsigned>((size_t)N);
    double* part = cv.take<double>(nparts);
    double* part2 = cv.take<double>(nparts);
    void* sort_scratch = cv.take<unsigned char>(sort_bytes);
    unsigned long long* totals = cv.take<unsigned long long>((size_t)N + 1);
    CntCost* loop_cc = cv.take<CntCost>(2 * LOOP_MAX_CTAS);
    long long* loop_ll = cv.take<long long>(LOOP_MAX_CTAS);
    double* loop_d = cv.take<double>(2 * LOOP_MAX_CTAS);
    unsigned long long* loop_u64 = cv.take<unsigned long long>(2 * LOOP_MAX_CTAS);
    unsigned* loop_u32 = cv.take<unsigned>(2 * LOOP_MAX_CTAS);
    sb_alloc_report* own_rep = cv.take<sb_alloc_report>(1);
    if (own_report) report_dev = own_rep;

    // total weights -> cap.  Uniform blocks: closed form; else a device sum via the scan.
    const unsigned long long* total_dev = nullptr;
    if (block_elems) {
        stt = sb_scan_exclusive_u64(ctx, reinterpret_cast<const unsigned long long*>(block_elems), totals, N);
        if (stt != SB_OK) return stt;
        total_dev = totals + N;
    }

    AllocArgs a{};
    a.err = err; a.block_elems = reinterpret_cast<const long long*>(block_elems);
    a.uniform = uniform_block_elems; a.N = N; a.L = L;
    for (int l = 0; l < 8; ++l) a.bits[l] = l < L ? bits[l] : 0;
    a.level = level; a.st = dst; a.ds = ctx->dstate;
    a.upsr = upsr; a.upcum = upcum; a.upde = upde; a.mark = mark;
    a.part = part;

    init_state_kernel<<<1, 1, 0, ctx->stream>>>(dst, total_dev, (long long)N * uniform_block_elems, budget,
                                                gamma0, gammaT, (long long)N, mode == SB_ALLOC_SCALEBITS);
    SB_LAUNCHED(ctx);
    init_levels_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, l0, 1);
    SB_LAUNCHED(ctx);
    init_finish_kernel<<<1, 1, 0, ctx->stream>>>(a, nblkB);
    SB_LAUNCHED(ctx);

    const int* greedy_steps = nullptr;
    if (mode == SB_ALLOC_GREEDY) {
        // a lowest candidate that does not fit leaves no slack: no step is applied, and the
        // report kernel latches SB_ERR_BUDGET
        if (nsteps > 0) {
            int* level32 = reinterpret_cast<int*>(upsr);
            int* steps = reinterpret_cast<int*>(mark);
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
            greedy_steps = steps;
        }
        // recompute used / loss / histogram from the final levels
        SB_CUDA(ctx, cudaMemsetAsync(&dst->used, 0, sizeof(long long), ctx->stream));
        eval_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, part2, 1);
        SB_LAUNCHED(ctx);
    } else {
        if (nsteps > 0) {
            const unsigned g = (unsigned)((nsteps + 255) / 256);
            step_keys_kernel<<<g, 256, 0, ctx->stream>>>(a, kA, vA);
            SB_LAUNCHED(ctx);
            stt = sb_radix_sort_u64(ctx, kA, kB, vA, vB, nsteps, sort_scratch);
            if (stt != SB_OK) return stt;
            // down list = up list reversed run by run (vB: heads, vD: their prefix, kB: run starts);
            // the sorted keys in kA are dead after tie_heads_kernel and hold the down entries
            unsigned* run_start = reinterpret_cast<unsigned*>(kB);
            tie_heads_kernel<<<g, 256, 0, ctx->stream>>>(kA, nsteps, vB);
            SB_LAUNCHED(ctx);
            stt = sb_scan_exclusive_u32(ctx, vB, vD, nsteps);
            if (stt != SB_OK) return stt;
            run_starts_kernel<<<g, 256, 0, ctx->stream>>>(vB, vD, nsteps, run_start);
            SB_LAUNCHED(ctx);
            unsigned* up_ent = vC; unsigned* dn_ent = reinterpret_cast<unsigned*>(kA);
            double* up_de = reinterpret_cast<double*>(kC); double* dn_de = reinterpret_cast<double*>(kD);
            entry_info_kernel<<<g, 256, 0, ctx->stream>>>(a, vA, vB, vD, run_start, nsteps, up_ent, up_de,
                                                          dn_ent, dn_de);
            SB_LAUNCHED(ctx);
            LoopWork lw;
            lw.up_tot = loop_cc; lw.dn_tot = loop_cc + LOOP_MAX_CTAS;
            lw.up_first = loop_ll;
            lw.dD = loop_d; lw.dU = loop_d + LOOP_MAX_CTAS;
            lw.freed = loop_u64; lw.costU = loop_u64 + LOOP_MAX_CTAS;
            lw.nD = loop_u32; lw.nU = loop_u32 + LOOP_MAX_CTAS;
            const unsigned* up_ent_c = up_ent; const unsigned* dn_ent_c = dn_ent;
            const double* up_de_c = up_de; const double* dn_de_c = dn_de;
            long long ne = nsteps;
            void* kargs[] = {&a, &up_ent_c, &up_de_c, &dn_ent_c, &dn_de_c, &ne, &lw};
            bool launched = false;
            // Small problems: one thread-block cluster of 16 CTAs x 512 threads; its hardware
            // barrier is several times cheaper than a grid-wide one, and a handful of list
            // entries per thread is all the parallelism the passes need.
            if (nsteps <= (long long)CL_CTAS * CL_THREADS * 16) {
                auto kern = scalebits_loop_masked_kernel<CL_THREADS, true>;       // <= 16 entries per thread
                SB_FUNC_ATTR(ctx, kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(CL_CTAS);
                cfg.blockDim = dim3(CL_THREADS);
                cfg.stream = ctx->stream;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = CL_CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                cfg.attrs = at; cfg.numAttrs = 1;
                cudaError_t e = cudaLaunchKernelExC(&cfg, (const void*)kern, kargs);
                if (e == cudaSuccess) launched = true;
                else (void)cudaGetLastError();        // no room for such a cluster: use the grid form
            }
            if (!launched) {
                // the whole loop in one cooperative launch
                auto kern = scalebits_loop_kernel<GL_THREADS, false>;
                auto kern_masked = scalebits_loop_masked_kernel<GL_THREADS, false>;
                int occ = 0, occ_m = 0;
                SB_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, GL_THREADS, 0));
                SB_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_m, kern_masked, GL_THREADS, 0));
                auto grid_for = [&](int o) {
                    long long G = (long long)o * ctx->sm_count;
                    // a few list entries per thread: grid barriers cost more with more CTAs than
                    // the short passes gain
                    const long long want = (nsteps + LC * GL_THREADS - 1) / (LC * GL_THREADS);
                    if (G > want) G = want;
                    if (G > LOOP_MAX_CTAS) G = LOOP_MAX_CTAS;
                    if (G < 1) G = 1;
                    return G;
                };
                // the masked form needs at most 32 list entries per thread
                long long G = grid_for(occ_m);
                const long long per_cta = (nsteps + G - 1) / G;
                const bool masked = (per_cta + GL_THREADS - 1) / GL_THREADS <= 32;
                if (!masked) G = grid_for(occ);
                SB_CUDA(ctx, cudaLaunchCooperativeKernel(masked ? (const void*)kern_masked : (const void*)kern,
                                                         dim3((unsigned)G), dim3(GL_THREADS), kargs, 0,
                                                         ctx->stream));
            }
            ctx->launches++;
        }
        // single candidate (or finished): histogram of the final levels
        eval_kernel<<<nblkB, BT, 0, ctx->stream>>>(a, part2, 0);
        SB_LAUNCHED(ctx);
    }
    report_kernel<<<1, 1, 0, ctx->stream>>>(a, greedy_steps, mode == SB_ALLOC_GREEDY, report_dev);
    SB_LAUNCHED(ctx);
    if (own_report) {
        SB_CUDA(ctx, cudaMemcpyAsync(ctx->pinned, report_dev, sizeof(sb_alloc_report), cudaMemcpyDeviceToHost,
                                     ctx->stream));
    }
    return SB_OK;
}

extern "C" sb_status sb_allocate_bits_async(sb_ctx* ctx, const float* err, int64_t N,
                                            const int64_t* block_elems, int64_t uniform_block_elems,
                                            const int* bits, int n_bits, double budget, int mode,
                                            double gamma0, double gammaT, uint8_t* level,
                                            sb_alloc_report* report_dev) {
    if (ctx && !report_dev) return sb_fail(ctx, SB_ERR_INVALID, "allocate: null report");
    return allocate_enqueue(ctx, err, N, block_elems, uniform_block_elems, bits, n_bits, budget, mode,
                            gamma0, gammaT, level, report_dev, false);
}

extern "C" sb_status sb_allocate_bits(sb_ctx* ctx, const float* err, int64_t N,
                                      const int64_t* block_elems, int64_t uniform_block_elems,
                                      const int* bits, int n_bits, double budget, int mode,
                                      double gamma0, double gammaT, uint8_t* level,
                                      sb_alloc_report* report) {
    if (!ctx) return SB_ERR_INVALID;
    if (!report) return sb_fail(ctx, SB_ERR_INVALID, "allocate: null or empty");
    memset(report, 0, sizeof *report);
    sb_status stt = allocate_enqueue(ctx, err, N, block_elems, uniform_block_elems, bits, n_bits, budget, mode,
                                     gamma0, gammaT, level, nullptr, true);
    if (stt != SB_OK) return stt;
    SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    memcpy(report, ctx->pinned, sizeof *report);
    // device status (look-back timeouts, non-finite inputs latched earlier, a budget below the
    // smallest candidate in greedy mode, the iteration cap)
    return sb_sync(ctx);
}

// Hand-written device-wide primitives: exclusive scans (decoupled look-back) and a stable
// LSD radix sort of 64-bit keys with 32-bit payloads (8-bit digits: per-tile histogram,
// one scan over the digit-major histogram, stable scatter).
#include <cooperative_groups.h>

#include "lookback.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

template <typename T>
__global__ void __launch_bounds__(SCAN_THREADS)
scan_exclusive_kernel(const T* __restrict__ in, T* __restrict__ out, int64_t n, int write_total,
                      LookbackBuf lb, SbDeviceState* st) {
    const unsigned tile = lookback_tile_id(st);
    const int64_t base = (int64_t)tile * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    T v[SCAN_ITEMS];
    T sum = t_zero((T*)nullptr);
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        v[k] = (base + k < n) ? in[base + k] : t_zero((T*)nullptr);
        sum = t_add(sum, v[k]);
    }
    T tile_total;
    T ex = block_exclusive_scan<T, SCAN_THREADS>(sum, tile_total);
    const T prefix = lookback_prefix<T>(tile_total, tile, lb, st);
    T run = t_add(prefix, ex);
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        if (base + k < n) out[base + k] = run;
        run = t_add(run, v[k]);
    }
    if (write_total && tile == gridDim.x - 1 && threadIdx.x == SCAN_THREADS - 1) out[n] = run;
    lookback_finish(st, lb);
}

// ---- radix sort ---------------------------------------------------------------------------
// Stable LSD sort, 8-bit digits, "one sweep" per digit: the digit histograms of all passes come
// from one read of the keys; each pass then ranks its tile, publishes the tile's digit counts and
// resolves its global offsets by decoupled look-back over the earlier tiles' descriptors (one
// thread per digit), and scatters -- one launch per pass instead of histogram + scan + scatter.
constexpr int SORT_THREADS = 256;
constexpr int SORT_ITEMS = 8;                          // consecutive 32-item warp steps
constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;   // 2048 keys per CTA
constexpr int RADIX = 256;
constexpr int SORT_PASSES = 8;
constexpr unsigned OS_AGG = 1u << 30, OS_INC = 2u << 30, OS_MASK = (1u << 30) - 1u;

// ghist[pass][digit] += number of keys with that digit in that pass
__global__ void __launch_bounds__(SORT_THREADS)
radix_hist_all_kernel(const unsigned long long* __restrict__ keys, int64_t n, unsigned* __restrict__ ghist) {
    __shared__ unsigned h[SORT_PASSES][RADIX];
    for (int i = threadIdx.x; i < SORT_PASSES * RADIX; i += SORT_THREADS) (&h[0][0])[i] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * SORT_TILE;
    for (int k = 0; k < SORT_ITEMS; ++k) {
        const int64_t i = base + k * SORT_THREADS + threadIdx.x;
        if (i < n) {
            const unsigned long long key = keys[i];
#pragma unroll
            for (int p = 0; p < SORT_PASSES; ++p) atomicAdd(&h[p][(unsigned)(key >> (8 * p)) & 0xffu], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < SORT_PASSES * RADIX; i += SORT_THREADS) {
        const unsigned c = (&h[0][0])[i];
        if (c) atomicAdd(ghist + i, c);
    }
}

// gbase[pass][digit] = number of keys with a smaller digit in that pass (one CTA per pass)
__global__ void __launch_bounds__(RADIX)
radix_base_kernel(const unsigned* __restrict__ ghist, unsigned* __restrict__ gbase) {
    unsigned total;
    const unsigned v = ghist[blockIdx.x * RADIX + threadIdx.x];
    gbase[blockIdx.x * RADIX + threadIdx.x] = block_exclusive_scan<unsigned, RADIX>(v, total);
}

// One pass.  Warp w of the CTA owns the contiguous keys [w*256, (w+1)*256) of the tile and walks
// them 32 at a time; within a step equal digits are ranked by lane (__match_any_sync), across
// steps by a per-warp running count, across warps by a prefix over the warps' digit counts,
// across tiles by the look-back over desc[tile][digit] = flag | count.
__global__ void __launch_bounds__(SORT_THREADS)
onesweep_pass_kernel(const unsigned long long* __restrict__ keys_in, const unsigned* __restrict__ vals_in,
                     unsigned long long* __restrict__ keys_out, unsigned* __restrict__ vals_out,
                     int64_t n, int shift, const unsigned* __restrict__ gbase, unsigned* __restrict__ desc,
                     unsigned* __restrict__ ticket, SbDeviceState* st) {
    constexpr int WARPS = SORT_THREADS / 32;
    __shared__ unsigned cnt[WARPS][RADIX];          // running count per warp and digit
    __shared__ unsigned basepos[RADIX];
    __shared__ unsigned tile_sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) tile_sh = atomicAdd(ticket, 1u);
    for (int d = lane; d < RADIX; d += 32) cnt[warp][d] = 0;
    __syncthreads();
    const unsigned tile = tile_sh;
    const int64_t wbase = (int64_t)tile * SORT_TILE + (int64_t)warp * (32 * SORT_ITEMS);
    unsigned long long key[SORT_ITEMS];
    unsigned val[SORT_ITEMS], rank[SORT_ITEMS];
#pragma unroll
    for (int k = 0; k < SORT_ITEMS; ++k) {
        const int64_t i = wbase + k * 32 + lane;
        const bool ok = i < n;
        key[k] = ok ? keys_in[i] : 0ull;
        val[k] = ok ? vals_in[i] : 0u;
        const unsigned d = (unsigned)(key[k] >> shift) & 0xffu;
        // lanes past the end vote in a digit of their own (256) so they never disturb ranks
        const unsigned peers = __match_any_sync(0xffffffffu, ok ? d : 256u);
        const unsigned before = __popc(peers & ((1u << lane) - 1u));
        unsigned prior = 0;
        if (ok) prior = cnt[warp][d];
        __syncwarp();
        if (ok && before == 0) cnt[warp][d] = prior + __popc(peers);
        __syncwarp();
        rank[k] = prior + before;
    }
    __syncthreads();
    {
        // thread d: prefix over the warps, publish the tile's count, look back for the offset
        const int d = threadIdx.x;
        unsigned run = 0;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
            const unsigned c = cnt[w][d];
            cnt[w][d] = run;
            run += c;
        }
        unsigned* mine = desc + (size_t)tile * RADIX + d;
        unsigned excl = 0;
        if (tile == 0) {
            st_release_u32(mine, OS_INC | run);
        } else {
            st_release_u32(mine, OS_AGG | run);
            bool timed_out = false;
            for (int t = (int)tile - 1; t >= 0 && !timed_out; --t) {
                const unsigned* p = desc + (size_t)t * RADIX + d;
                unsigned v = ld_acquire_u32(p);
                unsigned long long t_start = 0;
                int spins = 0;
                while ((v & ~OS_MASK) == 0u) {
                    // bounded wait: a predecessor that never publishes must not hang the GPU
                    if ((++spins & 63) == 0) {
                        const unsigned long long now = lb_now_ns();
                        if (t_start == 0) t_start = now;
                        else if (now - t_start > LB_WAIT_NS) { timed_out = true; break; }
                    }
                    __nanosleep(64);
                    v = ld_acquire_u32(p);
                }
                if (timed_out) break;
                excl += v & OS_MASK;
                if (v & OS_INC) break;
            }
            if (timed_out) sb_latch(st, SB_ERR_TIMEOUT, SBK_SORT);
            st_release_u32(mine, OS_INC | ((excl + run) & OS_MASK));
        }
        basepos[d] = gbase[d] + excl;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SORT_ITEMS; ++k) {
        const int64_t i = wbase + k * 32 + lane;
        if (i < n) {
            const unsigned d = (unsigned)(key[k] >> shift) & 0xffu;
            const int64_t pos = (int64_t)basepos[d] + cnt[warp][d] + rank[k];
            if (SB_IN_BOUNDS(st, SBK_SORT, pos, n)) {
                keys_out[pos] = key[k];
                vals_out[pos] = val[k];
            }
        }
    }
}

}  // namespace

// Descriptors for `tiles` tiles.  Every look-back kernel leaves its flags zeroed, so the
// buffer is cleared only when it is (re)allocated.
LookbackBuf sb_lookback(sb_ctx* ctx, unsigned tiles, sb_status* st) {
    *st = SB_OK;
    if (tiles > ctx->lb_max_tiles) {
        unsigned want = 1u << 14;
        while (want < tiles) want <<= 1;
        // the outgrown buffer is retired, not freed: captured launches may still point at it
        void* fresh = nullptr;
        if (cudaMalloc(&fresh, (size_t)want * 36) != cudaSuccess) {
            (void)cudaGetLastError();
            *st = sb_fail(ctx, SB_ERR_SCRATCH, "look-back descriptors for %u tiles", want);
            return LookbackBuf{};
        }
        if (ctx->lb_mem) ctx->retired.push_back(ctx->lb_mem);
        ctx->lb_mem = fresh;
        ctx->lb_max_tiles = want;
        cudaMemsetAsync(ctx->lb_mem, 0, (size_t)ctx->lb_max_tiles * 36, ctx->stream);
    }
    LookbackBuf lb;
    unsigned char* p = static_cast<unsigned char*>(ctx->lb_mem);
    lb.agg = p;
    lb.inc = p + (size_t)ctx->lb_max_tiles * 16;
    lb.flags = reinterpret_cast<unsigned*>(p + (size_t)ctx->lb_max_tiles * 32);
    lb.max_tiles = ctx->lb_max_tiles;
    return lb;
}

// ---- small and medium inputs: the whole sort in ONE launch of one thread-block cluster ----------
// Up to CL_SORT_PER_CTA keys (with their payloads) per CTA live in shared memory, twice over; a
// cluster of up to 16 CTAs holds 65536 keys, CTA c the keys [c m, (c + 1) m) of the current order.
// The eight passes run back to back inside one launch instead of as eight launches with look-back
// chains that cost about 11 us each whatever n is.  Per pass: every warp counts the digits of its
// tiles of 32 consecutive keys into its own histogram (match_any: one leader per distinct digit
// of a tile adds the group's size); after a cluster barrier every CTA reads all CTAs' digit totals
// through distributed shared memory and derives, in the same order everywhere, the first output
// position of each of its warps per digit; the warps walk their tiles again in order, ranking
// inside a tile by the lanes below with the same digit, and store each key into the shared memory
// of the CTA that owns its output position.  Stable, like the large sort, so both give the same
// permutation.
constexpr int CL_SORT_PER_CTA = 4096;
constexpr int CL_SORT_MAX_CTAS = 16;
constexpr int CL_SORT_THREADS = 1024;
constexpr int CL_SORT_WARPS = CL_SORT_THREADS / 32;
constexpr int CL_SORT_SMEM = 2 * CL_SORT_PER_CTA * 8 + 2 * CL_SORT_PER_CTA * 4 + CL_SORT_WARPS * RADIX * 4 +
                             CL_SORT_WARPS * RADIX * 2 + 2 * RADIX * 4 + 256;

__global__ void __launch_bounds__(CL_SORT_THREADS, 1)
cluster_sort_kernel(unsigned long long* __restrict__ keys, unsigned* __restrict__ vals, int n, int m,
                    SbDeviceState* ds) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ unsigned long long cs_smem[];
    unsigned long long* kbase = cs_smem;                                          // two key buffers
    unsigned* vbase = reinterpret_cast<unsigned*>(cs_smem + 2 * CL_SORT_PER_CTA); // two payload buffers
    unsigned* wbase = vbase + 2 * CL_SORT_PER_CTA;                                // [warp][digit] next output position
    unsigned short* hist = reinterpret_cast<unsigned short*>(wbase + CL_SORT_WARPS * RADIX);   // [warp][digit] counts
    // [2][digit] this CTA's totals, alternating by pass: a skipped pass has no second barrier, so the
    // next pass must not write where a slower CTA may still be reading
    unsigned* ctot2 = reinterpret_cast<unsigned*>(hist + CL_SORT_WARPS * RADIX);
    unsigned* wtot = ctot2 + 2 * RADIX;                                                // [8] scan scratch
    const int G = (int)gridDim.x, c = (int)blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int lo = min(n, c * m), n_loc = min(n, lo + m) - lo;
    for (int i = tid; i < n_loc; i += CL_SORT_THREADS) { kbase[i] = keys[lo + i]; vbase[i] = vals[lo + i]; }
    const int tiles = (n_loc + 31) / 32;
    const int tpw = (tiles + CL_SORT_WARPS - 1) / CL_SORT_WARPS;
    const int tile_lo = min(tiles, warp * tpw), tile_hi = min(tiles, tile_lo + tpw);
    int cur = 0;
    for (int pass = 0; pass < SORT_PASSES; ++pass) {
        const int shift = 8 * pass;
        unsigned* ctot = ctot2 + (pass & 1) * RADIX;
        for (int i = tid; i < CL_SORT_WARPS * RADIX / 2; i += CL_SORT_THREADS)
            reinterpret_cast<unsigned*>(hist)[i] = 0u;
        __syncthreads();                                   // also: the load of the input is done
        const unsigned long long* kin = kbase + cur * CL_SORT_PER_CTA;
        unsigned short* myh = hist + warp * RADIX;
        // (1) digit counts of this warp's tiles
        for (int t = tile_lo; t < tile_hi; ++t) {
            const int i = t * 32 + lane;
            const bool live = i < n_loc;
            const unsigned d = live ? (unsigned)(kin[i] >> shift) & 255u : 256u + lane;     // dead lanes match nobody
            const unsigned peers = __match_any_sync(0xffffffffu, d);
            if (live && (peers & lt_mask) == 0u) myh[d] += (unsigned short)__popc(peers);
            __syncwarp();
        }
        __syncthreads();
        if (tid < RADIX) {
            unsigned t = 0;
            for (int w = 0; w < CL_SORT_WARPS; ++w) t += hist[w * RADIX + tid];
            ctot[tid] = t;
        }
        cluster.sync();                                    // every CTA's digit totals are published
        // (2) first output position of this CTA per digit: all keys with smaller digits, then the
        // lower CTAs' keys with this digit; then of each warp
        bool same_digit = false;                           // all keys share this pass's digit
        if (tid < RADIX) {
            // all remote loads first: they are independent, and one at a time each would cost a full
            // round trip through the cluster's shared-memory network
            unsigned v[CL_SORT_MAX_CTAS];
#pragma unroll
            for (int cc = 0; cc < CL_SORT_MAX_CTAS; ++cc)
                v[cc] = cc < G ? *cluster.map_shared_rank(ctot + tid, cc) : 0u;
            unsigned all = 0, before = 0;
#pragma unroll
            for (int cc = 0; cc < CL_SORT_MAX_CTAS; ++cc) {
                all += v[cc];
                if (cc < c) before += v[cc];
            }
            same_digit = all == (unsigned)n;
            unsigned incl = all;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += y;
            }
            if (lane == 31) wtot[warp] = incl;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            unsigned base = incl - all + before;
            for (int w = 0; w < warp; ++w) base += wtot[w];
            for (int w = 0; w < CL_SORT_WARPS; ++w) {
                wbase[w * RADIX + tid] = base;
                base += hist[w * RADIX + tid];
            }
        }
        // A pass in which every key has the same digit (the top bytes of keys of one sign and a
        // narrow range of magnitudes) moves nothing: every CTA sees that from the same totals and
        // skips the scatter and its barrier.
        if (__syncthreads_or(same_digit)) continue;
        // (3) stable scatter: tiles in order, lanes in order inside a group of equal digits; the
        // destination is the shared memory of the CTA that owns the output position
        const unsigned* vin = vbase + cur * CL_SORT_PER_CTA;
        unsigned long long* kout = kbase + (cur ^ 1) * CL_SORT_PER_CTA;
        unsigned* vout = vbase + (cur ^ 1) * CL_SORT_PER_CTA;
        unsigned* myb = wbase + warp * RADIX;
        for (int t = tile_lo; t < tile_hi; ++t) {
            const int i = t * 32 + lane;
            const bool live = i < n_loc;
            const unsigned long long key = live ? kin[i] : 0ull;
            const unsigned d = live ? (unsigned)(key >> shift) & 255u : 256u + lane;
            const unsigned peers = __match_any_sync(0xffffffffu, d);
            unsigned pos = 0;
            if (live) pos = myb[d] + __popc(peers & lt_mask);
            __syncwarp();
            if (live && (peers & lt_mask) == 0u) myb[d] += __popc(peers);
            __syncwarp();
            if (live) {
                const unsigned dest = pos / (unsigned)m, idx = pos - dest * (unsigned)m;
                if (SB_IN_BOUNDS(ds, SBK_SORT, pos, n)) {
                    *cluster.map_shared_rank(kout + idx, dest) = key;
                    *cluster.map_shared_rank(vout + idx, dest) = vin[i];
                }
            }
        }
        cur ^= 1;
        cluster.sync();                // every CTA has received its keys; counters and totals may be reused
    }
    // A skipped last pass ends with remote reads of the peers' digit totals and no barrier after
    // them: no CTA may exit (and give up its shared memory) while a peer can still be reading it.
    cluster.sync();
    for (int i = tid; i < n_loc; i += CL_SORT_THREADS) {
        keys[lo + i] = kbase[cur * CL_SORT_PER_CTA + i];
        vals[lo + i] = vbase[cur * CL_SORT_PER_CTA + i];
    }
}

template <typename T>
static sb_status scan_launch(sb_ctx* ctx, const T* in, T* out, int64_t n, int write_total) {
    if (n <= 0) {
        if (write_total) SB_CUDA(ctx, cudaMemsetAsync(out, 0, sizeof(T), ctx->stream));
        return SB_OK;
    }
    const unsigned tiles = (unsigned)((n + SCAN_TILE - 1) / SCAN_TILE);
    sb_status st;
    LookbackBuf lb = sb_lookback(ctx, tiles, &st);
    if (st != SB_OK) return st;
    scan_exclusive_kernel<T><<<tiles, SCAN_THREADS, 0, ctx->stream>>>(
        in, out, n, write_total, lb, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

sb_status sb_scan_exclusive_u32(sb_ctx* ctx, const unsigned* in, unsigned* out, int64_t n) {
    return scan_launch<unsigned>(ctx, in, out, n, 0);
}
sb_status sb_scan_exclusive_u64(sb_ctx* ctx, const unsigned long long* in, unsigned long long* out,
                                int64_t n) {
    return scan_launch<unsigned long long>(ctx, in, out, n, 1);
}

size_t sb_radix_sort_scratch_bytes(int64_t n) {
    const int64_t tiles = (n + SORT_TILE - 1) / SORT_TILE;
    // histograms, bases, tickets, then the per-pass tile descriptors
    return (size_t)(2 * SORT_PASSES * RADIX + 64) * sizeof(unsigned) +
           (size_t)SORT_PASSES * tiles * RADIX * sizeof(unsigned) + 1024;
}

sb_status sb_radix_sort_u64(sb_ctx* ctx, unsigned long long* keys, unsigned long long* keys_tmp,
                            unsigned* vals, unsigned* vals_tmp, int64_t n, void* scratch) {
    if (n <= 0) return SB_OK;
    if (n >= (1ll << 30)) return sb_fail(ctx, SB_ERR_SHAPE, "sort: more than 2^30 keys");
    if (n <= (int64_t)CL_SORT_PER_CTA * CL_SORT_MAX_CTAS) {
        // one launch of one cluster, everything in shared memory; sorted in place (the eight passes
        // of the large path also end in `keys` / `vals`).  If the cluster cannot be placed, the
        // large path below takes over.
        int G = 1;
        while ((int64_t)G * CL_SORT_PER_CTA < n) G *= 2;
        const int m = (int)((n + G - 1) / G);
        const void* kfn = reinterpret_cast<const void*>(cluster_sort_kernel);
        if (!ctx->configured.count(kfn)) {                 // two attributes, once per context
            SB_CUDA(ctx, cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, CL_SORT_SMEM));
            SB_CUDA(ctx, cudaFuncSetAttribute(kfn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
            ctx->configured.insert(kfn);
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(G);
        cfg.blockDim = dim3(CL_SORT_THREADS);
        cfg.dynamicSmemBytes = CL_SORT_SMEM;
        cfg.stream = ctx->stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = G; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int nn = (int)n;
        SbDeviceState* ds = ctx->dstate;
        void* kargs[] = {&keys, &vals, &nn, (void*)&m, &ds};
        if (cudaLaunchKernelExC(&cfg, kfn, kargs) == cudaSuccess) {
            SB_LAUNCHED(ctx);
            return SB_OK;
        }
        (void)cudaGetLastError();
    }
    const int tiles = (int)((n + SORT_TILE - 1) / SORT_TILE);
    Carver cv(scratch);
    unsigned* ghist = cv.take<unsigned>(SORT_PASSES * RADIX);
    unsigned* tickets = ghist + SORT_PASSES * RADIX;            // contiguous: one memset clears both
    cv.take<unsigned>(64);
    unsigned* gbase = cv.take<unsigned>(SORT_PASSES * RADIX);
    unsigned* desc = cv.take<unsigned>((size_t)SORT_PASSES * tiles * RADIX);
    SB_CUDA(ctx, cudaMemsetAsync(ghist, 0, (SORT_PASSES * RADIX + 64) * sizeof(unsigned), ctx->stream));
    SB_CUDA(ctx, cudaMemsetAsync(desc, 0, (size_t)SORT_PASSES * tiles * RADIX * sizeof(unsigned), ctx->stream));
    radix_hist_all_kernel<<<tiles, SORT_THREADS, 0, ctx->stream>>>(keys, n, ghist);
    SB_LAUNCHED(ctx);
    radix_base_kernel<<<SORT_PASSES, RADIX, 0, ctx->stream>>>(ghist, gbase);
    SB_LAUNCHED(ctx);
    unsigned long long* kin = keys; unsigned long long* kout = keys_tmp;
    unsigned* vin = vals; unsigned* vout = vals_tmp;
    for (int pass = 0; pass < SORT_PASSES; ++pass) {
        onesweep_pass_kernel<<<tiles, SORT_THREADS, 0, ctx->stream>>>(
            kin, vin, kout, vout, n, pass * 8, gbase + pass * RADIX, desc + (size_t)pass * tiles * RADIX,
            tickets + pass, ctx->dstate);
        SB_LAUNCHED(ctx);
        unsigned long long* tk = kin; kin = kout; kout = tk;
        unsigned* tv = vin; vin = vout; vout = tv;
    }
    return SB_OK;
}

// Device-wide prefix sums without CUB: single-pass chained scan with decoupled look-back.
// Every tile publishes its aggregate, then walks back over its predecessors' descriptors
// until it meets an inclusive prefix.  Tile ids come from an atomic ticket, so a tile's
// predecessors have always started; every wait is bounded and latches SB_ERR_TIMEOUT
// instead of spinning forever.
#pragma once
#include "common.cuh"

struct CntCost {                       // (how many selected before me, their summed cost)
    unsigned long long cost;
    unsigned cnt;
    unsigned pad;
};

struct LookbackBuf {                   // context-owned; all flags are zero between launches
    unsigned* flags;                   // [max_tiles]  0 = empty, 1 = aggregate, 2 = inclusive
    unsigned char* agg;                // [max_tiles] * 16 bytes
    unsigned char* inc;                // [max_tiles] * 16 bytes
    unsigned max_tiles;
};
LookbackBuf sb_lookback(sb_ctx* ctx, unsigned tiles, sb_status* st);

#ifdef __CUDACC__
constexpr unsigned LB_AGG = 1u, LB_INC = 2u;
constexpr unsigned long long LB_WAIT_NS = 250ull * 1000 * 1000;   // default: give up after 250 ms
__device__ __forceinline__ unsigned long long lb_now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned t_zero(unsigned*) { return 0u; }
__device__ __forceinline__ unsigned long long t_zero(unsigned long long*) { return 0ull; }
__device__ __forceinline__ CntCost t_zero(CntCost*) { return CntCost{0ull, 0u, 0u}; }
__device__ __forceinline__ unsigned t_add(unsigned a, unsigned b) { return a + b; }
__device__ __forceinline__ unsigned long long t_add(unsigned long long a, unsigned long long b) { return a + b; }
__device__ __forceinline__ CntCost t_add(CntCost a, CntCost b) { return CntCost{a.cost + b.cost, a.cnt + b.cnt, 0u}; }
__device__ __forceinline__ unsigned t_shfl_up(unsigned v, int d) { return __shfl_up_sync(0xffffffffu, v, d); }
__device__ __forceinline__ unsigned long long t_shfl_up(unsigned long long v, int d) { return __shfl_up_sync(0xffffffffu, v, d); }
__device__ __forceinline__ CntCost t_shfl_up(CntCost v, int d) {
    return CntCost{__shfl_up_sync(0xffffffffu, v.cost, d), __shfl_up_sync(0xffffffffu, v.cnt, d), 0u};
}
__device__ __forceinline__ unsigned t_shfl_xor(unsigned v, int d) { return __shfl_xor_sync(0xffffffffu, v, d); }
__device__ __forceinline__ unsigned long long t_shfl_xor(unsigned long long v, int d) { return __shfl_xor_sync(0xffffffffu, v, d); }
__device__ __forceinline__ CntCost t_shfl_xor(CntCost v, int d) {
    return CntCost{__shfl_xor_sync(0xffffffffu, v.cost, d), __shfl_xor_sync(0xffffffffu, v.cnt, d), 0u};
}

// exclusive scan of one value per thread across a CTA of NT threads (NT <= 1024);
// returns the exclusive prefix, block_total valid in every thread
template <typename T, int NT>
__device__ __forceinline__ T block_exclusive_scan(T v, T& block_total) {
    __shared__ T warp_tot[NT / 32];
    __shared__ T total_sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T o = t_shfl_up(inc, d);
        if (lane >= d) inc = t_add(inc, o);
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        T w = lane < NT / 32 ? warp_tot[lane] : t_zero((T*)nullptr);
        T winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            T o = t_shfl_up(winc, d);
            if (lane >= d) winc = t_add(winc, o);
        }
        // exclusive prefix of the warp totals (the shuffle is executed by the whole warp)
        T wex = t_shfl_up(winc, 1);
        if (lane == 0) wex = t_zero((T*)nullptr);
        if (lane < NT / 32) warp_tot[lane] = wex;
        if (lane == NT / 32 - 1) total_sh = winc;
    }
    __syncthreads();
    T ex = t_shfl_up(inc, 1);
    if (lane == 0) ex = t_zero((T*)nullptr);
    ex = t_add(ex, warp_tot[warp]);
    block_total = total_sh;
    __syncthreads();
    return ex;
}

// dynamic tile id (call from all threads of the CTA)
__device__ __forceinline__ unsigned lookback_tile_id(SbDeviceState* st) {
    __shared__ unsigned tile_sh;
    if (threadIdx.x == 0) {
        tile_sh = atomicAdd(&st->ticket, 1u);             // reset by lookback_finish
    }
    __syncthreads();
    return tile_sh;
}

// Call from all threads at the very end of a look-back kernel: the last CTA to get here clears
// the descriptors this launch used and the tile ticket, so the next launch (stream order)
// starts from zeroed flags.  No host-side state is involved: a captured launch can be replayed.
__device__ __forceinline__ void lookback_finish(SbDeviceState* st, LookbackBuf lb) {
    __shared__ bool last_sh;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_sh = atomicAdd(&st->pad, 1u) == gridDim.x - 1;
    __syncthreads();
    if (last_sh) {
        for (unsigned t = threadIdx.x; t < gridDim.x; t += blockDim.x) lb.flags[t] = 0u;
        if (threadIdx.x == 0) { st->pad = 0u; st->ticket = 0u; }
    }
}

// exclusive prefix of this tile's aggregate over all earlier tiles; call from all threads
template <typename T>
__device__ __forceinline__ T lookback_prefix(T aggregate, unsigned tile, LookbackBuf lb, SbDeviceState* st) {
    __shared__ T prefix_sh;
    T* aggs = reinterpret_cast<T*>(lb.agg);
    T* incs = reinterpret_cast<T*>(lb.inc);
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        // test hook (sb_debug_lookback): a muted tile behaves like a predecessor that never
        // publishes, so that its successors' bounded waits can be seen to run out
        const bool muted = tile == st->lb_mute_tile;
        if (tile == 0) {
            if (lane == 0) {
                incs[0] = aggregate;
                __threadfence();
                if (!muted) st_release_u32(lb.flags, LB_INC);
                prefix_sh = t_zero((T*)nullptr);
            }
        } else {
            if (lane == 0) {
                aggs[tile] = aggregate;
                __threadfence();
                if (!muted) st_release_u32(lb.flags + tile, LB_AGG);
            }
            const unsigned long long wait_ns = st->lb_wait_ns;
            T running = t_zero((T*)nullptr);
            int base = (int)tile - 1;
            bool timed_out = false;
            while (true) {
                const int t = base - lane;
                unsigned state = LB_INC;
                T v = t_zero((T*)nullptr);
                if (t >= 0) {
                    unsigned f = ld_acquire_u32(lb.flags + t);
                    unsigned long long t_start = 0;
                    int spins = 0;
                    while ((f & 3u) == 0u) {
                        // bounded wait: a predecessor that never publishes must not hang the GPU
                        if ((++spins & 63) == 0) {
                            const unsigned long long now = lb_now_ns();
                            if (t_start == 0) t_start = now;
                            else if (now - t_start > wait_ns) { timed_out = true; break; }
                        }
                        __nanosleep(64);
                        f = ld_acquire_u32(lb.flags + t);
                    }
                    state = timed_out ? LB_INC : (f & 3u);
                    if (!timed_out) v = (state == LB_INC) ? incs[t] : aggs[t];
                }
                const unsigned incmask = __ballot_sync(0xffffffffu, state == LB_INC);
                const int first = incmask ? __ffs(incmask) - 1 : 32;
                T c = (lane <= first) ? v : t_zero((T*)nullptr);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) c = t_add(c, t_shfl_xor(c, o));
                running = t_add(running, c);
                if (first < 32) break;
                base -= 32;
            }
            if (__any_sync(0xffffffffu, timed_out) && lane == 0) sb_latch(st, SB_ERR_TIMEOUT, SBK_SCAN);
            if (lane == 0) {
                incs[tile] = t_add(running, aggregate);
                __threadfence();
                if (!muted) st_release_u32(lb.flags + tile, LB_INC);
                prefix_sh = running;
            }
        }
    }
    __syncthreads();
    T p = prefix_sh;
    __syncthreads();
    return p;
}
#endif

// host-callable primitives (scan_sort.cu)
sb_status sb_scan_exclusive_u32(sb_ctx* ctx, const unsigned* in, unsigned* out, int64_t n);
// out has n + 1 entries (out[n] = total)
sb_status sb_scan_exclusive_u64(sb_ctx* ctx, const unsigned long long* in, unsigned long long* out, int64_t n);
// stable LSD radix sort of 64-bit keys with 32-bit payloads, ascending.  Buffers ping-pong;
// after an even number of 8-bit passes the result is back in keys / vals.
size_t sb_radix_sort_scratch_bytes(int64_t n);
sb_status sb_radix_sort_u64(sb_ctx* ctx, unsigned long long* keys, unsigned long long* keys_tmp,
                            unsigned* vals, unsigned* vals_tmp, int64_t n, void* scratch);

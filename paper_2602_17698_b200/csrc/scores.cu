// Block scores (Section 4.1: one precision per m x n block; Section 5 "Implementation":
// round-to-nearest uniform quantiser, groups along the input axis): for every block of the
// permuted matrix and every candidate bitwidth b_l,
//     E[i][l] = sum over the block of a_r c_j (W' - Q_{b_l}(W'))^2
// and the per-bit gain of each one-level step.  Every weight is read from HBM once for all
// candidates.
//
// Quantiser (asymmetric min-max, min-anchored): per (row, group) lo = min, range = max - min,
// t = (v - lo) * qmax / range, q = rint(t), v - vhat = (v - lo) - q * range / qmax.
//
// The matrix is cut into slabs of 16 rows x 128 columns (4 KB), numbered tile by tile, chunk
// column by chunk column, top to bottom, and dealt to the warps of a persistent grid (one CTA of
// 16 warps per SM) in contiguous, equally long ranges.  Every warp is autonomous:
//
//   * it stages its own slabs in its own shared-memory ring, one TMA tile load per slab issued by
//     lane 0 into the slot it has just finished reading, a ring's depth ahead; the only
//     synchronisation is the slot's mbarrier, on which the load counts its bytes;
//   * when a slab has landed the warp first reduces every (row, group) to its min and max (exact
//     bf16 min/max; all 8 rows of a lane at once in a transposed butterfly, so a slab costs 8
//     shuffles) and leaves one small record per (row, group) beside the slab: -lo and, when the
//     group is the whole chunk, the ready-made packed constants of every candidate;
//   * then a lane owns 8 consecutive columns and RPL rows per step, unpacks its weights from the
//     slab, centres them with the record and evaluates all candidates from registers in packed
//     fp32 pairs (fma/add.f32x2): four instructions per pair and candidate (FMA to round with
//     the 1.5 * 2^23 constant, subtract it, FMA for the residual, FMA to accumulate).  c_j
//     multiplies the per-column accumulators once per stretch of a chunk column, not once per
//     element.
//
// The kernel is bound by the instruction issue of the SM sub-partitions (a packed instruction
// occupies the FP32 pipe for two cycles, everything else takes a cycle of its own), so the design
// minimises instructions per weight: no per-step control flow (a slab is four unrolled steps), no
// address arithmetic in the loop (shared-memory offsets are immediates), per-row constants loaded
// as packed pairs instead of being rebuilt in registers.  Every wait is bounded: on a time-out the
// warp latches SB_ERR_TIMEOUT, waits (bounded) for its own loads in flight and leaves.
//
// When a warp leaves a chunk column (or its range ends) it writes the partial block errors
// of that stretch as record (chunk number + warp number) -- unique, because either number only
// grows along the slab sequence -- and a second tiny kernel adds the records of a block in order
// (deterministic, no float atomics).
//
// NFINE = how many of the L candidates (the last ones: bits ascend) keep the grid step as a
// two-float sum: with many levels q * scale carries the fp32 rounding of the step times q, a
// bias shared by the whole group; the residual range - scale * qmax is exact in one FMA.
// A row weight a_r multiplies the squared residual itself (one more multiply per pair and
// candidate in the weighted instances): scaling v - lo by sqrt(a_r) instead would round an
// otherwise exact difference and cost two digits of accuracy at 8 bits.
#include <cuda.h>

#include "common.cuh"
#include "quant_common.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int SLAB_ROWS = 16;
constexpr int SLAB_BYTES = SLAB_ROWS * 256;
constexpr int SC_THREADS = 512;                 // one CTA of 16 warps per SM
constexpr int SC_WARPS = SC_THREADS / 32;
constexpr int SC_STREAMS = SC_WARPS;             // every warp walks its own range of slabs
constexpr int MAX_RING = 6;                     // slab slots per stream: as many as shared memory holds
constexpr int SC_SMEM_MAX = 227 * 1024;
constexpr int SC_CPL = 8;                       // columns per lane
constexpr int SC_NW = SC_CPL / 2;               // packed pairs per lane and row
constexpr int SC_BAR_BYTES = 2048;              // barriers + abort flag at the head of shared memory
constexpr unsigned long long SC_WAIT_NS = 2000ull * 1000 * 1000;   // a wait gives up after 2 s
static_assert(SC_STREAMS * MAX_RING * 8 + 8 <= SC_BAR_BYTES, "barrier block");

struct ScoreGeom {
    int br, bc, group;
    int chunks, tile_w, spb;       // 128-column chunks per tile; tile width; slabs per chunk column
    int nsub, lanes_per_sub;       // blocks side by side in a chunk (bc < 128); lanes across one block
    int gpc, rec_bytes;            // groups per 128-column chunk; bytes of one slab's records
    int ring;                      // slab slots per stream
    int n_rows, n_cols;            // rows / columns of the matrix (the last slab / chunk may reach past them)
    unsigned n_tile_cols, n_slabs, n_warps;   // n_warps = warps of the grid
};

struct ScoreArgs {
    const int32_t* c_perm;           // original column of permuted j
    const float* col_moment;
    BitsArg ba;
    float* rec;                      // scores: partial block errors; statistics: partial column sums
    float* rowpart;                  // statistics: [strip][row] partial row sums
    SbDeviceState* ds;               // status word; sizes of the two buffers in floats (checked build)
    long long rec_limit, rowpart_limit;
};

// owner of slab s when stream w takes slabs [n_slabs * w / n_warps, n_slabs * (w + 1) / n_warps)
__device__ __forceinline__ unsigned slab_owner(unsigned s, unsigned n_slabs, unsigned n_warps) {
    return (unsigned)((((unsigned long long)s + 1ull) * n_warps - 1ull) / n_slabs);
}
// streams between two owners may have an empty range (more streams than slabs): they write no record
__device__ __forceinline__ bool slab_range_empty(unsigned w, unsigned n_slabs, unsigned n_warps) {
    return (unsigned long long)n_slabs * w / n_warps == (unsigned long long)n_slabs * (w + 1) / n_warps;
}

struct SlabCursor { int sl, ch; unsigned bx, by; };

__device__ __forceinline__ SlabCursor cursor_at(unsigned s, const ScoreGeom& g) {
    SlabCursor c;
    const unsigned q = s / (unsigned)g.spb;
    c.sl = (int)(s - q * (unsigned)g.spb);
    const unsigned t = q / (unsigned)g.chunks;
    c.ch = (int)(q - t * (unsigned)g.chunks);
    c.by = t / g.n_tile_cols;
    c.bx = t - c.by * g.n_tile_cols;
    return c;
}
__device__ __forceinline__ void advance(SlabCursor& c, const ScoreGeom& g) {
    if (++c.sl == g.spb) {
        c.sl = 0;
        if (++c.ch == g.chunks) {
            c.ch = 0;
            if (++c.bx == g.n_tile_cols) { c.bx = 0; ++c.by; }
        }
    }
}

// ---- mbarriers in shared memory ------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// one TMA tile load (16 rows x 128 columns of the weight matrix, 4 KB, rows 256 bytes apart in
// shared memory); the bytes are counted on the mbarrier.  No multicast: a slab is read by one CTA.
__device__ __forceinline__ void tma_load_slab(unsigned dst, const CUtensorMap* map, int col, int row, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(col), "r"(row)
        : "memory");
}
__device__ __forceinline__ bool mbar_test(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.acquire.cta.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// waits in hardware (the warp is suspended, it issues nothing) until the phase completes or about
// `hint_ns` have passed
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity, unsigned hint_ns = 4000u) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cta.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// bounded wait: false (and the abort flag raised) if the phase does not complete in time or
// another warp has already given up
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 15u) == 15u) {
            const unsigned long long now = now_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > SC_WAIT_NS) { *abort_flag = 1; return false; }
        }
    }
}

// explicit shared-space loads and stores (32-bit shared addresses: no generic-address translation)
__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void lds128_pairs(unsigned addr, f32x2& a, f32x2& b) {
    asm volatile("ld.shared.v2.u64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr));
}
__device__ __forceinline__ f32x2 lds64(unsigned addr) {
    f32x2 v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds128f(unsigned addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// Records of a slab when the group is the whole 128-column chunk, no row weights and at most four
// candidates (PRE): per row, ready-made packed pairs
//   +0            (-lo, -lo)
//   +16 + 16 l    (qmax_l / range, same), (-range / qmax_l, same)        l < L
//   +16 + 16 L + 8 f   -(residual of the grid step) / qmax, twice         f < NFINE (the last candidates)
// Otherwise (general form): one float4 (-lo, 1 / range, range, a_r) per (row, group).
__host__ __device__ constexpr int pre_stride(int L, int nfine) { return 16 + 16 * L + 16 * ((nfine + 1) / 2); }
__host__ __device__ constexpr bool use_pre(int L, bool fullg) { return fullg && L <= 4; }

// the "landed" barrier of a ring slot
__device__ __forceinline__ unsigned bar_addr(unsigned bars, int stream, int slot) {
    return bars + (unsigned)((stream * MAX_RING + slot) * 8);
}

// ---- (row, group) ranges of one staged slab -> records ---------------------------------------
__device__ __forceinline__ void sts128(unsigned addr, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void sts64(unsigned addr, float x, float y) {
    asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}

// (min, -max) of a lane's 8 columns of one row as a bf16 pair in one register: its lanewise
// minimum over the lanes of a group is (group min, -group max).  Exact: bf16 min/max.
__device__ __forceinline__ uint32_t lane_minmax(const uint4 x) {
    const __nv_bfloat162 mn = __hmin2(__hmin2(b162(x.x), b162(x.y)), __hmin2(b162(x.z), b162(x.w)));
    const __nv_bfloat162 mx = __hmax2(__hmax2(b162(x.x), b162(x.y)), __hmax2(b162(x.z), b162(x.w)));
    const uint32_t mnu = u32(mn), nmx = u32(mx) ^ 0x80008000u;          // -max of the even / odd columns
    // (min even, -max even) against (min odd, -max odd)
    return u32(__hmin2(b162(__byte_perm(mnu, nmx, 0x5410)), b162(__byte_perm(mnu, nmx, 0x7632))));
}

struct GroupRange { float nlo, rinv, rng; };
__device__ __forceinline__ GroupRange range_of(uint32_t p) {
    const float lo = bf16lo(p), hi = -bf16hi(p);
    const float range = hi - lo;
    const bool live = range >= MIN_RANGE;
    GroupRange r;
    r.nlo = -lo;
    r.rinv = live ? rcp_approx(range) : 0.f;
    r.rng = live ? range : 0.f;
    return r;
}

// the PRE record of one row: -lo and the packed constants of the candidates [l0, l1)
template <int L, int NFINE>
__device__ __forceinline__ void pre_record(unsigned dst, const GroupRange& r, const BitsArg& ba, bool with_lo,
                                           int l0, int l1) {
    if (with_lo) sts64(dst, r.nlo, r.nlo);
#pragma unroll
    for (int l = 0; l < L; ++l) {
        if (l >= l0 && l < l1) {
            const float inv = ba.qmax[l] * r.rinv;
            const float ns = -ba.inv_qmax[l] * r.rng;                 // -(range / qmax)
            sts128(dst + 16 + 16 * l, inv, inv, ns, ns);
            if (l >= L - NFINE) {
                const float nslo = fmaf(ns, ba.qmax[l], r.rng) * -ba.inv_qmax[l];   // -(residual / qmax)
                sts64(dst + 16 + 16 * L + 8 * (l - (L - NFINE)), nslo, nslo);
            }
        }
    }
}

// A full slab (shared-memory addresses): a lane (cl, slot2) holds 8 columns of the 8 rows
// slot2 + 2 i.  The group reduction runs over the `team` lanes of a group for all 8 rows at once,
// transposed: at every level a lane hands half of its rows to its partner and keeps the other
// half, so the 8 rows cost 4 + 2 + 1 (+ 1) shuffles instead of 8 per level, and the lane that ends
// up with a row's range is the one that writes its record.  After the levels a lane of index t
// inside its team holds the rows (t >> (log2 team - h)) * n + k, k < n = 8 >> h, h = min(3, log2 team)
// halving levels.
template <int L, int NFINE, bool FULLG, bool ROWW>
__device__ __forceinline__ void slab_records(unsigned slab, unsigned rec, int row0, const ScoreGeom& g,
                                             const BitsArg& ba, int team, int cl, int slot2,
                                             const int32_t* __restrict__ a_perm,
                                             const float* __restrict__ row_weight) {
    uint32_t v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = lane_minmax(lds128(slab + (slot2 + 2 * i) * 256 + cl * 16));
    if (FULLG) team = 16;
    const int t = cl & (team - 1);
#pragma unroll
    for (int k = 0; k < 4; ++k) {                 // level k: partner at distance team >> (k + 1)
        const int o = team >> (k + 1);
        if (o > 0) {                              // (the same for the whole warp)
            if (k < 3) {
                constexpr int H[3] = {4, 2, 1};   // rows kept at this level
                const int h = H[k];
                const bool up = (t & o) != 0;     // this lane keeps the upper half of its rows
                uint32_t got[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (i < h) got[i] = __shfl_xor_sync(0xffffffffu, up ? v[i] : v[i + h], o);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (i < h) v[i] = u32(__hmin2(b162(up ? v[i + h] : v[i]), b162(got[i])));
            } else {
                v[0] = u32(__hmin2(b162(v[0]), b162(__shfl_xor_sync(0xffffffffu, v[0], o))));
            }
        }
    }
    if (use_pre(L, FULLG)) {
        // team = 16: lanes t and t ^ 1 both hold row t >> 1 and share the work: the even lane writes
        // -lo and the first candidates, the odd one the other candidates
        constexpr int LH = (L + 1) / 2;
        const int rr = slot2 + 2 * (t >> 1);
        const bool odd = (t & 1) != 0;
        pre_record<L, NFINE>(rec + rr * pre_stride(L, NFINE), range_of(v[0]), ba, !odd, odd ? LH : 0, odd ? L : LH);
    } else if (FULLG) {
        // 32 bytes per row, every value twice (packed pairs): -lo, 1/range | range
        const int rr = slot2 + 2 * (t >> 1);
        const GroupRange r = range_of(v[0]);
        if (t & 1) sts128(rec + rr * 32 + 16, r.rng, r.rng, 1.f, 1.f);
        else sts128(rec + rr * 32, r.nlo, r.nlo, r.rinv, r.rinv);
    } else {
        // n rows per lane (team 2: 4, team 4: 2, team 8 and 16: 1; with 16 the odd lane has a copy)
        const int lg = team == 16 ? 4 : team == 8 ? 3 : team == 4 ? 2 : 1;
        const int h = lg < 3 ? lg : 3;
        const int nn = 8 >> h;
        const int first = (t >> (lg - h)) * nn;
        const int grp = cl / team;
        if (team < 16 || (t & 1) == 0) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (k < nn) {
                    const int rr = slot2 + 2 * (first + k);
                    const GroupRange r = range_of(v[k]);
                    float ar = 1.f;
                    if (ROWW) {
                        const int row = row0 + rr;
                        ar = row < g.n_rows ? row_weight[a_perm ? a_perm[row] : row] : 0.f;
                    }
                    sts128(rec + (rr * g.gpc + grp) * 16, r.nlo, r.rinv, r.rng, ar);
                }
            }
        }
    }
}

// A slab at the bottom of a block whose height is not a multiple of 16: row by row.
template <int L, int NFINE, bool FULLG, bool ROWW>
__device__ __forceinline__ void slab_records_ragged(unsigned slab, unsigned rec, int rows_here, int row0,
                                                    const ScoreGeom& g, const BitsArg& ba, int team, int cl,
                                                    int slot2, const int32_t* __restrict__ a_perm,
                                                    const float* __restrict__ row_weight) {
    for (int rr = slot2; rr < rows_here; rr += 2) {
        uint32_t p = lane_minmax(lds128(slab + rr * 256 + cl * 16));
        for (int o = team >> 1; o > 0; o >>= 1)
            p = u32(__hmin2(b162(p), b162(__shfl_xor_sync(0xffffffffu, p, o))));
        const GroupRange r = range_of(p);
        float ar = 1.f;
        if (ROWW) {
            const int row = row0 + rr;
            ar = row < g.n_rows ? row_weight[a_perm ? a_perm[row] : row] : 0.f;
        }
        if (use_pre(L, FULLG)) {
            if (cl == 0) pre_record<L, NFINE>(rec + rr * pre_stride(L, NFINE), r, ba, true, 0, L);
        } else if (FULLG) {
            if (cl == 0) {
                sts128(rec + rr * 32, r.nlo, r.nlo, r.rinv, r.rinv);
                sts128(rec + rr * 32 + 16, r.rng, r.rng, 1.f, 1.f);
            }
        } else if ((cl & (team - 1)) == 0) {
            sts128(rec + (rr * g.gpc + cl / team) * 16, r.nlo, r.rinv, r.rng, ar);
        }
    }
}

// ---- all candidates from registers, per-column accumulators ---------------------------------
template <int L_, int RPL_, int NFINE_, bool FULLG_, bool ROWW_>
struct Scorer {
    static constexpr int L = L_, RPL = RPL_, NFINE = NFINE_;
    static constexpr bool FULLG = FULLG_, ROWW = ROWW_;
    static constexpr bool FULL_SLABS = false;      // a block's height need not be a multiple of 16
    __device__ __forceinline__ void begin_column(int) {}
    __device__ __forceinline__ void slab_done(int, unsigned) {}
    const ScoreArgs& a;
    const ScoreGeom& g;
    const unsigned gs;             // warp number in the grid
    const int cl, slot2;
    f32x2 acc[SC_NW][L];
    __device__ __forceinline__ Scorer(const ScoreArgs& a_, const ScoreGeom& g_, unsigned gs_, int cl_, int slot_)
        : a(a_), g(g_), gs(gs_), cl(cl_), slot2(slot_) {
#pragma unroll
        for (int k = 0; k < SC_NW; ++k)
#pragma unroll
            for (int l = 0; l < L; ++l) acc[k][l] = 0ull;
    }
    static constexpr bool PRE = use_pre(L, FULLG);
    // v - lo of the lane's 8 weights of one row, exact: both are bf16 values of one group
    __device__ __forceinline__ void centre(const uint4 x, const f32x2 nlo2, f32x2 (&vm)[SC_NW]) {
        const uint32_t w[SC_NW] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) {
            // low half through the byte permuter: a shift would take a slot of the FP32 pipe
            const float v0 = __uint_as_float(__byte_perm(w[k], 0u, 0x1044));
            vm[k] = add2(pk2(v0, bf16hi(w[k])), nlo2);
        }
    }
    // one candidate on the lane's 8 weights of one row
    template <bool FINE>
    __device__ __forceinline__ void candidate(int l, const f32x2 (&vm)[SC_NW], const f32x2 inv2, const f32x2 ns2,
                                              const f32x2 nslo2, const f32x2 ar2) {
        const f32x2 magic2 = pk2(RNE_MAGIC, RNE_MAGIC), nmagic2 = pk2(-RNE_MAGIC, -RNE_MAGIC);
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) {
            const f32x2 qq = add2(fma2(vm[k], inv2, magic2), nmagic2);
            const f32x2 e = FINE ? fma2(qq, nslo2, fma2(qq, ns2, vm[k])) : fma2(qq, ns2, vm[k]);
            acc[k][l] = fma2(ROWW ? mul2(e, ar2) : e, e, acc[k][l]);
        }
    }
    // one step (2 * RPL rows of the slab, RPL of them this lane's); lane_slab / lane_rec are the
    // shared-memory addresses of the lane's columns of row slot2 and of that row's (group's) record
    __device__ __forceinline__ void step(unsigned lane_slab, unsigned lane_rec, int rec_pitch, int r0) {
        uint4 x[RPL];
#pragma unroll
        for (int i = 0; i < RPL; ++i) x[i] = lds128(lane_slab + (r0 + 2 * i) * 256);
        if (PRE) {
            constexpr int STRIDE = pre_stride(L, NFINE);
#pragma unroll
            for (int i = 0; i < RPL; ++i) {
                const unsigned rec = lane_rec + (r0 + 2 * i) * STRIDE;
                f32x2 vm[SC_NW];
                centre(x[i], lds64(rec), vm);
#pragma unroll
                for (int l = 0; l < L; ++l) {
                    f32x2 inv2, ns2;
                    lds128_pairs(rec + 16 + 16 * l, inv2, ns2);
                    if (l >= L - NFINE) candidate<true>(l, vm, inv2, ns2, lds64(rec + 16 + 16 * L + 8 * (l - (L - NFINE))), 0ull);
                    else candidate<false>(l, vm, inv2, ns2, 0ull, 0ull);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < RPL; ++i) {
                f32x2 nlo2, rinv2, range2, ar2 = 0ull;
                if (FULLG) {
                    lds128_pairs(lane_rec + (r0 + 2 * i) * 32, nlo2, rinv2);
                    range2 = lds64(lane_rec + (r0 + 2 * i) * 32 + 16);
                } else {
                    const float4 r = lds128f(lane_rec + (r0 + 2 * i) * rec_pitch);
                    nlo2 = pk2(r.x, r.x); rinv2 = pk2(r.y, r.y); range2 = pk2(r.z, r.z); ar2 = pk2(r.w, r.w);
                }
                f32x2 vm[SC_NW];
                centre(x[i], nlo2, vm);
#pragma unroll
                for (int l = 0; l < L; ++l) {
                    const f32x2 q2 = *reinterpret_cast<const f32x2*>(&a.ba.q2[l]);
                    const f32x2 niq2 = *reinterpret_cast<const f32x2*>(&a.ba.niq2[l]);
                    const f32x2 inv2 = mul2(q2, rinv2);
                    const f32x2 ns2 = mul2(niq2, range2);                   // -(range / qmax)
                    if (l >= L - NFINE) candidate<true>(l, vm, inv2, ns2, mul2(fma2(ns2, q2, range2), niq2), ar2);
                    else candidate<false>(l, vm, inv2, ns2, 0ull, ar2);
                }
            }
        }
    }
    // column factors, lanes of the same block, record (chunk number + warp number)
    __device__ __forceinline__ void flush(unsigned q, int col0) {
        const int col = col0 + cl * SC_CPL;
        f32x2 c2[SC_NW];
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) {
            const int j = col + 2 * k;
            c2[k] = pk2(__ldg(a.col_moment + (a.c_perm ? a.c_perm[j] : j)),
                        __ldg(a.col_moment + (a.c_perm ? a.c_perm[j + 1] : j + 1)));
        }
        float tot[L];
#pragma unroll
        for (int l = 0; l < L; ++l) {
            f32x2 t2 = 0ull;
#pragma unroll
            for (int k = 0; k < SC_NW; ++k) { t2 = fma2(c2[k], acc[k][l], t2); acc[k][l] = 0ull; }
            float a0, a1;
            upk2(t2, a0, a1);
            float v = a0 + a1;
            for (int o = g.lanes_per_sub >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            tot[l] = v;
        }
        if (slot2 == 0 && (cl % g.lanes_per_sub) == 0 &&
            SB_IN_BOUNDS(a.ds, SBK_SCORES, ((long long)(q + gs) * g.nsub + cl / g.lanes_per_sub) * L + L - 1, a.rec_limit)) {
            float* dst = a.rec + ((size_t)(q + gs) * g.nsub + cl / g.lanes_per_sub) * L;
#pragma unroll
            for (int l = 0; l < L; ++l) dst[l] = tot[l];
        }
    }
};

// ---- reorder statistics on the same walk (Section 4.1: per-channel aggregates of the element
// sensitivities a_r c_j (W - Q(W))^2 at the warm-start precision, on the ORIGINAL layout) ----------
// One candidate.  The matrix is one block row as tall as the matrix, so a chunk column is a strip of
// 128 columns from top to bottom.  Column sums: per-column accumulators over the warp's stretch of a
// strip, written as a record of 128 partial sums at its end (c_j applied there).  Row sums: a lane's
// 8 rows of a slab each get sum_j c_j e^2 over the lane's 8 columns; the 16 lanes of a row are reduced
// for all 8 rows at once by the same transposed butterfly as the ranges, and the lane that ends up with
// a row writes rowpart[strip][row].  A second kernel adds the partials in a fixed order: no float
// atomics, reruns are bit-identical.
template <int NFINE_, bool FULLG_, bool ROWW_>
struct StatsScorer {
    static constexpr int L = 1, RPL = 2, NFINE = NFINE_;
    static constexpr bool FULLG = FULLG_, ROWW = ROWW_;
    static constexpr bool PRE = use_pre(1, FULLG);
    static constexpr bool FULL_SLABS = true;       // the strip is padded to whole slabs (zero rows add nothing)
    const ScoreArgs& a;
    const ScoreGeom& g;
    const unsigned gs;
    const int cl, slot2;
    f32x2 colacc[SC_NW], c2[SC_NW];
    float rowsum[8];
    __device__ __forceinline__ StatsScorer(const ScoreArgs& a_, const ScoreGeom& g_, unsigned gs_, int cl_, int slot_)
        : a(a_), g(g_), gs(gs_), cl(cl_), slot2(slot_) {
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) colacc[k] = c2[k] = 0ull;
    }
    // column factors of the lane's 8 columns of the strip that starts at column col0
    __device__ __forceinline__ void begin_column(int col0) {
        const int col = col0 + cl * SC_CPL;
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) {
            const int j = col + 2 * k;
            c2[k] = pk2(j < g.n_cols ? __ldg(a.col_moment + j) : 0.f, j + 1 < g.n_cols ? __ldg(a.col_moment + j + 1) : 0.f);
        }
    }
    __device__ __forceinline__ void step(unsigned lane_slab, unsigned lane_rec, int rec_pitch, int r0) {
        const f32x2 magic2 = pk2(RNE_MAGIC, RNE_MAGIC), nmagic2 = pk2(-RNE_MAGIC, -RNE_MAGIC);
        uint4 x[RPL];
#pragma unroll
        for (int i = 0; i < RPL; ++i) x[i] = lds128(lane_slab + (r0 + 2 * i) * 256);
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            f32x2 nlo2, inv2, ns2, nslo2 = 0ull, ar2 = 0ull;
            if (PRE) {
                const unsigned rec = lane_rec + (r0 + 2 * i) * pre_stride(1, NFINE);
                nlo2 = lds64(rec);
                lds128_pairs(rec + 16, inv2, ns2);
                if (NFINE) nslo2 = lds64(rec + 32);
            } else {
                const float4 r = lds128f(lane_rec + (r0 + 2 * i) * rec_pitch);
                const f32x2 q2 = *reinterpret_cast<const f32x2*>(&a.ba.q2[0]);
                const f32x2 niq2 = *reinterpret_cast<const f32x2*>(&a.ba.niq2[0]);
                const f32x2 range2 = pk2(r.z, r.z);
                nlo2 = pk2(r.x, r.x);
                inv2 = mul2(q2, pk2(r.y, r.y));
                ns2 = mul2(niq2, range2);
                if (NFINE) nslo2 = mul2(fma2(ns2, q2, range2), niq2);
                ar2 = pk2(r.w, r.w);
            }
            const uint32_t w[SC_NW] = {x[i].x, x[i].y, x[i].z, x[i].w};
            f32x2 rs2 = 0ull;
#pragma unroll
            for (int k = 0; k < SC_NW; ++k) {
                const float v0 = __uint_as_float(__byte_perm(w[k], 0u, 0x1044));
                const f32x2 vm = add2(pk2(v0, bf16hi(w[k])), nlo2);
                const f32x2 qq = add2(fma2(vm, inv2, magic2), nmagic2);
                const f32x2 e = NFINE ? fma2(qq, nslo2, fma2(qq, ns2, vm)) : fma2(qq, ns2, vm);
                const f32x2 ea = ROWW ? mul2(e, ar2) : e;
                colacc[k] = fma2(ea, e, colacc[k]);
                rs2 = fma2(mul2(ea, c2[k]), e, rs2);
            }
            float s0, s1;
            upk2(rs2, s0, s1);
            rowsum[(r0 >> 1) + i] = s0 + s1;             // r0 is a compile-time constant in the unrolled slab
        }
    }
    // the 8 rows of the lane: sums over the 16 lanes of the row, transposed; lane t of its half warp
    // ends up with row slot2 + 2 (t >> 1)
    __device__ __forceinline__ void slab_done(int row0, unsigned strip) {
        const int t = cl;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const int o = 8 >> k, h = 4 >> k;
            const bool up = (t & o) != 0;
            float got[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (i < h) got[i] = __shfl_xor_sync(0xffffffffu, up ? rowsum[i] : rowsum[i + h], o);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (i < h) rowsum[i] = (up ? rowsum[i + h] : rowsum[i]) + got[i];
        }
        const float tot = rowsum[0] + __shfl_xor_sync(0xffffffffu, rowsum[0], 1);
        const int row = row0 + slot2 + 2 * (t >> 1);
        if (a.rowpart && (t & 1) == 0 && row < g.n_rows &&
            SB_IN_BOUNDS(a.ds, SBK_STATS, (long long)strip * g.br + row, a.rowpart_limit))
            a.rowpart[(size_t)strip * g.br + row] = tot;
    }
    // the stretch's column sums: c_j, the two half warps (different rows, the same columns), one
    // record of 128 floats
    __device__ __forceinline__ void flush(unsigned q, int) {
        float out[SC_CPL];
#pragma unroll
        for (int k = 0; k < SC_NW; ++k) {
            const f32x2 t2 = mul2(colacc[k], c2[k]);
            colacc[k] = 0ull;
            float a0, a1;
            upk2(t2, a0, a1);
            out[2 * k] = a0 + __shfl_xor_sync(0xffffffffu, a0, 16);
            out[2 * k + 1] = a1 + __shfl_xor_sync(0xffffffffu, a1, 16);
        }
        if (slot2 == 0 && a.rec &&
            SB_IN_BOUNDS(a.ds, SBK_STATS, (long long)(q + gs) * TILE_COLS + cl * SC_CPL + SC_CPL - 1, a.rec_limit)) {
            float4* dst = reinterpret_cast<float4*>(a.rec + (size_t)(q + gs) * TILE_COLS + cl * SC_CPL);
            dst[0] = make_float4(out[0], out[1], out[2], out[3]);
            dst[1] = make_float4(out[4], out[5], out[6], out[7]);
        }
    }
};

template <class P>
__global__ void __launch_bounds__(SC_THREADS, 1)
block_scores_kernel(const __grid_constant__ CUtensorMap wmap,     // the (permuted) weight matrix
                    const int32_t* __restrict__ a_perm,          // original row of permuted r
                    const float* __restrict__ row_weight, ScoreGeom g, ScoreArgs a, SbDeviceState* dstate) {
    constexpr int L = P::L, RPL = P::RPL, NFINE = P::NFINE;
    constexpr bool FULLG = P::FULLG, ROWW = P::ROWW;
    constexpr int STEP_ROWS = 2 * RPL;
    extern __shared__ unsigned char sc_smem_raw[];
    // TMA destinations want 128-byte alignment
    unsigned char* sc_smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(sc_smem_raw) + 127) & ~uintptr_t(127));
    const unsigned bars = smem_u32(sc_smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sc_smem + SC_BAR_BYTES - 8);
    const int lane = threadIdx.x & 31, stream = threadIdx.x >> 5;
    if (threadIdx.x < SC_STREAMS * MAX_RING)
        mbar_init(bars + threadIdx.x * 8, 1);        // the expect_tx arrival; the tile load counts bytes
    if (threadIdx.x == 0) *abort_flag = 0;
    __syncthreads();                                 // the only CTA-wide barrier
    const unsigned gs = blockIdx.x * SC_STREAMS + (unsigned)stream;
    const unsigned s_lo = (unsigned)((unsigned long long)g.n_slabs * gs / g.n_warps);
    const unsigned s_hi = (unsigned)((unsigned long long)g.n_slabs * (gs + 1) / g.n_warps);
    const unsigned n = s_hi - s_lo;
    if (n == 0) return;
    const unsigned slot_bytes = SLAB_BYTES + (unsigned)g.rec_bytes;
    const unsigned smem_base = smem_u32(sc_smem) + SC_BAR_BYTES + (unsigned)stream * g.ring * slot_bytes;
    const int cl = lane & 15, slot2 = lane >> 4;
    const int team = g.group / SC_CPL;
    P sc(a, g, gs, cl, slot2);
    const int rec_pitch = g.gpc * 16;                // bytes between the records of consecutive rows (general form)
    const unsigned lane_slab_off = (unsigned)(slot2 * 256 + cl * 16);
    const unsigned lane_rec_off =
        SLAB_BYTES + (use_pre(L, FULLG) ? (unsigned)(slot2 * pre_stride(L, NFINE))
                      : FULLG           ? (unsigned)(slot2 * 32)
                                        : (unsigned)((slot2 * g.gpc + cl / team) * 16));
    SlabCursor rc = cursor_at(s_lo, g);
    unsigned r_q = s_lo / (unsigned)g.spb;           // chunk column of the cursor
    // staging: one TMA tile load per slab, issued by lane 0, a ring's depth ahead
    SlabCursor ic = rc;
    unsigned issued = 0, i_slot = 0;
    auto stage_next = [&]() {
        if (lane == 0) {
            // a slab at the bottom of a block of odd height takes the rows below along (or zeros past
            // the end of the matrix); they are not used
            const unsigned landed = bar_addr(bars, stream, (int)i_slot);
            mbar_expect_tx(landed, SLAB_BYTES);
            tma_load_slab(smem_base + i_slot * slot_bytes, &wmap, (int)(ic.bx * (unsigned)g.tile_w) + ic.ch * TILE_COLS,
                          (int)(ic.by * (unsigned)g.br) + ic.sl * SLAB_ROWS, landed);
        }
        advance(ic, g);
        ++issued;
        if (++i_slot == (unsigned)g.ring) i_slot = 0;
    };
    while (issued < n && issued < (unsigned)g.ring) stage_next();
    unsigned slot = 0, ph = 0;
    bool ok = true;
    unsigned k = 0;
    sc.begin_column((int)(rc.bx * (unsigned)g.tile_w) + rc.ch * TILE_COLS);
    for (; k < n; ++k) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_addr(bars, stream, (int)slot), ph, abort_flag));
        if (!ok) break;
        const unsigned slab = smem_base + slot * slot_bytes;
        const int rows_here = min(SLAB_ROWS, g.br - rc.sl * SLAB_ROWS);
        const int row0 = (int)(rc.by * (unsigned)g.br) + rc.sl * SLAB_ROWS;
        if (P::FULL_SLABS || rows_here == SLAB_ROWS) {
            slab_records<L, NFINE, FULLG, ROWW>(slab, slab + SLAB_BYTES, row0, g, a.ba, team, cl, slot2, a_perm, row_weight);
            __syncwarp();                            // the records are written
#pragma unroll
            for (int r0 = 0; r0 < SLAB_ROWS; r0 += STEP_ROWS) sc.step(slab + lane_slab_off, slab + lane_rec_off, rec_pitch, r0);
        } else if constexpr (!P::FULL_SLABS) {
            slab_records_ragged<L, NFINE, FULLG, ROWW>(slab, slab + SLAB_BYTES, rows_here, row0, g, a.ba, team, cl, slot2,
                                                       a_perm, row_weight);
            __syncwarp();
            for (int r0 = 0; r0 < rows_here; r0 += STEP_ROWS) sc.step(slab + lane_slab_off, slab + lane_rec_off, rec_pitch, r0);
        }
        __syncwarp();                                // every lane is done with the slot:
        if (issued < n) stage_next();                // refill it (i_slot == slot)
        sc.slab_done(row0, r_q);
        const bool last_of_column = rc.sl == g.spb - 1;
        if (last_of_column || k + 1 == n)
            sc.flush(r_q, (int)(rc.bx * (unsigned)g.tile_w) + rc.ch * TILE_COLS);
        if (last_of_column) ++r_q;
        advance(rc, g);
        if (last_of_column && k + 1 < n) sc.begin_column((int)(rc.bx * (unsigned)g.tile_w) + rc.ch * TILE_COLS);
        if (++slot == (unsigned)g.ring) { slot = 0; ph ^= 1u; }
    }
    if (!ok) {
        // Gave up (a wait ran out, or another warp did).  Tile loads of this warp may still be in
        // flight: wait for each of them (bounded) so that none lands after the CTA has left.
        if (lane == 0) sb_latch(dstate, SB_ERR_TIMEOUT, SBK_SCORES);
        for (; k < issued; ++k) {
            const unsigned long long t0 = now_ns();
            while (!mbar_test(bar_addr(bars, stream, (int)slot), ph) && now_ns() - t0 < SC_WAIT_NS) { }
            if (++slot == (unsigned)g.ring) { slot = 0; ph ^= 1u; }
        }
    }
}

// err[blk][l] = sum of the records of the block's chunk columns, in slab order; gains;
// non-finite check
__global__ void scores_finish_kernel(const float* __restrict__ rec, ScoreGeom g, int64_t n_blocks,
                                     int64_t n_block_cols, int L, BitsArg ba, float M,
                                     float* __restrict__ err, float* __restrict__ gain,
                                     SbDeviceState* dstate) {
    const int64_t blk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    const unsigned by = (unsigned)(blk / n_block_cols), bxb = (unsigned)(blk - (int64_t)by * n_block_cols);
    const unsigned bx = bxb / (unsigned)g.nsub, sb = bxb - bx * (unsigned)g.nsub;
    const unsigned t = by * g.n_tile_cols + bx;
    float e[8];
    for (int l = 0; l < L; ++l) e[l] = 0.f;
    for (int ch = 0; ch < g.chunks; ++ch) {
        const unsigned q = t * (unsigned)g.chunks + (unsigned)ch;
        const unsigned s0 = q * (unsigned)g.spb, s1 = s0 + (unsigned)g.spb - 1u;
        const unsigned w0 = slab_owner(s0, g.n_slabs, g.n_warps), w1 = slab_owner(s1, g.n_slabs, g.n_warps);
        for (unsigned w = w0; w <= w1; ++w) {
            if (slab_range_empty(w, g.n_slabs, g.n_warps)) continue;
            const float* src = rec + ((size_t)(q + w) * g.nsub + sb) * L;
            for (int l = 0; l < L; ++l) e[l] += src[l];
        }
    }
    bool finite = true;
    for (int l = 0; l < L; ++l) {
        err[blk * L + l] = e[l];
        finite = finite && isfinite(e[l]);
    }
    if (!finite) sb_latch(dstate, SB_ERR_NONFINITE, SBK_SCORES);
    if (gain)
        for (int l = 0; l + 1 < L; ++l)
            gain[blk * (L - 1) + l] = (e[l] - e[l + 1]) / ((float)(ba.bits[l + 1] - ba.bits[l]) * M);
}

template <int L, int RPL, int NFINE, bool FULLG, bool ROWW>
sb_status launch_scores_k(sb_ctx* ctx, const CUtensorMap& wmap,
                          const int32_t* cperm, const int32_t* aperm, const float* cm, const float* rw,
                          const ScoreGeom& g, const BitsArg& ba, int64_t n_blocks, int64_t nbc, int grid,
                          float* err, float* gain, float* rec, long long rec_limit) {
    const size_t smem = 128 + SC_BAR_BYTES + (size_t)SC_STREAMS * g.ring * (SLAB_BYTES + g.rec_bytes);
    auto kern = block_scores_kernel<Scorer<L, RPL, NFINE, FULLG, ROWW>>;
    SB_FUNC_ATTR(ctx, kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SC_SMEM_MAX);   // one instance serves several group sizes
    ScoreArgs pa{cperm, cm, ba, rec, nullptr, ctx->dstate, rec_limit, 0};
    kern<<<(unsigned)grid, SC_THREADS, smem, ctx->stream>>>(wmap, aperm, rw, g, pa, ctx->dstate);
    SB_LAUNCHED(ctx);
    scores_finish_kernel<<<(unsigned)((n_blocks + 255) / 256), 256, 0, ctx->stream>>>(
        rec, g, n_blocks, nbc, L, ba, (float)g.br * (float)g.bc, err, gain, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

// the common case (group = 128 columns, no row weights) gets its own instance with the
// group reduction unrolled and ready-made packed pairs in the records; everything else shares
// the general one
template <int L, int RPL, int NFINE, typename... A>
sb_status launch_scores_n(int group, const float* rw, A... args) {
    if (group == 128 && !rw) return launch_scores_k<L, RPL, NFINE, true, false>(args...);
    if (!rw) return launch_scores_k<L, RPL, NFINE, false, false>(args...);
    return launch_scores_k<L, RPL, NFINE, false, true>(args...);
}

// candidates with >= 6 bits keep a two-float grid step; they are the last `nfine` of the list.
// Compiled for 0..2 such candidates and for "all of them" (always correct, a little slower).
template <int L, int RPL, typename... A>
sb_status launch_scores(int nfine, A... args) {
    if (nfine == 0) return launch_scores_n<L, RPL, 0>(args...);
    if (nfine == 1 && L >= 1) return launch_scores_n<L, RPL, (L >= 1 ? 1 : L)>(args...);
    if (nfine == 2 && L >= 2) return launch_scores_n<L, RPL, (L >= 2 ? 2 : L)>(args...);
    return launch_scores_n<L, RPL, L>(args...);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// a bf16 matrix as a 2-D tensor (columns innermost) in tiles of 128 columns x 16 rows; rows and
// columns past the end read as zero
sb_status weight_tile_map(sb_ctx* ctx, const __nv_bfloat16* W, int64_t R, int64_t C, int64_t ld, CUtensorMap* map) {
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SB_CUDA(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess)
            return sb_fail(ctx, SB_ERR_CUDA, "the driver does not export cuTensorMapEncodeTiled");
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)R};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TILE_COLS, (cuuint32_t)SLAB_ROWS};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(W), dims, strides,
                              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return sb_fail(ctx, SB_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return SB_OK;
}

// row_score[r] (+)= sum over strips of rowpart[strip][r]; col_score[j] (+)= sum of the records of
// strip j / 128 in slab order; accumulate: bit 0 rows, bit 1 columns.  A CTA is 32 outputs x 8
// slices of the partial list: every thread's few loads are independent (one round trip to L2), the
// slices are added in slice order (a fixed order: reruns are bit-identical).
constexpr int SF_SLICES = 8;
__global__ void __launch_bounds__(32 * SF_SLICES)
stats_finish_kernel(const float* __restrict__ rec, const float* __restrict__ rowpart, ScoreGeom g,
                    float* __restrict__ row_score, float* __restrict__ col_score, int accumulate,
                    SbDeviceState* dstate) {
    __shared__ float part[SF_SLICES][32];
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
    // outputs: the rows padded to a multiple of 32, then the columns
    const int64_t rows32 = ((int64_t)g.n_rows + 31) / 32 * 32;
    const int64_t i = (int64_t)blockIdx.x * 32 + x;
    const bool is_row = i < rows32;
    const int64_t idx = is_row ? i : i - rows32;
    const bool live = is_row ? (idx < g.n_rows && row_score != nullptr) : (idx < g.n_cols && col_score != nullptr);
    float v = 0.f;
    if (live) {
        if (is_row) {
            const float* src = rowpart + idx;
            for (unsigned s = (unsigned)y; s < g.n_tile_cols; s += SF_SLICES) v += __ldg(src + (size_t)s * g.br);
        } else {
            const int j = (int)idx;
            const unsigned q = (unsigned)j / TILE_COLS;
            const unsigned s0 = q * (unsigned)g.spb, s1 = s0 + (unsigned)g.spb - 1u;
            const unsigned w0 = slab_owner(s0, g.n_slabs, g.n_warps), w1 = slab_owner(s1, g.n_slabs, g.n_warps);
            const float* src = rec + (size_t)q * TILE_COLS + (j - (int)q * TILE_COLS);
            const bool gaps = g.n_warps > g.n_slabs;      // warps without slabs write no record
            for (unsigned w = w0 + (unsigned)y; w <= w1; w += SF_SLICES)
                if (!gaps || !slab_range_empty(w, g.n_slabs, g.n_warps)) v += __ldg(src + (size_t)w * TILE_COLS);
        }
    }
    part[y][x] = v;
    __syncthreads();
    if (y == 0 && live) {
        float t = 0.f;
#pragma unroll
        for (int k = 0; k < SF_SLICES; ++k) t += part[k][x];
        if (is_row) row_score[idx] = (accumulate & 1) ? row_score[idx] + t : t;
        else col_score[idx] = (accumulate & 2) ? col_score[idx] + t : t;
        if (!isfinite(t)) sb_latch(dstate, SB_ERR_NONFINITE, SBK_STATS);
    }
}

template <int NFINE, bool FULLG, bool ROWW>
sb_status launch_stats(sb_ctx* ctx, const CUtensorMap& wmap, const float* rw, const ScoreGeom& g, const ScoreArgs& pa,
                       int grid) {
    const size_t smem = 128 + SC_BAR_BYTES + (size_t)SC_STREAMS * g.ring * (SLAB_BYTES + g.rec_bytes);
    auto kern = block_scores_kernel<StatsScorer<NFINE, FULLG, ROWW>>;
    SB_FUNC_ATTR(ctx, kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SC_SMEM_MAX);
    kern<<<(unsigned)grid, SC_THREADS, smem, ctx->stream>>>(wmap, nullptr, rw, g, pa, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

}  // namespace

// Reorder statistics of one matrix on the slab walk (second-moment form).  Scratch (floats, from the
// caller's arena): col_rec [sb_stats_col_rec_floats], rowpart [sb_stats_rowpart_floats].
size_t sb_stats_col_rec_floats(int64_t C, int sm_count) {
    return (size_t)((C + TILE_COLS - 1) / TILE_COLS + (int64_t)sm_count * SC_STREAMS) * TILE_COLS;
}
size_t sb_stats_rowpart_floats(int64_t R, int64_t C) {
    return (size_t)((C + TILE_COLS - 1) / TILE_COLS) * (size_t)((R + SLAB_ROWS - 1) / SLAB_ROWS * SLAB_ROWS);
}
sb_status sb_reorder_stats_slab(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                const float* col_moment, const float* row_weight, int ref_bits, int group,
                                float* row_score, float* col_score, int accumulate, float* col_rec, float* rowpart) {
    if (R >= (1ll << 30) || C >= (1ll << 30)) return sb_fail(ctx, SB_ERR_SHAPE, "reorder: matrix too large");
    ScoreGeom geo{};
    geo.br = (int)((R + SLAB_ROWS - 1) / SLAB_ROWS * SLAB_ROWS);     // one block row: strips of whole slabs
    geo.bc = TILE_COLS; geo.group = group;
    geo.tile_w = TILE_COLS; geo.chunks = 1;
    geo.spb = geo.br / SLAB_ROWS;
    geo.nsub = 1; geo.lanes_per_sub = TILE_COLS / SC_CPL;
    geo.gpc = TILE_COLS / group;
    const bool fullg = group == 128 && !row_weight;
    const int nfine = ref_bits >= 6 ? 1 : 0;
    geo.rec_bytes = use_pre(1, fullg) ? SLAB_ROWS * pre_stride(1, nfine) : SLAB_ROWS * geo.gpc * 16;
    geo.ring = (SC_SMEM_MAX - SC_BAR_BYTES - 128) / (SC_STREAMS * (SLAB_BYTES + geo.rec_bytes));
    if (geo.ring > MAX_RING) geo.ring = MAX_RING;
    geo.n_rows = (int)R; geo.n_cols = (int)C;
    geo.n_tile_cols = (unsigned)((C + TILE_COLS - 1) / TILE_COLS);
    const int64_t n_slabs = (int64_t)geo.n_tile_cols * geo.spb;
    if (n_slabs >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "reorder: matrix too large");
    geo.n_slabs = (unsigned)n_slabs;
    int64_t grid = (n_slabs + SC_STREAMS - 1) / SC_STREAMS;
    if (grid > ctx->sm_count) grid = ctx->sm_count;
    geo.n_warps = (unsigned)(grid * SC_STREAMS);
    CUtensorMap wmap;
    sb_status st = weight_tile_map(ctx, static_cast<const __nv_bfloat16*>(W), R, C, ldw, &wmap);
    if (st != SB_OK) return st;
    const int one_bit[1] = {ref_bits};
    ScoreArgs pa{nullptr, col_moment, make_bits(one_bit, 1), col_score ? col_rec : nullptr, row_score ? rowpart : nullptr,
                 ctx->dstate, (long long)sb_stats_col_rec_floats(C, ctx->sm_count), (long long)sb_stats_rowpart_floats(R, C)};
    if (row_weight) st = nfine ? launch_stats<1, false, true>(ctx, wmap, row_weight, geo, pa, (int)grid)
                               : launch_stats<0, false, true>(ctx, wmap, row_weight, geo, pa, (int)grid);
    else if (fullg) st = nfine ? launch_stats<1, true, false>(ctx, wmap, nullptr, geo, pa, (int)grid)
                               : launch_stats<0, true, false>(ctx, wmap, nullptr, geo, pa, (int)grid);
    else st = nfine ? launch_stats<1, false, false>(ctx, wmap, nullptr, geo, pa, (int)grid)
                    : launch_stats<0, false, false>(ctx, wmap, nullptr, geo, pa, (int)grid);
    if (st != SB_OK) return st;
    const int64_t n = (R + 31) / 32 * 32 + C;
    stats_finish_kernel<<<(unsigned)((n + 31) / 32), 32 * SF_SLICES, 0, ctx->stream>>>(col_rec, rowpart, geo, row_score,
                                                                                       col_score, accumulate, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}

extern "C" sb_status sb_block_scores(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
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
    // geometry of the slab walk and the record buffer of the partial sums
    ScoreGeom geo{};
    geo.br = br; geo.bc = bc; geo.group = group;
    geo.tile_w = bc >= TILE_COLS ? bc : TILE_COLS;
    if (C % geo.tile_w) return sb_fail(ctx, SB_ERR_SHAPE, "scores: C must be a multiple of 128");
    geo.chunks = geo.tile_w / TILE_COLS;
    geo.spb = (br + SLAB_ROWS - 1) / SLAB_ROWS;
    geo.nsub = bc >= TILE_COLS ? 1 : TILE_COLS / bc;
    geo.lanes_per_sub = bc >= TILE_COLS ? TILE_COLS / SC_CPL : bc / SC_CPL;
    geo.gpc = TILE_COLS / group;
    int nfine = 0;
    for (int l = 0; l < n_bits; ++l) nfine += bits[l] >= 6;
    const bool fullg = group == 128 && !row_weight;
    // (the kernel is compiled for 0, 1, 2 or "all" fine candidates: see launch_scores)
    const int nfine_inst = nfine <= 2 ? nfine : n_bits;
    geo.rec_bytes = use_pre(n_bits, fullg) ? SLAB_ROWS * pre_stride(n_bits, nfine_inst)
                    : fullg                ? SLAB_ROWS * 32
                                           : SLAB_ROWS * geo.gpc * 16;
    geo.ring = (SC_SMEM_MAX - SC_BAR_BYTES - 128) / (SC_STREAMS * (SLAB_BYTES + geo.rec_bytes));
    if (geo.ring > MAX_RING) geo.ring = MAX_RING;
    geo.n_rows = (int)R; geo.n_cols = (int)C;
    geo.n_tile_cols = (unsigned)(C / geo.tile_w);
    const int64_t n_chunk_cols = (R / br) * (int64_t)geo.n_tile_cols * geo.chunks;
    const int64_t n_slabs = n_chunk_cols * geo.spb;
    if (n_slabs >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "scores: matrix too large");
    geo.n_slabs = (unsigned)n_slabs;
    int64_t grid = (n_slabs + SC_STREAMS - 1) / SC_STREAMS;   // persistent: one 16-warp CTA per SM
    if (grid > ctx->sm_count) grid = ctx->sm_count;
    geo.n_warps = (unsigned)(grid * SC_STREAMS);
    const int64_t nbc = C / bc, n_blocks = (R / br) * nbc;
    const size_t rec_bytes = (size_t)(n_chunk_cols + geo.n_warps) * geo.nsub * n_bits * sizeof(float);
    const bool need_copy = row_perm || col_perm || W_perm_out;   // the tile loads read a plain matrix
    void* arena;
    sb_status sst = sb_scratch(ctx, Carver::need({rec_bytes, (need_copy && !W_perm_out) ? (size_t)R * C * 2 : 0}),
                               &arena);
    if (sst != SB_OK) return sst;
    Carver cv(arena);
    float* rec = cv.take<float>(rec_bytes / sizeof(float));
    if (need_copy) {
        void* dst = W_perm_out ? W_perm_out : static_cast<void*>(cv.take<unsigned char>((size_t)R * C * 2));
        sb_status st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, dst);
        if (st != SB_OK) return st;
        src = static_cast<const __nv_bfloat16*>(dst);
        ld = C;
    }
    CUtensorMap wmap;
    {
        sb_status mst = weight_tile_map(ctx, src, R, C, ld, &wmap);
        if (mst != SB_OK) return mst;
    }
    const BitsArg ba = make_bits(bits, n_bits);
    sb_status st = SB_OK;
    // up to four candidates: a lane takes two rows per step; more: one row (fewer accumulators)
#define SB_SCORES(Lv, RPLv)                                                                        \
    st = launch_scores<Lv, RPLv>(nfine, group, row_weight, ctx, wmap, col_perm, row_perm, \
                                 col_moment, row_weight, geo, ba, n_blocks, nbc, (int)grid, err, gain, rec,        \
                                 (long long)(rec_bytes / sizeof(float)))
    switch (n_bits) {
        case 1: SB_SCORES(1, 2); break;
        case 2: SB_SCORES(2, 2); break;
        case 3: SB_SCORES(3, 2); break;
        case 4: SB_SCORES(4, 2); break;
        case 5: SB_SCORES(5, 1); break;
        case 6: SB_SCORES(6, 1); break;
        case 7: SB_SCORES(7, 1); break;
        default: SB_SCORES(8, 1); break;
    }
#undef SB_SCORES
    return st;
}

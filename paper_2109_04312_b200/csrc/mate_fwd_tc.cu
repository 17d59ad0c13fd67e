// Tensor-core forward of multi-view attention (head formula and pattern of Section 3) for bf16,
// d = 64, on sm_100a.  One persistent, warp-specialised CTA per SM walks the units that
// mate_plan assigned to it (see FwdUnit): 256 query rows of one (example, head) in the head's view
// order (Section 3.1: per-head traversal order) against the key tiles those rows may attend.
//
//   warps 0-3   softmax of half 0 (query rows 0..127 of the unit), one thread per row
//   warps 4-7   softmax of half 1 (rows 128..255)
//   warps 8, 9  one thread each issues the tcgen05.mma of half 0 / half 1
//   warps 10-11 loaders: gather Q, K, V rows by view-order index into 128-byte swizzled shared
//               memory with 16-byte cp.async (the gather of Section 3.1 fused into the loads); K/V
//               tiles whose rows lie in place in the tensors come in by one bulk tensor copy each
//
// Per key tile and half:   S = Q K^T  (tcgen05.mma, M = 128, N <= 128, K = 64, accumulator in TMEM)
//                          online softmax in the exp2 domain: P = exp2(S c - m), row sum.  P is
//                          formed in one pass over S with the running max m (for a unit's first
//                          tile: the max over its first 32 columns); the tile's own max is tracked
//                          on the way and only a growth by more than 2^8 sends the tile through
//                          the two-pass path (max, rescale O, exp)
//                          O += P V   (tcgen05.mma, M = 128, N = 64, P read from TMEM; O stays there)
// S is released to the MMA issuer as soon as its last 32 columns sit in registers, so the Q K^T of
// the half's next tile runs under the rest of the exponentials.
// The two halves share every K/V tile and alternate on the tensor pipe, so the exponentials of
// one half overlap the MMAs of the other.  Key tiles of range B are visited by a half only where
// they meet the segments of its rows, and inside a tile a warp evaluates only the 32-column chunks
// that meet the segments of its 32 rows.  The scatter back to the original token order is fused
// into the epilogue (each thread stores its 128-byte row at the row's original position).
#include <cuda.h>
#include <cuda_bf16.h>

#include "mate_internal.h"
#include "sm100_ptx.cuh"

namespace mate {

#ifdef MATE_TRACE
__device__ long long g_trace[kTraceCtas * 32];
#endif

namespace {

using namespace ptx;

constexpr int kSoftmaxWarps = 8;
constexpr int kMmaWarp = 8;   // warps 8 and 9: one MMA-issuing thread per half
constexpr int kMmaWarps = 2;
constexpr int kLoadWarp0 = 10;
constexpr int kLoadWarps = 2;
constexpr int kLoadThreads = 32 * kLoadWarps;
constexpr int kThreads = 32 * (kLoadWarp0 + kLoadWarps);
constexpr int kStages = 5;                   // K/V ring
constexpr int kLag = 2;                      // loader: copy groups in flight behind the newest one

constexpr int kRowBytes = 128;                 // 64 bf16
constexpr int kTileBytes = kTile * kRowBytes;  // 16 KB: 128 rows
constexpr uint32_t kOffQ = 0;                                // [2 buffers][2 halves] x 16 KB
constexpr uint32_t kOffKV = 4 * kTileBytes;                  // [kStages] x (K 16 KB, V 16 KB)
constexpr uint32_t kOffBar = kOffKV + kStages * 2 * kTileBytes;
constexpr uint32_t kSmemBytes = kOffBar + 512 + 1024;        // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 232448, "shared memory per CTA");
// tensor memory: S of half h at column 128 h; O at 256 + 64 h; P (bf16 pairs) at 384 + 64 h
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = 256;
constexpr uint32_t kTmemP = 384;
constexpr uint32_t kWaitLimit = 4096;        // tries (up to 1 ms each) before a wait gives up
constexpr float kRescaleThreshold = 8.f;     // log2 units

// barrier slots (8 bytes each) behind kOffBar
enum {
    kBarQFull = 0,    // [2] loader -> MMA         (count: loader warps)
    kBarQEmpty = 2,   // [2] MMA commit -> loader  (count 2: one per half)
    kBarKVFull = 4,   // [kStages] loader -> MMA   (count: loader warps)
    kBarKVEmpty = 9,  // [kStages] MMA -> loader   (count 2: one per half)
    kBarSFull = 14,   // [2] MMA commit -> softmax (count 1)
    kBarPFull = 16,   // [2] softmax -> MMA        (count 4: one per warp)
    kBarPVDone = 18,  // [2] MMA commit -> softmax: the P V of a tile is complete (count 1)
    kBarFinal = 20,       // [2]
    kBarSchedFull = 22,   // [kSchedDepth] scheduler -> every warp that follows the unit list (count 1)
    kBarSchedEmpty = 26,  // [kSchedDepth] those warps -> scheduler (count kSchedReaders)
    kBarSFree = 30,       // [2] softmax -> MMA: S of a tile has been read for the last time (count 4: one per warp)
    kNumBars = 32
};
constexpr int kSchedDepth = 4;
constexpr int kSchedReaders = kSoftmaxWarps + kMmaWarps + kLoadWarps;
static_assert(kStages <= 5, "barrier slots");

struct Params {
    // 2-D tensor maps over K and V seen as [B H N rows, 64 columns]: boxes of 128 rows, 128-byte swizzle
    CUtensorMap tmK, tmV;
    int use_tma;     // 0: every tile is gathered row by row
    int view_order;  // 1: Q, K, V, O and LSE are laid out in each head's own order (no gather, no scatter)
    const __nv_bfloat16 *Q, *K, *V;
    __nv_bfloat16 *O;
    float *LSE;
    ViewPlan rowv, colv;
    const uint8_t *head_view;
    const FwdUnit *units;
    int n_units;
    int N, H;
    TensorRows tr;     // where (example, head) starts in the tensors
    float scale_log2;  // scale * log2(e)
    int32_t *status;
    int32_t *counters;
    uint8_t *ws;
};

struct TileInfo {
    int k0, w;    // first key and number of keys (<= 128)
    bool is_b;
};

__device__ __forceinline__ int n_tiles_a(const FwdUnit &u) {
    return u.kA_end > u.kA0 ? (u.kA_end - u.kA0 + kTile - 1) / kTile : 0;
}
__device__ __forceinline__ int n_tiles_b(const FwdUnit &u) {
    return u.kB_end > u.kB0 ? (u.kB_end - u.kB0 + kTile - 1) / kTile : 0;
}
__device__ __forceinline__ TileInfo tile_info(const FwdUnit &u, int i, int nA) {
    TileInfo t;
    if (i < nA) {
        t.k0 = u.kA0 + i * kTile;
        t.w = min(kTile, u.kA_end - t.k0);
        t.is_b = false;
    } else {
        t.k0 = u.kB0 + (i - nA) * kTile;
        t.w = min(kTile, u.kB_end - t.k0);
        t.is_b = true;
    }
    return t;
}
__device__ __forceinline__ int rows_of_half(const FwdUnit &u, int h) {
    return max(0, min(kTile, u.nq - h * kTile));
}
// Columns [c0, c1) of the tile (multiples of 16) needed by a half whose rows' segments span keys
// [lo, hi); c1 <= c0 when it skips the tile.
__device__ __forceinline__ void half_cols(int lo, int hi, const TileInfo &t, int &c0, int &c1) {
    if (!t.is_b) {
        c0 = 0;
        c1 = (t.w + 15) & ~15;
    } else {
        c0 = (max(lo, t.k0) - t.k0) & ~15;
        c1 = (min(hi, t.k0 + t.w) - t.k0 + 15) & ~15;
    }
}

__device__ __forceinline__ FwdUnit load_unit(const FwdUnit *p) {
    FwdUnit u;
    const int4 *s = reinterpret_cast<const int4 *>(p);
    int4 *d = reinterpret_cast<int4 *>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) d[i] = __ldg(s + i);
    return u;
}

// The loaders copy a tile of up to 128 rows (128 B each) in passes of kRowsPerPass rows, 8 threads
// per row.  Row rr of the tile comes from view position row0 + min(rr, clamp); its original
// position is looked up first for every pass (independent loads), then the 16-byte copies follow.
constexpr int kRowsPerPass = kLoadThreads / 8;
constexpr int kPasses = (kTile + kRowsPerPass - 1) / kRowsPerPass;

__device__ __forceinline__ void load_indices(int (&idx)[kPasses], const int32_t *perm, int row0,
                                             int n_rows, int clamp, int ltid) {
#pragma unroll
    for (int i = 0; i < kPasses; ++i) {
        const int rr = (ltid >> 3) + kRowsPerPass * i;
        const int t = row0 + min(rr, clamp);
        idx[i] = rr < n_rows ? (perm ? __ldg(perm + t) : t) : -1;  // no order given: the tensors are in view order
    }
}
__device__ __forceinline__ void copy_rows(uint32_t s_tile, const __nv_bfloat16 *src_bh,
                                          const int (&idx)[kPasses], int ltid) {
    const int chunk = ltid & 7;
#pragma unroll
    for (int i = 0; i < kPasses; ++i) {
        const int rr = (ltid >> 3) + kRowsPerPass * i;
        if (idx[i] >= 0)
            cp_async16(s_tile + rr * kRowBytes + ((chunk ^ (rr & 7)) << 4),
                       src_bh + (size_t)idx[i] * 64 + chunk * 8, 16u);
    }
}

// A chunk is 32 scores of one row (tile-local columns cb .. cb + 31).  A column c counts for the row
// iff r_lo <= c < r_lo + r_span; the scores of the other columns are replaced by -inf, which the row
// max ignores and the exponential turns into an exact 0 (the scale is positive).
__device__ __forceinline__ void chunk_mask(uint32_t (&v)[32], int cb, int r_lo, uint32_t r_span) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
        if ((uint32_t)(cb + e - r_lo) >= r_span) v[e] = 0xff800000u;
}
// Row max over one chunk, four partial maxima.
__device__ __forceinline__ void chunk_max(const uint32_t (&v)[32], float (&tm)[4]) {
#pragma unroll
    for (int e = 0; e < 32; e += 8) {
        tm[0] = fmax3(tm[0], __uint_as_float(v[e]), __uint_as_float(v[e + 1]));
        tm[1] = fmax3(tm[1], __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
        tm[2] = fmax3(tm[2], __uint_as_float(v[e + 4]), __uint_as_float(v[e + 5]));
        tm[3] = fmax3(tm[3], __uint_as_float(v[e + 6]), __uint_as_float(v[e + 7]));
    }
}
// P of one chunk: exp2(s * scale_log2 + neg_m), packed as bf16 pairs (even column in the low half);
// the row sums go to two packed pairs of partial sums.  The multiply-adds and the sums work on two
// columns per instruction (packed fp32 pairs); only the exponential is per column.
__device__ __forceinline__ void chunk_exp(const uint32_t (&v)[32], uint64_t scale2, uint64_t neg_m2,
                                          uint32_t (&packed)[16], uint64_t &l01, uint64_t &l23) {
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        float x0, x1, x2, x3;
        unpack_f32x2(fma_f32x2(pack_f32x2(v[e], v[e + 1]), scale2, neg_m2), x0, x1);
        unpack_f32x2(fma_f32x2(pack_f32x2(v[e + 2], v[e + 3]), scale2, neg_m2), x2, x3);
        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
        l01 = add_f32x2(l01, pack_f32x2(p0, p1));
        l23 = add_f32x2(l23, pack_f32x2(p2, p3));
        __nv_bfloat162 b01 = __floats2bfloat162_rn(p0, p1), b23 = __floats2bfloat162_rn(p2, p3);
        packed[e >> 1] = *reinterpret_cast<uint32_t *>(&b01);
        packed[(e >> 1) + 1] = *reinterpret_cast<uint32_t *>(&b23);
    }
}
__device__ __forceinline__ float sum_f32x2(uint64_t a, uint64_t b) {
    float a0, a1, b0, b1;
    unpack_f32x2(a, a0, a1);
    unpack_f32x2(b, b0, b1);
    return (a0 + a1) + (b0 + b1);
}

__global__ void __launch_bounds__(kThreads, 1) tc_fwd_kernel(const __grid_constant__ Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const uint32_t bars = base + kOffBar;
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(sm + kOffBar + 8 * kNumBars);
    volatile int *s_abort = (volatile int *)(sm + kOffBar + 8 * kNumBars + 4);
    volatile int *s_unit = (volatile int *)(sm + kOffBar + 8 * kNumBars + 8);  // [kSchedDepth] unit ids

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bars + 8 * (kBarQFull + i), kLoadWarps);
            mbar_init(bars + 8 * (kBarQEmpty + i), 2);
            mbar_init(bars + 8 * (kBarSFull + i), 1);
            mbar_init(bars + 8 * (kBarPFull + i), 4);
            mbar_init(bars + 8 * (kBarPVDone + i), 1);
            mbar_init(bars + 8 * (kBarSFree + i), 4);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bars + 8 * (kBarKVFull + i), kLoadWarps);
            mbar_init(bars + 8 * (kBarKVEmpty + i), 2);
        }
        for (int i = 0; i < kSchedDepth; ++i) {
            mbar_init(bars + 8 * (kBarSchedFull + i), 1);
            mbar_init(bars + 8 * (kBarSchedEmpty + i), kSchedReaders);
        }
        mbar_init(bars + 8 * kBarFinal, 1);
        mbar_init(bars + 8 * (kBarFinal + 1), 1);
        *s_abort = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32((const void *)tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // every wait is bounded; the first one to expire raises the abort flag, which ends all roles
    auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
        if (mbar_test_wait(bar, parity)) return true;  // already complete: no trip through the suspending form
        for (uint32_t it = 0; it < kWaitLimit; ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if (*s_abort) return false;
        }
        *s_abort = 1;
        atomicOr(p.status + 1, 1);
        return false;
    };

#ifdef MATE_TRACE
    long long tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const long long tr_start = clock64();
#endif
    // The unit list is shared by all CTAs: lane 0 of the first loader warp takes the next index from
    // a global counter and publishes it in a small ring; every warp that follows the list reads the
    // n-th entry here (-1 = the list is exhausted) and frees the slot for the scheduler.
    auto next_unit = [&](uint32_t n) -> int {
        const int slot = n % kSchedDepth;
        if (!wait(bars + 8 * (kBarSchedFull + slot), (n / kSchedDepth) & 1)) return -1;
        const int u = s_unit[slot];
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 8 * (kBarSchedEmpty + slot));
        return u;
    };

    if (warp < kSoftmaxWarps) {
        // ------------------------------------------------------------------ softmax + epilogue
        const int h = warp >> 2;
        const int r = tid & 127;  // row of the half; TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + h * kTile;
        const uint32_t tO = tmem + lane_base + kTmemO + h * 64;
        const uint32_t tP = tmem + lane_base + kTmemP + h * 64;
        const uint32_t bar_s = bars + 8 * (kBarSFull + h), bar_p = bars + 8 * (kBarPFull + h),
                       bar_pv = bars + 8 * (kBarPVDone + h), bar_sf = bars + 8 * (kBarSFree + h);
        uint32_t ph_s = 0, ph_pv = 0;
        bool alive = true;

        for (uint32_t n = 0; alive; ++n) {
            TR_T0(t_nu);
            const int u = next_unit(n);
            TR_ADD(7, t_nu);
            if (u < 0) break;
            TR_T0(t_setup);
            const FwdUnit un = load_unit(p.units + u);
            const int rows_h = rows_of_half(un, h);
            if (rows_h == 0) continue;
            const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
            const int32_t *perm = vp.perm + (size_t)un.b * p.N;
            const size_t bh = p.tr.base(un.b, un.h);
            const bool row_valid = r < rows_h;
            const int t_row = un.q0 + h * kTile + min(r, rows_h - 1);  // rows past the end shadow the last one
            const int orig = p.view_order ? t_row : perm[t_row];
            const int nA = n_tiles_a(un), nB = n_tiles_b(un), n_tiles = nA + nB;
            const int h_lo = h ? un.lo[1] : un.lo[0], h_hi = h ? un.hi[1] : un.hi[0];  // segments of this half's rows

            if (n_tiles == 0) {  // padding rows: O = 0, LSE = -inf
                if (row_valid && p.tr.exists(un.b, orig)) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.O + (bh + orig) * 64);
#pragma unroll
                    for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
                    p.LSE[bh + orig] = -INFINITY;
                }
                continue;
            }

            int my_lo = 0, my_hi = 0, w_lo_min = 0, w_lo_max = 0, w_hi_min = 0, w_hi_max = 0;
            if (nB > 0) {
                my_lo = vp.seg_lo[(size_t)un.b * p.N + t_row];
                my_hi = vp.seg_hi[(size_t)un.b * p.N + t_row];
                w_lo_min = w_lo_max = my_lo;
                w_hi_min = w_hi_max = my_hi;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    w_lo_min = min(w_lo_min, __shfl_xor_sync(0xffffffffu, w_lo_min, o));
                    w_lo_max = max(w_lo_max, __shfl_xor_sync(0xffffffffu, w_lo_max, o));
                    w_hi_min = min(w_hi_min, __shfl_xor_sync(0xffffffffu, w_hi_min, o));
                    w_hi_max = max(w_hi_max, __shfl_xor_sync(0xffffffffu, w_hi_max, o));
                }
            }

            TR_ADD(5, t_setup);
            float m2 = -INFINITY, l = 0.f;  // running max (log2 domain, scaled) and row sum
            bool first = true;

            for (int i = 0; i < n_tiles && alive; ++i) {
                const TileInfo t = tile_info(un, i, nA);
                int c0, c1;
                half_cols(h_lo, h_hi, t, c0, c1);
                if (c1 <= c0) continue;

                // this row's columns [r_lo, r_hi) and the warp's envelope, tile-local
                int r_lo, r_hi, e_lo_min, e_lo_max, e_hi_min, e_hi_max;
                if (!t.is_b) {
                    r_lo = e_lo_min = e_lo_max = 0;
                    r_hi = e_hi_min = e_hi_max = un.kA_end - t.k0;
                } else {
                    r_lo = my_lo - t.k0;
                    r_hi = my_hi - t.k0;
                    e_lo_min = w_lo_min - t.k0;
                    e_lo_max = w_lo_max - t.k0;
                    e_hi_min = w_hi_min - t.k0;
                    e_hi_max = w_hi_max - t.k0;
                }
                const uint32_t r_span = (uint32_t)max(r_hi - r_lo, 0);
                const int ch0 = c0 >> 5, ch1 = (c1 + 31) >> 5;

                TR_T0(t_ws);
                if (!(alive = wait(bar_s, ph_s))) break;
                ph_s ^= 1;
                tc_fence_after();
                TR_ADD(0, t_ws);
                // last chunk of the tile that this warp reads from tensor memory (-1: none): after it,
                // S may be overwritten
                int last_ld = -1;
                for (int ch = ch0; ch < ch1; ++ch)
                    if (!(ch * 32 + 32 <= e_lo_min || ch * 32 >= e_hi_max)) last_ld = ch;
                auto release_s = [&]() {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_sf);
                };
                // P of the previous tile is still being read, and O written, until that tile's P V is done
                bool pv_waited = first;
                auto wait_pv = [&]() -> bool {
                    if (pv_waited) return true;
                    TR_T0(t_wpv);
                    if (!(alive = wait(bar_pv, ph_pv))) return false;
                    ph_pv ^= 1;
                    tc_fence_after();
                    pv_waited = true;
                    TR_ADD(1, t_wpv);
                    return true;
                };

                bool two_pass = first;
                TR_T0(t_p2);
                if (first) {
                    // A unit's first tile has no running max yet.  The max over the first 32 columns in which
                    // the warp has keys serves as the base when every row of the warp has a key there: the
                    // one-pass path below then runs as for any other tile (and still falls back to two passes
                    // when a row's max over the whole tile lies more than the threshold above that base).
                    const int cq = max(ch0, e_lo_min > 0 ? e_lo_min >> 5 : 0);
                    if (cq < ch1 && cq * 32 < e_hi_max) {
                        float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        uint32_t v[32];
                        tmem_ld32(tS + cq * 32, v);
                        tc_wait_ld();
                        if (!(cq * 32 >= e_lo_max && cq * 32 + 32 <= e_hi_min)) chunk_mask(v, cq * 32, r_lo, r_span);
                        chunk_max(v, tm);
                        const float t = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])) * p.scale_log2;
                        if (__all_sync(0xffffffffu, t > -INFINITY)) {
                            m2 = t;
                            two_pass = false;
                        }
                    }
                }
                if (!two_pass) {
                    // one pass with the running max; the tile's own max is known before S is given up
                    float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                    const float neg_m = (m2 == -INFINITY) ? 0.f : -m2;
                    const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2), neg_m2 = pack_f32x2(neg_m, neg_m);
                    uint64_t lsum = 0ull, lsum1 = 0ull;  // packed pairs of partial row sums
                    bool redo = false;
#pragma unroll 1
                    for (int ch = ch0; ch < ch1; ++ch) {
                        const int cb = ch * 32;
                        uint32_t packed[16];
                        if (cb + 32 <= e_lo_min || cb >= e_hi_max) {
#pragma unroll
                            for (int e = 0; e < 16; ++e) packed[e] = 0u;
                        } else {
                            uint32_t v[32];
                            tmem_ld32(tS + cb, v);
                            tc_wait_ld();
                            if (!(cb >= e_lo_max && cb + 32 <= e_hi_min)) chunk_mask(v, cb, r_lo, r_span);
                            chunk_max(v, tm);
                            if (ch == last_ld) {
                                const float t2 = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])) * p.scale_log2;
                                redo = __any_sync(0xffffffffu, t2 > m2 + kRescaleThreshold);
                                if (redo) break;
                                release_s();
                            }
                            chunk_exp(v, scale2, neg_m2, packed, lsum, lsum1);
                        }
                        if (!wait_pv()) break;
                        tmem_st16(tP + ch * 16, packed);
                    }
                    if (!alive) break;
                    if (!redo) {
                        if (last_ld < 0) release_s();
                        l += sum_f32x2(lsum, lsum1);
                    }
                    two_pass = redo;
                }
                if (two_pass) {
                    // pass 1: row max of the raw scores, 32 columns at a time (chunks in which no row of
                    // the warp has a key are not looked at)
                    float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
                    for (int ch = ch0; ch < ch1; ++ch) {
                        const int cb = ch * 32;
                        if (cb + 32 <= e_lo_min || cb >= e_hi_max) continue;
                        uint32_t v[32];
                        tmem_ld32(tS + cb, v);
                        tc_wait_ld();
                        if (!(cb >= e_lo_max && cb + 32 <= e_hi_min)) chunk_mask(v, cb, r_lo, r_span);
                        chunk_max(v, tm);
                    }
                    const float tmax = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3]));
                    const float t2 = tmax * p.scale_log2;
                    const bool grow = t2 > m2 + kRescaleThreshold;  // also true for the first finite max
                    float alpha = 1.f;
                    if (grow) {
                        alpha = ex2(m2 - t2);  // 0 when m2 = -inf
                        m2 = t2;
                        l *= alpha;
                    }
                    if (!wait_pv()) break;
                    if (!first && __any_sync(0xffffffffu, grow)) {
#pragma unroll
                        for (int c2 = 0; c2 < 2; ++c2) {
                            uint32_t o[32];
                            tmem_ld32(tO + c2 * 32, o);
                            tc_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st32(tO + c2 * 32, o);
                        }
                        tc_wait_st();
                    }
                    const float neg_m = (m2 == -INFINITY) ? 0.f : -m2;

                    // pass 2: P = exp2(s * scale_log2 - m) as bf16 pairs into the P columns, row sum
                    const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2), neg_m2 = pack_f32x2(neg_m, neg_m);
                    uint64_t lsum = 0ull, lsum1 = 0ull;
                    if (last_ld < 0) release_s();
#pragma unroll 1
                    for (int ch = ch0; ch < ch1; ++ch) {
                        const int cb = ch * 32;
                        uint32_t packed[16];
                        if (cb + 32 <= e_lo_min || cb >= e_hi_max) {
#pragma unroll
                            for (int e = 0; e < 16; ++e) packed[e] = 0u;
                        } else {
                            uint32_t v[32];
                            tmem_ld32(tS + cb, v);
                            tc_wait_ld();
                            if (ch == last_ld) release_s();
                            if (!(cb >= e_lo_max && cb + 32 <= e_hi_min)) chunk_mask(v, cb, r_lo, r_span);
                            chunk_exp(v, scale2, neg_m2, packed, lsum, lsum1);
                        }
                        tmem_st16(tP + ch * 16, packed);
                    }
                    l += sum_f32x2(lsum, lsum1);
                }
                first = false;

                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p);
                TR_ADD(3, t_p2);
                TR_INC(4);
            }
            if (!alive) break;

            // epilogue: wait for the last P V of this half
            TR_T0(t_ep);
            if (!(alive = wait(bar_pv, ph_pv))) break;
            ph_pv ^= 1;
            tc_fence_after();
            TR_ADD(1, t_ep);
            uint32_t o0[32], o1[32];
            tmem_ld32(tO, o0);
            tmem_ld32(tO + 32, o1);
            tc_wait_ld();

            if (un.n_parts == 1) {
                const float inv_l = l > 0.f ? 1.f / l : 0.f;  // a row without any key (possible in the passes of the
                                                               // row-or-column pattern) gives O = 0, LSE = -inf
                if (row_valid) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.O + (bh + orig) * 64);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t *src = c < 4 ? o0 + 8 * c : o1 + 8 * (c - 4);
                        uint32_t wv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(src[2 * e]) * inv_l,
                                                                      __uint_as_float(src[2 * e + 1]) * inv_l);
                            wv[e] = *reinterpret_cast<uint32_t *>(&b2);
                        }
                        dst[c] = make_uint4(wv[0], wv[1], wv[2], wv[3]);
                    }
                    p.LSE[bh + orig] = (m2 + log2f(l)) * 0.6931471805599453f;
                }
            } else {
                // split unit: publish the un-normalised partial, the last part to arrive combines
                float *part = reinterpret_cast<float *>(p.ws + ((size_t)un.ws_off << 10));
                const int prow = h * kTile + r;
                float4 *po = reinterpret_cast<float4 *>(part + (size_t)prow * 64);
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    po[c] = make_float4(__uint_as_float(o0[4 * c]), __uint_as_float(o0[4 * c + 1]),
                                        __uint_as_float(o0[4 * c + 2]), __uint_as_float(o0[4 * c + 3]));
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    po[8 + c] = make_float4(__uint_as_float(o1[4 * c]), __uint_as_float(o1[4 * c + 1]),
                                            __uint_as_float(o1[4 * c + 2]), __uint_as_float(o1[4 * c + 3]));
                part[kUnitRows * 64 + prow] = m2;
                part[kUnitRows * 64 + kUnitRows + prow] = l;
                // every warp owns its 32 rows: publish, count the arrival, and the warp that comes
                // last for these rows combines all parts (no wait on another CTA anywhere)
                __threadfence();
                __syncwarp();
                int last = 0;
                if (lane == 0) {
                    int32_t *ctr = p.counters + kSchedWords + 8 * un.ctr + 4 * h + (warp & 3);
                    last = atomicAdd(ctr, 1) == un.n_parts - 1;
                    if (last) *ctr = 0;  // ready for the next launch
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    // The warp combines its 32 rows one row at a time with all lanes on the row's 64
                    // columns (two per lane), so every load of a partial row is one coalesced 256-byte
                    // request; a row's weights live in the lane of that row and travel by shuffle.
                    __threadfence();
                    const float *first_part = reinterpret_cast<const float *>(
                        p.ws + ((size_t)(un.ws_off - un.part * (int)(kPartialBytes >> 10)) << 10));
                    const size_t stride = kPartialBytes / sizeof(float);
                    const float *ml = first_part + kUnitRows * 64 + prow;  // this lane's row: max, then sum
                    float M = -INFINITY;
                    for (int q = 0; q < un.n_parts; ++q) M = fmaxf(M, __ldcg(ml + q * stride));
                    float L = 0.f;
                    for (int q = 0; q < un.n_parts; ++q)
                        L = fmaf(__ldcg(ml + q * stride + kUnitRows), ex2(__ldcg(ml + q * stride) - M), L);
                    const float inv_L = 1.f / L;
                    float2 acc[32];
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr) acc[rr] = make_float2(0.f, 0.f);
                    const int row0 = h * kTile + (warp & 3) * 32;  // first row of this warp in the partials
                    for (int q = 0; q < un.n_parts; ++q) {
                        const float wq = ex2(__ldcg(ml + q * stride) - M) * inv_L;
                        const float2 *src = reinterpret_cast<const float2 *>(first_part + q * stride + (size_t)row0 * 64) + lane;
#pragma unroll
                        for (int rr = 0; rr < 32; ++rr) {
                            const float2 x = __ldcg(src + rr * 32);
                            const float w = __shfl_sync(0xffffffffu, wq, rr);
                            acc[rr].x = fmaf(x.x, w, acc[rr].x);
                            acc[rr].y = fmaf(x.y, w, acc[rr].y);
                        }
                    }
#pragma unroll
                    for (int rr = 0; rr < 32; ++rr) {
                        const int dst_row = __shfl_sync(0xffffffffu, orig, rr);
                        const bool ok = __shfl_sync(0xffffffffu, (int)row_valid, rr) != 0;
                        if (ok) {
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[rr].x, acc[rr].y);
                            reinterpret_cast<__nv_bfloat162 *>(p.O + (bh + dst_row) * 64)[lane] = b2;
                        }
                    }
                    if (row_valid) p.LSE[bh + orig] = (M + log2f(L)) * 0.6931471805599453f;
                }
            }
            tc_fence_before();  // O was read; the next unit's first P V may overwrite it
            TR_ADD(6, t_ep);
        }
    } else if (warp < kLoadWarp0) {
        // ------------------------------------------------------------------ MMA issuers (one thread per half)
        // Per half: Q K^T of a tile -> (softmax) -> when P arrives, the Q K^T of the half's next tile
        // goes first (the softmax warps wait for it) and the P V of the finished tile behind it.  A
        // tile's ring stage is released by both halves: by the commit behind the P V, or, for a
        // tile the half skips, by a plain arrival once the tile has landed.
        if (lane == 0) {
            const int h = warp - kMmaWarp;
            uint32_t kv_cnt = 0, unit_cnt = 0, ph_p = 0, ph_sf = 0;
            bool alive = true;
            const uint32_t idesc_pv = idesc_bf16(128, 64, 0, 1);
            const uint32_t tSh0 = tmem + h * kTile, tOh = tmem + kTmemO + h * 64, tPh0 = tmem + kTmemP + h * 64;
            const uint32_t bar_p = bars + 8 * (kBarPFull + h), bar_s = bars + 8 * (kBarSFull + h),
                           bar_pv = bars + 8 * (kBarPVDone + h), bar_sf = bars + 8 * (kBarSFree + h);

            for (uint32_t n = 0; alive; ++n) {
                const int slot = n % kSchedDepth;
                if (!(alive = wait(bars + 8 * (kBarSchedFull + slot), (n / kSchedDepth) & 1))) break;
                const int u = s_unit[slot];
                mbar_arrive(bars + 8 * (kBarSchedEmpty + slot));
                if (u < 0) break;
                const FwdUnit un = load_unit(p.units + u);
                const int nA = n_tiles_a(un), nB = n_tiles_b(un), n_tiles = nA + nB;
                const int h_lo = h ? un.lo[1] : un.lo[0], h_hi = h ? un.hi[1] : un.hi[0];  // segments of this half's rows
                if (n_tiles == 0) continue;
                const int qb = unit_cnt & 1;
                TR_T0(t_qf);
                if (!(alive = wait(bars + 8 * (kBarQFull + qb), (unit_cnt >> 1) & 1))) break;
                tc_fence_after();
                TR_ADD(0, t_qf);
                const uint32_t q_lo = smem_desc_lo(base + kOffQ + (qb * 2 + h) * kTileBytes);
                const bool has_rows = rows_of_half(un, h) > 0;

                // `out`: a tile whose Q K^T has been issued and whose P V has not
                int o_c0 = 0, o_c1 = 0, o_stage = 0;
                bool out = false, acc = false;

                auto issue_pv = [&]() -> bool {  // waits for the P of the outstanding tile, then O += P V
                    TR_T0(t_wp);
                    if (!wait(bar_p, ph_p)) return false;
                    TR_ADD(1, t_wp);
                    ph_p ^= 1;
                    tc_fence_after();
                    TR_T0(t_pv);
                    const int ks0 = o_c0 >> 4, n_ks = (o_c1 - o_c0) >> 4;
                    // V rows 16 ks .. 16 ks + 15 (2 KB per step), P columns 8 ks .. 8 ks + 7
                    uint32_t v_lo = smem_desc_lo(base + kOffKV + o_stage * 2 * kTileBytes + kTileBytes + ks0 * 16 * kRowBytes);
                    uint32_t tPh = tPh0 + ks0 * 8;
                    mma_ts_lean_flag(tOh, tPh, v_lo, idesc_pv, acc);
#pragma unroll 1
                    for (int ks = 1; ks < n_ks; ++ks) {
                        v_lo += (16 * kRowBytes) >> 4;
                        tPh += 8;
                        mma_ts_lean<1>(tOh, tPh, v_lo, idesc_pv);
                    }
                    acc = true;
                    out = false;
                    mma_commit(bar_pv);
                    mma_commit(bars + 8 * (kBarKVEmpty + o_stage));
                    TR_ADD(3, t_pv);
                    return true;
                };
                auto wait_s_free = [&]() -> bool {  // S of the outstanding tile has been read for the last time
                    TR_T0(t_sf);
                    if (!wait(bar_sf, ph_sf)) return false;
                    ph_sf ^= 1;
                    TR_ADD(6, t_sf);
                    return true;
                };

                for (int i = 0; i < n_tiles && alive; ++i) {
                    const TileInfo t = tile_info(un, i, nA);
                    const uint32_t c = kv_cnt + i;
                    const int stage = c % kStages;
                    const uint32_t bar_kv = bars + 8 * (kBarKVFull + stage), par_kv = (c / kStages) & 1;
                    int c0 = 0, c1 = 0;
                    if (has_rows) half_cols(h_lo, h_hi, t, c0, c1);
                    if (c1 <= c0) {  // this half skips the tile
                        if (out) {  // nothing to issue ahead of the P V of the outstanding tile
                            if (!(alive = wait_s_free())) break;
                            if (!(alive = issue_pv())) break;
                        }
                        TR_T0(t_kv);
                        if (!(alive = wait(bar_kv, par_kv))) break;
                        TR_ADD(5, t_kv);
                        mbar_arrive(bars + 8 * (kBarKVEmpty + stage));
                        continue;
                    }
                    if (out && !(alive = wait_s_free())) break;
                    TR_T0(t_kv);
                    if (!(alive = wait(bar_kv, par_kv))) break;
                    TR_ADD(5, t_kv);
                    tc_fence_after();
                    {
                        TR_T0(t_qk);
                        const uint32_t idesc = idesc_bf16(128, c1 - c0, 0, 0);
                        const uint32_t k_lo = smem_desc_lo(base + kOffKV + stage * 2 * kTileBytes + c0 * kRowBytes);
                        const uint32_t tSh = tSh0 + c0;
                        mma_ss_lean<0>(tSh, q_lo, k_lo, idesc);  // K = 64 as four steps of 16 (32 bytes)
                        mma_ss_lean<1>(tSh, q_lo + 2, k_lo + 2, idesc);
                        mma_ss_lean<1>(tSh, q_lo + 4, k_lo + 4, idesc);
                        mma_ss_lean<1>(tSh, q_lo + 6, k_lo + 6, idesc);
                        mma_commit(bar_s);
                        TR_ADD(2, t_qk);
                        TR_INC(4);
                    }
                    if (out && !(alive = issue_pv())) break;  // P V of the previous tile, behind this tile's Q K^T
                    out = true;
                    o_c0 = c0;
                    o_c1 = c1;
                    o_stage = stage;
                }
                if (alive && out) {
                    if ((alive = wait_s_free())) alive = issue_pv();
                }
                kv_cnt += n_tiles;
                if (!alive) break;
                mma_commit(bars + 8 * (kBarQEmpty + qb));
                ++unit_cnt;
            }
            // nothing of this CTA may still run on the tensor pipe when TMEM is freed
            mma_commit(bars + 8 * (kBarFinal + h));
            mbar_wait_bounded(bars + 8 * (kBarFinal + h), 0, kWaitLimit);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ loaders
        const int ltid = tid - 32 * kLoadWarp0;
        uint32_t kv_cnt = 0, unit_cnt = 0;
        uint32_t pend[kLag];
#pragma unroll
        for (int i = 0; i < kLag; ++i) pend[i] = 0;
        bool alive = true;

        // Commits the copies issued so far as one group and signals the barrier of the group that
        // was committed kLag groups earlier (its copies have landed by then).
        auto commit_and_signal = [&](uint32_t bar) {
            cp_async_commit();
            const uint32_t oldest = pend[0];
#pragma unroll
            for (int i = 0; i + 1 < kLag; ++i) pend[i] = pend[i + 1];
            pend[kLag - 1] = bar;
            if (oldest) {
                cp_async_wait_group<kLag>();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(oldest);
            }
        };
        // Signals every group still pending, oldest first and each as soon as its own copies have
        // landed (an older group is not held back by the latency of a newer one).  Called before
        // this warp blocks on a buffer that is not free yet: the consumers may need exactly those
        // groups to free it.
        auto flush = [&]() {
            static_assert(kLag == 2, "written out for two pending groups");
            if (pend[0]) {
                cp_async_wait_group<1>();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(pend[0]);
                pend[0] = 0;
            }
            if (pend[1]) {
                cp_async_wait_group<0>();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(pend[1]);
                pend[1] = 0;
            }
        };
        auto wait_free = [&](uint32_t bar, uint32_t parity) -> bool {
            if (__all_sync(0xffffffffu, mbar_test_wait(bar, parity))) return true;
            TR_T0(t_fl);
            flush();
            TR_ADD(1, t_fl);
            TR_T0(t_wf);
            const bool ok = wait(bar, parity);
            TR_ADD(0, t_wf);
            return ok;
        };

        // scheduler state (lane 0 of the first loader warp only)
        uint32_t produced = 0;
        bool list_done = false;
        auto produce = [&]() -> bool {  // publishes one more entry; false = gave up
            const int slot = produced % kSchedDepth;
            if (produced >= (uint32_t)kSchedDepth) {
                const uint32_t par = ((produced / kSchedDepth) & 1) ^ 1;
                const uint32_t bar = bars + 8 * (kBarSchedEmpty + slot);
                if (!wait(bar, par)) return false;
            }
            // the first unit of a CTA is its own index; later ones come from the shared counter
            const int u = produced == 0 ? (int)blockIdx.x : atomicAdd(p.counters, 1) + (int)gridDim.x;
            const int val = u < p.n_units ? u : -1;
            s_unit[slot] = val;
            mbar_arrive(bars + 8 * (kBarSchedFull + slot));  // release: the store above is visible to the readers
            ++produced;
            if (val < 0) list_done = true;
            return true;
        };

        for (uint32_t n = 0; alive; ++n) {
            // Entry n is taken only now, when the loaders are about to start on it (they run a few key
            // tiles ahead of the other warps): taking units earlier would hand them out before it is
            // known which CTA becomes free first.  Before a loader warp blocks here it signals its
            // pending copy groups: the warps it would wait for may need exactly those tiles.
            {
                const int slot = n % kSchedDepth;
                bool must_wait;
                if (warp == kLoadWarp0) {  // the scheduler's warp: blocks only if the ring slot is still being read
                    must_wait = produced >= (uint32_t)kSchedDepth &&
                                !mbar_test_wait(bars + 8 * (kBarSchedEmpty + slot), ((produced / kSchedDepth) & 1) ^ 1);
                    must_wait = __shfl_sync(0xffffffffu, (int)must_wait, 0) != 0;
                } else {
                    must_wait = !__all_sync(0xffffffffu, mbar_test_wait(bars + 8 * (kBarSchedFull + slot),
                                                                       (n / kSchedDepth) & 1));
                }
                if (must_wait) flush();
            }
            if (ltid == 0) {
                while (!list_done && produced <= n)
                    if (!produce()) break;
            }
            __syncwarp();
            const int u = next_unit(n);
            if (u < 0) break;
            const FwdUnit un = load_unit(p.units + u);
            const int nA = n_tiles_a(un), nB = n_tiles_b(un), n_tiles = nA + nB;
            if (n_tiles == 0) continue;
            const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
            const int32_t *perm = p.view_order ? nullptr : vp.perm + (size_t)un.b * p.N;
            const size_t bh = p.tr.base(un.b, un.h);
            const __nv_bfloat16 *Qbh = p.Q + bh * 64, *Kbh = p.K + bh * 64, *Vbh = p.V + bh * 64;
            // Rows of the order that sit in place in the tensors ([0, ident)): a full K/V tile inside that
            // range is one contiguous [128, 64] box and comes in by one bulk tensor copy per matrix
            // (issued by one thread, completing on the tile's barrier by byte count) instead of 2 x 1024
            // gathered 16-byte copies.  That is the prefix block of every unit and, for a row-major
            // table, every tile of the row view.
            const int ident = !p.use_tma ? 0 : p.view_order ? p.N : __ldg(vp.ident + un.b);

            const int qb = unit_cnt & 1;
            if (!(alive = wait_free(bars + 8 * (kBarQEmpty + qb), ((unit_cnt >> 1) & 1) ^ 1))) break;
            // (Q tiles are always gathered: fetching them with bulk copies as well measured slower.)
            for (int h = 0; h < 2; ++h) {
                const int rows_h = rows_of_half(un, h);
                if (rows_h > 0) {
                    int idx[kPasses];
                    load_indices(idx, perm, un.q0 + h * kTile, kTile, rows_h - 1, ltid);
                    copy_rows(base + kOffQ + (qb * 2 + h) * kTileBytes, Qbh, idx, ltid);
                }
            }
            commit_and_signal(bars + 8 * (kBarQFull + qb));
            ++unit_cnt;

            for (int i = 0; i < n_tiles; ++i) {
                const TileInfo t = tile_info(un, i, nA);
                const int stage = kv_cnt % kStages;
                const bool bulk = t.w == kTile && t.k0 + kTile <= ident;
                int idx[kPasses];
                if (!bulk) load_indices(idx, perm, t.k0, (t.w + 15) & ~15, t.w - 1, ltid);
                if (!(alive = wait_free(bars + 8 * (kBarKVEmpty + stage), ((kv_cnt / kStages) & 1) ^ 1))) break;
                const uint32_t sK = base + kOffKV + stage * 2 * kTileBytes;
                const uint32_t bar_kv = bars + 8 * (kBarKVFull + stage);
                TR_T0(t_cp);
                if (bulk) {
                    if (ltid == 0) {
                        mbar_expect_tx(bar_kv, 2 * kTileBytes);
                        tma_load_2d(sK, &p.tmK, 0, (int)bh + t.k0, bar_kv);
                        tma_load_2d(sK + kTileBytes, &p.tmV, 0, (int)bh + t.k0, bar_kv);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_kv);
                } else {
                    copy_rows(sK, Kbh, idx, ltid);
                    copy_rows(sK + kTileBytes, Vbh, idx, ltid);
                    TR_ADD(2, t_cp);
                    TR_T0(t_cs);
                    commit_and_signal(bar_kv);
                    TR_ADD(3, t_cs);
                }
                // The very first tile of the CTA: the other warps are waiting for it, so it (and Q) are
                // signalled as soon as they have landed, not two tiles later.
                if (kv_cnt == 0) flush();
                TR_INC(4);
                ++kv_cnt;
            }
        }
        flush();  // drain: signal the groups still pending
    }

#ifdef MATE_TRACE
    if (lane == 0 && (warp == 0 || warp == 4 || warp == kMmaWarp || warp == kLoadWarp0) &&
        blockIdx.x < kTraceCtas) {  // MMA: half 0's thread
        const int role = warp == 0 ? 0 : warp == 4 ? 1 : warp == kMmaWarp ? 2 : 3;
        long long *o = g_trace + blockIdx.x * 32 + role * 8;
        for (int i = 0; i < 7; ++i) o[i] = tr[i];
        o[7] = clock64() - tr_start;
    }
#endif
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
    if (tid == 0) {
        // the CTA that finishes last puts the scheduling counters back to zero for the next launch
        // (every CTA has taken its last index by the time it counts itself as finished)
        __threadfence();
        if (atomicAdd(p.counters + 1, 1) == (int)gridDim.x - 1) {
            p.counters[0] = 0;
            p.counters[1] = 0;
        }
    }
}

SmemAttrOnce g_smem_attr;

// cuTensorMapEncodeTiled, taken from the driver through the runtime (the library does not link libcuda)
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(ptr);
    }();
    return fn;
}

// Map over a [rows, 64] bf16 matrix (row = 128 bytes): boxes of 128 rows, written to shared memory in
// the 128-byte swizzle the tensor-core descriptors expect (16-byte chunk index XOR row & 7).
bool make_row_map(CUtensorMap *map, const void *base, size_t rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {64, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {kRowBytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc_supported(int d, int dtype) { return d == 64 && dtype == MATE_BF16; }

int tc_fwd_ctas_per_sm() { return 1; }

size_t tc_fwd_workspace(const mate_plan_t *plan, int) { return plan->fwd_ws_bytes; }

int tc_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, float scale, void *O,
           float *LSE, void *workspace, unsigned flags, cudaStream_t stream) {
    if (!(scale > 0.f)) return MATE_ERR_UNSUPPORTED;  // the row max is taken before scaling (the caller falls back)
    if (plan->n_fwd_units == 0) return MATE_OK;
    if (g_smem_attr.ensure((const void *)tc_fwd_kernel, (int)kSmemBytes, plan->device) != MATE_OK) return MATE_ERR_CUDA;
    Params p;
    const size_t rows = plan->n_rows();
    // Bulk tensor copies for the K/V tiles that are contiguous in the caller's tensors, unless the caller
    // asks for gathers (back to back the bulk copies measured 2-3 % faster on two workloads, equal on one,
    // 0.6 % slower on one); tensors in view order always take them.  When the driver entry point for
    // tensor maps is missing every tile is gathered.
    const bool want_bulk = !(flags & MATE_FLAG_GATHER_TILES) || (flags & MATE_FLAG_VIEW_ORDER);
    p.use_tma = want_bulk && rows < (size_t(1) << 31) && make_row_map(&p.tmK, K, rows) && make_row_map(&p.tmV, V, rows);
    p.view_order = (flags & MATE_FLAG_VIEW_ORDER) ? 1 : 0;
    p.Q = (const __nv_bfloat16 *)Q;
    p.K = (const __nv_bfloat16 *)K;
    p.V = (const __nv_bfloat16 *)V;
    p.O = (__nv_bfloat16 *)O;
    p.LSE = LSE;
    p.rowv = plan->view[0];
    p.colv = plan->view[1];
    p.head_view = plan->head_view_dev;
    p.units = plan->fwd_units_dev;
    p.n_units = plan->n_fwd_units;
    p.N = plan->N;
    p.H = plan->H;
    p.tr = plan->rows();
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = plan->status_dev;
    p.counters = plan->fwd_counters_dev;
    p.ws = (uint8_t *)workspace;
    tc_fwd_kernel<<<plan->n_ctas, kThreads, kSmemBytes, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

}  // namespace mate

#ifdef MATE_TRACE
// copies the cycle counters of the last forward launch to the host: [kTraceCtas CTAs][4 roles][8]
extern "C" int mate_debug_trace(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, mate::g_trace, sizeof(long long) * mate::kTraceCtas * 32) == cudaSuccess ? 0 : -4;
}
#endif

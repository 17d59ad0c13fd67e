// Tensor-core backward of multi-view attention for bf16, d = 64, on sm_100a (derived from the head
// formula of Section 3; the paper states no backward).  With P = exp(scale S - LSE) on the pattern,
// D_k = sum_e dO_ke O_ke and dS = P o (dP - D):
//     dV_j = sum_k P_kj dO_k      dP_kj = dO_k . V_j
//     dQ_k = scale sum_j dS_kj K_j      dK_j = scale sum_k dS_kj Q_k
// The work is the forward's unit list walked twice, once per side, with the tiles of a head taken
// in the head's view order (Section 3.1); the pattern is symmetric, so the same (rows, column
// tiles) units serve both sides:
//   query side  rows = queries, columns = their keys:  S = Q K^T, dP = dO V^T -> dS -> dQ += dS K
//   key side    rows = keys, columns = the queries that attend them:  S^T = K Q^T, dP^T = V dO^T
//               -> P^T, dS^T -> dV += P^T dO, dK += dS^T Q
// so no gradient is accumulated across CTAs (the backward's list splits no unit).
//
// One persistent, warp-specialised CTA per SM (12 warps); work items (unit, half, side) are handed
// out through a counter in the order of the plan's unit list.
//   warps 0-7   arithmetic: two threads (r, r + 128) share row r of the 128-row tile, the lane of
//               tensor memory; each takes 64 of the 128 columns of a column tile, 32 at a time.
//               S and dP (fp32) come out of tensor memory, P / dS (bf16 pairs) go back into it as
//               MMA operands.  (Sixteen warps with 32 columns each were measured 3% slower.)
//   warp  8     one thread issues every tcgen05.mma: S and dP of tile n + 1 are issued as soon as
//               those of tile n sit in registers, ahead of the gradient MMAs of tile n, so both
//               run under the arithmetic
//   warps 9-11  loaders: gather rows by view-order index with 16-byte cp.async into 128-byte
//               swizzled shared memory (row operands double buffered, column tiles in a ring of 4)
// The gradients accumulate in tensor memory and are scattered to the rows' original positions in
// the epilogue.
#include <cuda_bf16.h>

#include <type_traits>

#include "mate_internal.h"
#include "sm100_ptx.cuh"

namespace mate {

#ifdef MATE_TRACE
__device__ long long g_trace_bwd[kTraceCtas * 32];
#endif

namespace {

using namespace ptx;

constexpr int kComputeWarps = 8;                       // 4 per group of 32 columns-per-thread
constexpr int kColsPerThread = 128 / (kComputeWarps / 4);  // columns of a tile per arithmetic thread
constexpr int kRound = 32;                             // columns worked on at a time (16 or 32)
constexpr int kRounds = kColsPerThread / kRound;
constexpr int kMmaWarp = kComputeWarps;
constexpr int kLoadWarp0 = kComputeWarps + 1;
constexpr int kLoadWarps = 3;
constexpr int kLoadThreads = 32 * kLoadWarps;
constexpr int kThreads = 32 * (kLoadWarp0 + kLoadWarps);
constexpr int kStages = 4;  // ring of column tiles
constexpr int kLag = 2;     // loader: copy groups in flight behind the newest one
constexpr int kRowBytes = 128;
constexpr int kTileBytes = kTile * kRowBytes;  // 16 KB
constexpr uint32_t kOffR = 0;                  // [2 buffers] x (Ra: Q or K, Rb: dO or V), 16 KB each
constexpr uint32_t kOffC = 4 * kTileBytes;     // [kStages] x (Ca 16 KB, Cb 16 KB)
constexpr uint32_t kOffVec = kOffC + kStages * 2 * kTileBytes;  // [kStages] x (128 lse, 128 D) floats
constexpr uint32_t kOffBar = kOffVec + kStages * 1024;
constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;
// barrier slots (8 bytes each) behind kOffBar
enum {
    kBarRFull = 0,    // [2] loaders -> MMA                  (count: loader warps)
    kBarREmpty = 2,   // [2] MMA commit -> loaders           (count 1)
    kBarCFull = 4,    // [kStages] loaders -> MMA            (count: loader warps)
    kBarCEmpty = 8,   // [kStages] MMA commit -> loaders     (count 1)
    kBarSFull = 12,   // MMA commit -> arithmetic: S and dP of a tile are complete (count 1)
    kBarAFull = 13,   // arithmetic -> MMA: the bf16 operands of a tile are written (count: one per warp)
    kBarGDone = 14,   // MMA commit -> arithmetic: the gradient MMAs of a tile are complete (count 1)
    kBarFinal = 15,
    kBarSchedFull = 16,   // [kSchedDepth] scheduler -> every warp (count 1)
    kBarSchedEmpty = 20,  // [kSchedDepth] every warp -> scheduler (count kSchedReaders)
    kBarSTFree = 24,      // arithmetic -> MMA: S and dP of a tile are in registers (count: one per warp)
    kNumBars = 25
};
constexpr int kSchedDepth = 4;
constexpr int kSchedReaders = kComputeWarps + 1 + kLoadWarps;
// tensor memory columns
constexpr uint32_t kTmS = 0, kTmT = 128, kTmA1 = 256, kTmA2 = 320, kTmAcc1 = 384, kTmAcc2 = 448;
constexpr uint32_t kWaitLimit = 4096;  // tries (up to 1 ms each) before a wait gives up

struct Params {
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *LSE, *D;  // [B, H, N], original order
    __nv_bfloat16 *dQ, *dK, *dV;
    ViewPlan rowv, colv;
    const uint8_t *head_view;
    const FwdUnit *units;
    int n_units, N, H;
    TensorRows tr;         // where (example, head) starts in the tensors
    float scale, scale_log2;
    int32_t *status;
    int32_t *counter;      // next work item (zeroed before the launch)
};

struct TileInfo {
    int k0, w;
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
// Columns [c0, c1) of the tile (multiples of 16) needed by a half whose rows' segments span keys [lo, hi).
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

// The loaders copy a tile of up to 128 rows (128 B each) of two tensors in passes of kRowsPerPass
// rows, 8 threads per row.  Row rr of the tile comes from view position row0 + min(rr, clamp); its
// original position is looked up first for every pass, then the 16-byte copies follow.
constexpr int kRowsPerPass = kLoadThreads / 8;
constexpr int kPasses = (kTile + kRowsPerPass - 1) / kRowsPerPass;

__device__ __forceinline__ void load_indices(int (&idx)[kPasses], const int32_t *perm, int row0,
                                             int n_rows, int clamp, int ltid) {
#pragma unroll
    for (int i = 0; i < kPasses; ++i) {
        const int rr = (ltid >> 3) + kRowsPerPass * i;
        idx[i] = rr < n_rows ? __ldg(perm + row0 + min(rr, clamp)) : -1;
    }
}
__device__ __forceinline__ void copy_pair(uint32_t s_a, uint32_t s_b, const __nv_bfloat16 *a_bh,
                                          const __nv_bfloat16 *b_bh, const int (&idx)[kPasses], int ltid) {
    const int chunk = ltid & 7;
#pragma unroll
    for (int i = 0; i < kPasses; ++i) {
        const int rr = (ltid >> 3) + kRowsPerPass * i;
        if (idx[i] >= 0) {
            const uint32_t off = rr * kRowBytes + ((chunk ^ (rr & 7)) << 4);
            cp_async16(s_a + off, a_bh + (size_t)idx[i] * 64 + chunk * 8, 16u);
            cp_async16(s_b + off, b_bh + (size_t)idx[i] * 64 + chunk * 8, 16u);
        }
    }
}

// tensor-memory access of one round of columns, by array size
[[maybe_unused]] __device__ __forceinline__ void tmem_ld_round(uint32_t taddr, uint32_t (&v)[16]) { tmem_ld16(taddr, v); }
__device__ __forceinline__ void tmem_ld_round(uint32_t taddr, uint32_t (&v)[32]) { tmem_ld32(taddr, v); }
[[maybe_unused]] __device__ __forceinline__ void tmem_st_round(uint32_t taddr, const uint32_t (&v)[8]) { tmem_st8(taddr, v); }
__device__ __forceinline__ void tmem_st_round(uint32_t taddr, const uint32_t (&v)[16]) { tmem_st16(taddr, v); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&b2);
}

// D_k = sum_e dO_ke O_ke per row (original order), d = 64: eight threads per row, 16 bytes of each
// tensor per thread.  The first thread also clears the work-item counter of the kernel that follows.
__global__ void __launch_bounds__(256) rowdot_kernel(const __nv_bfloat16 *__restrict__ dO,
                                                     const __nv_bfloat16 *__restrict__ O,
                                                     float *__restrict__ D, size_t rows, int32_t *counter) {
    if (blockIdx.x == 0 && threadIdx.x < 64) counter[threadIdx.x] = 0;
    const size_t r = (size_t)blockIdx.x * 32 + (threadIdx.x >> 3);
    const int part = threadIdx.x & 7;
    float acc = 0.f;
    if (r < rows) {
        const uint4 a = __ldg(reinterpret_cast<const uint4 *>(dO + r * 64) + part);
        const uint4 b = __ldg(reinterpret_cast<const uint4 *>(O + r * 64) + part);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&aw[i]));
            const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&bw[i]));
            acc = fmaf(fa.x, fb.x, acc);
            acc = fmaf(fa.y, fb.y, acc);
        }
    }
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (part == 0 && r < rows) D[r] = acc;
}

// Everything an item needs that does not depend on the role of the warp.
struct Item {
    FwdUnit un;
    int h, n_tiles, nA, rows_h, row0, lo, hi;  // lo, hi: un.lo[h], un.hi[h]
    bool key_side;
};
__device__ __forceinline__ Item make_item(const Params &p, int it) {
    Item x;
    x.un = load_unit(p.units + (it >> 2));
    x.h = it & 1;
    x.key_side = (it & 2) != 0;
    x.nA = n_tiles_a(x.un);
    x.n_tiles = x.nA + n_tiles_b(x.un);
    x.rows_h = max(0, min(kTile, x.un.nq - x.h * kTile));
    x.row0 = x.un.q0 + x.h * kTile;
    x.lo = x.h ? x.un.lo[1] : x.un.lo[0];
    x.hi = x.h ? x.un.hi[1] : x.un.hi[0];
    return x;
}
// Next tile at or after i that this half takes part in (n_tiles if none).
__device__ __forceinline__ int next_tile(const Item &x, int i, TileInfo &t, int &c0, int &c1) {
    for (; i < x.n_tiles; ++i) {
        t = tile_info(x.un, i, x.nA);
        half_cols(x.lo, x.hi, t, c0, c1);
        if (c1 > c0) return i;
    }
    return x.n_tiles;
}

__global__ void __launch_bounds__(kThreads, 1) tc_bwd_kernel(const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const uint32_t bars = base + kOffBar;
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(sm + kOffBar + 8 * kNumBars);
    volatile int *s_abort = (volatile int *)(sm + kOffBar + 8 * kNumBars + 4);
    volatile int *s_item = (volatile int *)(sm + kOffBar + 8 * kNumBars + 8);  // [kSchedDepth]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bars + 8 * (kBarRFull + i), kLoadWarps);
            mbar_init(bars + 8 * (kBarREmpty + i), 1);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bars + 8 * (kBarCFull + i), kLoadWarps);
            mbar_init(bars + 8 * (kBarCEmpty + i), 1);
        }
        mbar_init(bars + 8 * kBarSFull, 1);
        mbar_init(bars + 8 * kBarAFull, kComputeWarps);
        mbar_init(bars + 8 * kBarSTFree, kComputeWarps);
        mbar_init(bars + 8 * kBarGDone, 1);
        mbar_init(bars + 8 * kBarFinal, 1);
        for (int i = 0; i < kSchedDepth; ++i) {
            mbar_init(bars + 8 * (kBarSchedFull + i), 1);
            mbar_init(bars + 8 * (kBarSchedEmpty + i), kSchedReaders);
        }
        *s_abort = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32((const void *)tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

#ifdef MATE_TRACE
    long long tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const long long tr_start = clock64();
#endif
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
    // n-th entry of the item list of this CTA (-1 = exhausted); see the scheduler in the loader role
    auto next_item = [&](uint32_t n) -> int {
        const int slot = n % kSchedDepth;
        if (!wait(bars + 8 * (kBarSchedFull + slot), (n / kSchedDepth) & 1)) return -1;
        const int it = s_item[slot];
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 8 * (kBarSchedEmpty + slot));
        return it;
    };

    if (warp < kComputeWarps) {
        // ------------------------------------------------------------------ arithmetic + epilogue
        const int r = tid & 127;   // row of the tile = lane of tensor memory
        const int cq = warp >> 2;  // columns kColsPerThread * cq .. + kColsPerThread - 1 of a column tile
        const uint32_t tm = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        uint32_t ph_s = 0, ph_g = 0, c_cnt = 0;
        bool alive = true;

        for (uint32_t n = 0; alive; ++n) {
            const int it = next_item(n);
            if (it < 0) break;
            const Item x = make_item(p, it);
            if (x.rows_h == 0) continue;
            const FwdUnit &un = x.un;
            const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
            const int32_t *perm = vp.perm + (size_t)un.b * p.N;
            const size_t bh = p.tr.base(un.b, un.h);
            const bool row_valid = r < x.rows_h;
            const int t_row = x.row0 + min(r, x.rows_h - 1);  // rows past the end shadow the last one
            const int orig = perm[t_row];

            if (x.n_tiles == 0) {  // padding rows: zero gradients
                if (row_valid && cq == 0 && p.tr.exists(un.b, orig)) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (!x.key_side) reinterpret_cast<uint4 *>(p.dQ + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                        if (x.key_side) {
                            reinterpret_cast<uint4 *>(p.dK + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                            reinterpret_cast<uint4 *>(p.dV + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                continue;
            }

            // own segment of this row and the envelope over the 32 rows of the warp
            int my_lo = 0, my_hi = 0, w_lo_min = 0, w_lo_max = 0, w_hi_min = 0, w_hi_max = 0;
            if (x.n_tiles > x.nA) {
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
            float row_lse2 = 0.f, row_D = 0.f;  // query side: this row's LSE (log2 domain) and D
            if (!x.key_side) {
                row_lse2 = p.LSE[bh + orig] * 1.4426950408889634f;
                row_D = p.D[bh + orig];
            }

            // the tile loop is compiled once per side (the side is a compile-time constant inside)
            auto tile_loop = [&](auto side) {
            constexpr bool kKeySide = decltype(side)::value;
            TileInfo t;
            int c0 = 0, c1 = 0;
            bool first = true;
            for (int i = next_tile(x, 0, t, c0, c1); i < x.n_tiles && alive; i = next_tile(x, i + 1, t, c0, c1)) {
                const int st = c_cnt % kStages;
                ++c_cnt;
                // this thread's columns [r_lo, r_hi) of the tile and the warp's envelope
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
                const float4 *vec4 = reinterpret_cast<const float4 *>(sm + kOffVec + st * 1024);

                TR_T0(t_ws);
                if (!(alive = wait(bars + 8 * kBarSFull, ph_s))) break;
                ph_s ^= 1;
                tc_fence_after();
                TR_ADD(0, t_ws);
                TR_T0(t_cmp);
                bool a_free = first;  // the operand columns are free once the gradient MMAs of the previous tile are done
                // S and dP may be overwritten as soon as this warp's last load of them has completed
                int last_ld = -1;  // last round of this warp that reads tensor memory
#pragma unroll
                for (int cc = 0; cc < kRounds; ++cc) {
                    const int cbx = cq * kColsPerThread + cc * kRound;
                    if (!(cbx >= c1 || cbx + kRound <= c0) && !(cbx + kRound <= e_lo_min || cbx >= e_hi_max)) last_ld = cc;
                }
                bool st_signalled = false;
                auto signal_st = [&]() {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bars + 8 * kBarSTFree);
                    st_signalled = true;
                };
#pragma unroll 1
                for (int cc = 0; cc < kRounds && alive; ++cc) {
                    const int cb = cq * kColsPerThread + cc * kRound;  // kRound columns at a time
                    if (cb >= c1 || cb + kRound <= c0) continue;  // outside the columns the MMAs touch
                    uint32_t pk_p[kRound / 2], pk_ds[kRound / 2];
                    if (cb + kRound <= e_lo_min || cb >= e_hi_max) {
                        // no row of the warp has a pair here
#pragma unroll
                        for (int e = 0; e < kRound / 2; ++e) pk_p[e] = pk_ds[e] = 0u;
                    } else {
                        uint32_t sv[kRound], tv[kRound];
                        TR_T0(t_ld);
                        tmem_ld_round(tm + kTmS + cb, sv);
                        tmem_ld_round(tm + kTmT + cb, tv);
                        tc_wait_ld();
                        TR_ADD(4, t_ld);
                        if (cc == last_ld) signal_st();
                        // Rounds that lie inside the segment of every row of the warp take the
                        // path without the per-element column test (the side and this flag are
                        // compile-time constants inside).  Two columns at a time, packed fp32.
                        const bool full = cb >= e_lo_max && cb + kRound <= e_hi_min;
                        const uint64_t scale2 = pack_f32x2(p.scale_log2, p.scale_log2);
                        const uint64_t row_nlse2 = pack_f32x2(-row_lse2, -row_lse2), row_D2 = pack_f32x2(row_D, row_D);
                        auto math = [&](auto full_tag) {
                            constexpr bool kFull = decltype(full_tag)::value;
#pragma unroll
                            for (int e = 0; e < kRound; e += 4) {
                                uint64_t nlse[2], Dv[2];
                                if (kKeySide) {
                                    const float4 a = vec4[(cb + e) >> 2], d4 = vec4[32 + ((cb + e) >> 2)];
                                    nlse[0] = pack_f32x2(a.x, a.y);  // the loaders store -LSE
                                    nlse[1] = pack_f32x2(a.z, a.w);
                                    Dv[0] = pack_f32x2(d4.x, d4.y);
                                    Dv[1] = pack_f32x2(d4.z, d4.w);
                                } else {
                                    nlse[0] = nlse[1] = row_nlse2;
                                    Dv[0] = Dv[1] = row_D2;
                                }
#pragma unroll
                                for (int q = 0; q < 2; ++q) {
                                    const int k = e + 2 * q;
                                    float x0, x1;
                                    unpack_f32x2(fma_f32x2(pack_f32x2(sv[k], sv[k + 1]), scale2, nlse[q]), x0, x1);
                                    float p0 = ex2(x0), p1 = ex2(x1);
                                    if (!kFull) {
                                        if ((uint32_t)(cb + k - r_lo) >= r_span) p0 = 0.f;
                                        if ((uint32_t)(cb + k + 1 - r_lo) >= r_span) p1 = 0.f;
                                    }
                                    float d0, d1;
                                    unpack_f32x2(mul_f32x2(pack_f32x2(p0, p1), sub_f32x2(pack_f32x2(tv[k], tv[k + 1]), Dv[q])),
                                                 d0, d1);
                                    pk_p[k >> 1] = pack_bf16(p0, p1);
                                    pk_ds[k >> 1] = pack_bf16(d0, d1);
                                }
                            }
                        };
                        if (full) math(std::true_type{});
                        else math(std::false_type{});
                    }
                    if (!a_free) {
                        TR_T0(t_wg);
                        if (!(alive = wait(bars + 8 * kBarGDone, ph_g))) break;
                        ph_g ^= 1;
                        tc_fence_after();
                        a_free = true;
                        TR_ADD(1, t_wg);
                    }
                    if (kKeySide) tmem_st_round(tm + kTmA1 + (cb >> 1), pk_p);
                    tmem_st_round(tm + (kKeySide ? kTmA2 : kTmA1) + (cb >> 1), pk_ds);
                }
                if (!alive) break;
                if (!st_signalled) signal_st();
                // Nothing written in this tile: the phase is consumed all the same.  The wait also keeps this
                // warp's arrival below out of the barrier phase of the previous tile, which a slower
                // warp may not have reached yet (two arrivals of one warp would complete it early).
                if (!a_free) {
                    if (!(alive = wait(bars + 8 * kBarGDone, ph_g))) break;
                    ph_g ^= 1;
                }
                first = false;
                TR_T0(t_sig);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * kBarAFull);
                TR_ADD(6, t_sig);
                TR_ADD(2, t_cmp);
                TR_INC(7);
            }
            };
            if (x.key_side) tile_loop(std::true_type{});
            else tile_loop(std::false_type{});
            if (!alive) break;

            // epilogue: wait for the last gradient MMAs, then scatter the rows to their original positions
            TR_T0(t_ep);
            if (!(alive = wait(bars + 8 * kBarGDone, ph_g))) break;
            ph_g ^= 1;
            tc_fence_after();
            {
                // The accumulator columns (dQ: 64; key side: dV | dK = 128) are shared out evenly among
                // the column groups of the arithmetic warps, 16 columns at a time.
                constexpr int kGroups = kComputeWarps / 4;
                const int n_cols = (x.key_side ? 128 : 64) / kGroups;
#pragma unroll 1
                for (int sub = 0; sub < n_cols / 16; ++sub) {
                    const int cacc = cq * n_cols + 16 * sub;
                    const bool second = cacc >= 64;  // dK
                    const int col = second ? cacc - 64 : cacc;
                    uint32_t a0[16];
                    tmem_ld16(tm + (second ? kTmAcc2 : kTmAcc1) + col, a0);
                    tc_wait_ld();
                    if (!row_valid) continue;
                    const float mul = (!x.key_side || second) ? p.scale : 1.f;
                    __nv_bfloat16 *out = !x.key_side ? p.dQ : (second ? p.dK : p.dV);
                    uint4 *dst = reinterpret_cast<uint4 *>(out + (bh + orig) * 64 + col);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const uint32_t *src = a0 + 8 * q;
                        dst[q] = make_uint4(pack_bf16(__uint_as_float(src[0]) * mul, __uint_as_float(src[1]) * mul),
                                            pack_bf16(__uint_as_float(src[2]) * mul, __uint_as_float(src[3]) * mul),
                                            pack_bf16(__uint_as_float(src[4]) * mul, __uint_as_float(src[5]) * mul),
                                            pack_bf16(__uint_as_float(src[6]) * mul, __uint_as_float(src[7]) * mul));
                    }
                }
            }
            tc_fence_before();  // the accumulators were read; the next item may overwrite them
            TR_ADD(3, t_ep);
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            uint32_t c_cnt = 0, item_cnt = 0, ph_a = 0, ph_st = 0;
            bool alive = true;
            const uint32_t idesc_g = idesc_bf16(128, 64, 0, 1);  // B = 16 rows of the column tile x 64, MN-major
            for (uint32_t n = 0; alive; ++n) {
                const int slot = n % kSchedDepth;
                if (!(alive = wait(bars + 8 * (kBarSchedFull + slot), (n / kSchedDepth) & 1))) break;
                const int it = s_item[slot];
                mbar_arrive(bars + 8 * (kBarSchedEmpty + slot));
                if (it < 0) break;
                const Item x = make_item(p, it);
                if (x.rows_h == 0 || x.n_tiles == 0) continue;
                const int rb = item_cnt & 1;
                TR_T0(t_rf);
                if (!(alive = wait(bars + 8 * (kBarRFull + rb), (item_cnt >> 1) & 1))) break;
                tc_fence_after();
                TR_ADD(0, t_rf);
                const uint32_t ra = smem_desc_lo(base + kOffR + rb * 2 * kTileBytes), rbb = ra + (kTileBytes >> 4);

                // gradient MMAs of the tile whose operands are (being) written: columns [g0, g1) of stage g_st
                int g0 = 0, g1 = 0, g_st = 0;
                bool have_g = false, acc = false;
                auto issue_grad = [&]() {
                    TR_T0(t_g);
                    const uint32_t sCa = base + kOffC + g_st * 2 * kTileBytes;
                    uint32_t a_lo = smem_desc_lo(sCa + g0 * kRowBytes), b_lo = a_lo + (kTileBytes >> 4);
                    uint32_t tA1 = tmem + kTmA1 + (g0 >> 1), tA2 = tmem + kTmA2 + (g0 >> 1);
                    const int n_ks = (g1 - g0) >> 4;
                    constexpr uint32_t kStepLo = (16 * kRowBytes) >> 4;  // 16 rows of the column tile per step
                    if (x.key_side) {
                        mma_ts_lean_flag(tmem + kTmAcc1, tA1, b_lo, idesc_g, acc);  // dV += P^T dO
                        mma_ts_lean_flag(tmem + kTmAcc2, tA2, a_lo, idesc_g, acc);  // dK += dS^T Q
#pragma unroll 1
                        for (int ks = 1; ks < n_ks; ++ks) {
                            a_lo += kStepLo;
                            b_lo += kStepLo;
                            tA1 += 8;
                            tA2 += 8;
                            mma_ts_lean<1>(tmem + kTmAcc1, tA1, b_lo, idesc_g);
                            mma_ts_lean<1>(tmem + kTmAcc2, tA2, a_lo, idesc_g);
                        }
                    } else {
                        mma_ts_lean_flag(tmem + kTmAcc1, tA1, a_lo, idesc_g, acc);  // dQ += dS K
#pragma unroll 1
                        for (int ks = 1; ks < n_ks; ++ks) {
                            a_lo += kStepLo;
                            tA1 += 8;
                            mma_ts_lean<1>(tmem + kTmAcc1, tA1, a_lo, idesc_g);
                        }
                    }
                    acc = true;
                    mma_commit(bars + 8 * kBarGDone);
                    mma_commit(bars + 8 * (kBarCEmpty + g_st));
                    TR_ADD(3, t_g);
                };

                TileInfo t;
                int c0 = 0, c1 = 0;
                for (int i = next_tile(x, 0, t, c0, c1); i < x.n_tiles && alive; i = next_tile(x, i + 1, t, c0, c1)) {
                    const int st = c_cnt % kStages;
                    TR_T0(t_cf);
                    if (!(alive = wait(bars + 8 * (kBarCFull + st), (c_cnt / kStages) & 1))) break;
                    TR_ADD(1, t_cf);
                    ++c_cnt;
                    if (have_g) {  // S and dP are free again once the previous tile's values are in registers
                        TR_T0(t_wa);
                        if (!(alive = wait(bars + 8 * kBarSTFree, ph_st))) break;
                        ph_st ^= 1;
                        TR_ADD(2, t_wa);
                    }
                    tc_fence_after();
                    {
                        TR_T0(t_s);
                        const uint32_t idesc = idesc_bf16(128, c1 - c0, 0, 0);
                        const uint32_t sCa = base + kOffC + st * 2 * kTileBytes;
                        const uint32_t ca = smem_desc_lo(sCa + c0 * kRowBytes), cb = ca + (kTileBytes >> 4);
                        mma_ss_lean<0>(tmem + kTmS + c0, ra, ca, idesc);  // S = Ra Ca^T, K = 64 as four steps of 16
                        mma_ss_lean<1>(tmem + kTmS + c0, ra + 2, ca + 2, idesc);
                        mma_ss_lean<1>(tmem + kTmS + c0, ra + 4, ca + 4, idesc);
                        mma_ss_lean<1>(tmem + kTmS + c0, ra + 6, ca + 6, idesc);
                        mma_ss_lean<0>(tmem + kTmT + c0, rbb, cb, idesc);  // dP = Rb Cb^T
                        mma_ss_lean<1>(tmem + kTmT + c0, rbb + 2, cb + 2, idesc);
                        mma_ss_lean<1>(tmem + kTmT + c0, rbb + 4, cb + 4, idesc);
                        mma_ss_lean<1>(tmem + kTmT + c0, rbb + 6, cb + 6, idesc);
                        mma_commit(bars + 8 * kBarSFull);
                        TR_ADD(4, t_s);
                        TR_INC(7);
                    }
                    if (have_g) {  // gradient MMAs of the previous tile, behind this tile's S and dP
                        TR_T0(t_wa2);
                        if (!(alive = wait(bars + 8 * kBarAFull, ph_a))) break;
                        ph_a ^= 1;
                        tc_fence_after();
                        TR_ADD(5, t_wa2);
                        issue_grad();
                    }
                    have_g = true;
                    g0 = c0;
                    g1 = c1;
                    g_st = st;
                }
                if (!alive) break;
                if (have_g) {
                    if (!(alive = wait(bars + 8 * kBarSTFree, ph_st))) break;
                    ph_st ^= 1;
                    if (!(alive = wait(bars + 8 * kBarAFull, ph_a))) break;
                    ph_a ^= 1;
                    tc_fence_after();
                    issue_grad();
                }
                mma_commit(bars + 8 * (kBarREmpty + rb));
                ++item_cnt;
            }
            // nothing of this CTA may still run on the tensor pipe when tensor memory is freed
            mma_commit(bars + 8 * kBarFinal);
            mbar_wait_bounded(bars + 8 * kBarFinal, 0, kWaitLimit);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ loaders
        const int ltid = tid - 32 * kLoadWarp0;
        uint32_t c_cnt = 0, item_cnt = 0;
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
            flush();
            TR_T0(t_wf);
            const bool ok = wait(bar, parity);
            TR_ADD(0, t_wf);
            return ok;
        };

        // scheduler (lane 0 of the first loader warp): the first item of a CTA is its own index,
        // later ones come from the shared counter, each taken when the loaders are about to start on it
        uint32_t produced = 0;
        bool list_done = false;
        const int n_items = p.n_units * 4;
        auto produce = [&]() -> bool {
            const int slot = produced % kSchedDepth;
            if (produced >= (uint32_t)kSchedDepth &&
                !wait(bars + 8 * (kBarSchedEmpty + slot), ((produced / kSchedDepth) & 1) ^ 1))
                return false;
            const int it = produced == 0 ? (int)blockIdx.x : atomicAdd(p.counter, 1) + (int)gridDim.x;
            const int val = it < n_items ? it : -1;
            s_item[slot] = val;
            mbar_arrive(bars + 8 * (kBarSchedFull + slot));
            ++produced;
            if (val < 0) list_done = true;
            return true;
        };

        for (uint32_t n = 0; alive; ++n) {
            {   // before a loader warp blocks on the item list it signals its pending copy groups
                const int slot = n % kSchedDepth;
                bool must_wait;
                if (warp == kLoadWarp0) {
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
            const int it = next_item(n);
            if (it < 0) break;
            const Item x = make_item(p, it);
            if (x.rows_h == 0 || x.n_tiles == 0) continue;
            const FwdUnit &un = x.un;
            const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
            const int32_t *perm = vp.perm + (size_t)un.b * p.N;
            const size_t bh = p.tr.base(un.b, un.h);
            const __nv_bfloat16 *Ra_bh = (x.key_side ? p.K : p.Q) + bh * 64, *Rb_bh = (x.key_side ? p.V : p.dO) + bh * 64;
            const __nv_bfloat16 *Ca_bh = (x.key_side ? p.Q : p.K) + bh * 64, *Cb_bh = (x.key_side ? p.dO : p.V) + bh * 64;

            {   // row operands
                const int rb = item_cnt & 1;
                int idx[kPasses];
                load_indices(idx, perm, x.row0, kTile, x.rows_h - 1, ltid);
                if (!(alive = wait_free(bars + 8 * (kBarREmpty + rb), ((item_cnt >> 1) & 1) ^ 1))) break;
                const uint32_t sRa = base + kOffR + rb * 2 * kTileBytes;
                copy_pair(sRa, sRa + kTileBytes, Ra_bh, Rb_bh, idx, ltid);
                commit_and_signal(bars + 8 * (kBarRFull + rb));
                ++item_cnt;
            }
            TileInfo t;
            int c0 = 0, c1 = 0;
            for (int i = next_tile(x, 0, t, c0, c1); i < x.n_tiles; i = next_tile(x, i + 1, t, c0, c1)) {
                const int st = c_cnt % kStages;
                const int n16 = (t.w + 15) & ~15;
                int idx[kPasses];
                load_indices(idx, perm, t.k0, n16, t.w - 1, ltid);
                float v_lse[2] = {0.f, 0.f}, v_D[2] = {0.f, 0.f};
                if (x.key_side) {  // LSE (log2 domain) and D of the query columns
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int cidx = ltid + q * kLoadThreads;
                        if (cidx < kTile) {
                            const int o = perm[t.k0 + min(cidx, t.w - 1)];
                            v_lse[q] = p.LSE[bh + o] * -1.4426950408889634f;  // stored negated: the addend of the exponent
                            v_D[q] = p.D[bh + o];
                        }
                    }
                }
                if (!(alive = wait_free(bars + 8 * (kBarCEmpty + st), ((c_cnt / kStages) & 1) ^ 1))) break;
                const uint32_t sCa = base + kOffC + st * 2 * kTileBytes;
                copy_pair(sCa, sCa + kTileBytes, Ca_bh, Cb_bh, idx, ltid);
                if (x.key_side) {
                    float *vec = reinterpret_cast<float *>(sm + kOffVec + st * 1024);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int cidx = ltid + q * kLoadThreads;
                        if (cidx < kTile) {
                            vec[cidx] = v_lse[q];
                            vec[128 + cidx] = v_D[q];
                        }
                    }
                }
                commit_and_signal(bars + 8 * (kBarCFull + st));
                ++c_cnt;
            }
        }
        flush();  // drain: signal the groups still pending
    }

#ifdef MATE_TRACE
    if (lane == 0 && (warp == 0 || warp == 4 || warp == kMmaWarp || warp == kLoadWarp0) && blockIdx.x < kTraceCtas) {
        const int role = warp == 0 ? 0 : warp == 4 ? 1 : warp == kMmaWarp ? 2 : 3;
        long long *o = g_trace_bwd + blockIdx.x * 32 + role * 8;
        for (int i = 0; i < 8; ++i) o[i] = tr[i];
        if (role == 0) o[5] = clock64() - tr_start;
    }
#endif
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

SmemAttrOnce g_smem_attr;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

// workspace: [256 B counters][D: B*H*N floats]
size_t tc_bwd_workspace(const mate_plan_t *plan) {
    return 256 + align256((size_t)plan->B * plan->H * plan->N * sizeof(float));
}

int tc_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
           const float *LSE, const void *dO, float scale, void *dQ, void *dK, void *dV, void *workspace,
           cudaStream_t stream) {
    if (plan->n_bwd_units == 0) return MATE_OK;
    if (g_smem_attr.ensure((const void *)tc_bwd_kernel, (int)kSmemBytes, plan->device) != MATE_OK) return MATE_ERR_CUDA;
    const size_t bhn = plan->n_rows();
    uint8_t *ws = (uint8_t *)workspace;
    Params p;
    p.Q = (const __nv_bfloat16 *)Q;
    p.K = (const __nv_bfloat16 *)K;
    p.V = (const __nv_bfloat16 *)V;
    p.dO = (const __nv_bfloat16 *)dO;
    p.LSE = LSE;
    p.counter = (int32_t *)ws;
    float *D = (float *)(ws + 256);
    p.D = D;
    p.dQ = (__nv_bfloat16 *)dQ;
    p.dK = (__nv_bfloat16 *)dK;
    p.dV = (__nv_bfloat16 *)dV;
    p.rowv = plan->view[0];
    p.colv = plan->view[1];
    p.head_view = plan->head_view_dev;
    p.units = plan->bwd_units_dev;
    p.n_units = plan->n_bwd_units;
    p.N = plan->N;
    p.H = plan->H;
    p.tr = plan->rows();
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = plan->status_dev;

    rowdot_kernel<<<(unsigned)((bhn + 31) / 32), 256, 0, stream>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, D, bhn,
                                                                   reinterpret_cast<int32_t *>(ws));
    tc_bwd_kernel<<<plan->n_ctas, kThreads, kSmemBytes, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

}  // namespace mate

#ifdef MATE_TRACE
// copies the cycle counters of the last backward launch to the host: [kTraceCtas CTAs][4 roles][8]
extern "C" int mate_debug_trace_bwd(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, mate::g_trace_bwd, sizeof(long long) * mate::kTraceCtas * 32) == cudaSuccess ? 0 : -4;
}
#endif

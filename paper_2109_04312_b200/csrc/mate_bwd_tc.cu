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
// so no gradient is accumulated across CTAs except for prefix rows whose column range was split
// at plan time; those add fp32 partial sums into a scratch buffer that a last small kernel rounds.
//
// One CTA per SM, 512 threads.  Four threads (r, r + 128, r + 256, r + 384) share row r of a
// 128-row tile, the lane of tensor memory; each takes 32 of the 128 columns of a column tile.  Per
// column tile: two tcgen05.mma groups fill S and dP (fp32, tensor memory), the threads turn them
// into bf16 P / dS operands written back to tensor memory, and further MMAs read those operands
// from tensor memory and accumulate the gradients there.  Rows are gathered by view-order index
// with 16-byte cp.async into 128-byte swizzled shared memory (next tile in flight during the
// arithmetic) and scattered back in the epilogue.
#include <cuda_bf16.h>

#include "mate_internal.h"
#include "sm100_ptx.cuh"

namespace mate {

#ifdef MATE_TRACE
__device__ long long g_trace_bwd[148 * 16];
#endif

namespace {

using namespace ptx;

constexpr int kThreads = 512;
constexpr int kRowBytes = 128;
constexpr int kTileBytes = kTile * kRowBytes;  // 16 KB
constexpr uint32_t kOffRa = 0;                 // row operand a (Q or K)
constexpr uint32_t kOffRb = kTileBytes;        // row operand b (dO or V)
constexpr uint32_t kOffC = 2 * kTileBytes;     // [2 stages] x (Ca 16 KB, Cb 16 KB)
constexpr uint32_t kOffVec = kOffC + 4 * kTileBytes;  // [2 stages] x (128 lse, 128 D) floats
constexpr uint32_t kOffBar = kOffVec + 2 * 2 * 128 * 4;
constexpr uint32_t kSmemBytes = kOffBar + 128 + 1024;
// tensor memory columns
constexpr uint32_t kTmS = 0, kTmT = 128, kTmA1 = 256, kTmA2 = 320, kTmAcc1 = 384, kTmAcc2 = 448;
constexpr uint32_t kWaitLimit = 4096;  // tries (up to 1 ms each) before a wait gives up

struct Params {
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *LSE, *D;  // [B, H, N], original order
    __nv_bfloat16 *dQ, *dK, *dV;
    float *acc32;          // [3][B, H, P, 64] partial sums of split prefix rows (dQ, dK, dV)
    size_t plane;          // floats per plane of acc32
    ViewPlan rowv, colv;
    const uint8_t *head_view;
    const FwdUnit *units;
    int n_units, N, H, P;
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
// Columns [c0, c1) of the tile (multiples of 16) that half h of the unit needs.
__device__ __forceinline__ void half_cols(const FwdUnit &u, int h, const TileInfo &t, int &c0, int &c1) {
    if (!t.is_b) {
        c0 = 0;
        c1 = (t.w + 15) & ~15;
    } else {
        c0 = (max(u.lo[h], t.k0) - t.k0) & ~15;
        c1 = (min(u.hi[h], t.k0 + t.w) - t.k0 + 15) & ~15;
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

// Gathers rows of two tensors into two swizzled tiles: row rr comes from view position
// row0 + min(rr, clamp).  64 rows per pass, 8 threads per row.
__device__ __forceinline__ void load_pair(uint32_t s_a, uint32_t s_b, const __nv_bfloat16 *a_bh,
                                          const __nv_bfloat16 *b_bh, const int32_t *perm, int row0,
                                          int n_rows, int clamp, int tid) {
    const int chunk = tid & 7;
    int idx[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int rr = (tid >> 3) + 64 * i;
        idx[i] = rr < n_rows ? __ldg(perm + row0 + min(rr, clamp)) : -1;
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int rr = (tid >> 3) + 64 * i;
        if (idx[i] >= 0) {
            const uint32_t off = rr * kRowBytes + ((chunk ^ (rr & 7)) << 4);
            cp_async16(s_a + off, a_bh + (size_t)idx[i] * 64 + chunk * 8, 16u);
            cp_async16(s_b + off, b_bh + (size_t)idx[i] * 64 + chunk * 8, 16u);
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&b2);
}

// D_k = sum_e dO_ke O_ke per row (original order), one warp per row, d = 64.
__global__ void __launch_bounds__(256) rowdot_kernel(const __nv_bfloat16 *__restrict__ dO,
                                                     const __nv_bfloat16 *__restrict__ O,
                                                     float *__restrict__ D, size_t rows) {
    const size_t r = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const __nv_bfloat162 a = reinterpret_cast<const __nv_bfloat162 *>(dO + r * 64)[lane];
    const __nv_bfloat162 b = reinterpret_cast<const __nv_bfloat162 *>(O + r * 64)[lane];
    float acc = __bfloat162float(a.x) * __bfloat162float(b.x) + __bfloat162float(a.y) * __bfloat162float(b.y);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) D[r] = acc;
}

// Rounds the fp32 sums of the split prefix rows into the outputs: blocks (u, y) cover unit u in
// gridDim.y slices of rows; only the first part of a split unit does anything.  The rows of such a unit are prefix rows, whose view
// position is their original position.
__global__ void __launch_bounds__(256) finalize_kernel(const Params p) {
    const FwdUnit un = load_unit(p.units + blockIdx.x);
    if (un.n_parts <= 1 || un.part != 0) return;
    const size_t bh = (size_t)un.b * p.H + un.h;
    for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < un.nq * 32; i += blockDim.x * gridDim.y) {
        const int row = un.q0 + (i >> 5), c2 = i & 31;
        const float *a = p.acc32 + (bh * p.P + row) * 64 + 2 * c2;
        const size_t dst = (bh * p.N + row) * 64 + 2 * c2;
        const float2 q = *reinterpret_cast<const float2 *>(a);
        const float2 k = *reinterpret_cast<const float2 *>(a + p.plane);
        const float2 v = *reinterpret_cast<const float2 *>(a + 2 * p.plane);
        *reinterpret_cast<__nv_bfloat162 *>(p.dQ + dst) = __floats2bfloat162_rn(q.x, q.y);
        *reinterpret_cast<__nv_bfloat162 *>(p.dK + dst) = __floats2bfloat162_rn(k.x, k.y);
        *reinterpret_cast<__nv_bfloat162 *>(p.dV + dst) = __floats2bfloat162_rn(v.x, v.y);
    }
}

// One work item: half `h` (128 rows) of unit `un`, on the query side (kKeySide = false: rows are
// queries, dQ is produced) or on the key side (rows are keys, dK and dV are produced).
struct Cta {
    uint32_t base, bars, tmem;
    int tid, warp, lane;
    volatile int *s_abort;
#ifdef MATE_TRACE
    long long *tr;
#endif
};

template <bool kKeySide>
__device__ void process_item(const Params &p, const Cta &c, const FwdUnit &un, int h, uint32_t &ph_s,
                             uint32_t &ph_fin) {
    const int tid = c.tid, warp = c.warp;
#ifdef MATE_TRACE
    long long *tr = c.tr;
#endif
    TR_T0(t_item);
    const int r = tid & 127;         // row of the tile = lane of tensor memory
    const int cq = warp >> 2;        // which 32 columns of a column tile this thread works on
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tm = c.tmem + lane_base;
    const uint32_t bar_s = c.bars, bar_fin = c.bars + 8;

    const int rows_h = max(0, min(kTile, un.nq - h * kTile));
    if (rows_h == 0) return;
    const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
    const int32_t *perm = vp.perm + (size_t)un.b * p.N;
    const size_t bh = ((size_t)un.b * p.H + un.h) * p.N;
    const bool row_valid = r < rows_h;
    const int row0 = un.q0 + h * kTile;
    const int t_row = row0 + min(r, rows_h - 1);  // rows past the end shadow the last one
    const int orig = perm[t_row];
    const int nA = n_tiles_a(un), nB = n_tiles_b(un), n_tiles = nA + nB;

    if (n_tiles == 0) {  // padding rows: zero gradients
        if (row_valid && cq == 0) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (!kKeySide) reinterpret_cast<uint4 *>(p.dQ + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                if (kKeySide) {
                    reinterpret_cast<uint4 *>(p.dK + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                    reinterpret_cast<uint4 *>(p.dV + (bh + orig) * 64)[q] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        return;
    }

    const __nv_bfloat16 *Ra_bh = (kKeySide ? p.K : p.Q) + bh * 64, *Rb_bh = (kKeySide ? p.V : p.dO) + bh * 64;
    const __nv_bfloat16 *Ca_bh = (kKeySide ? p.Q : p.K) + bh * 64, *Cb_bh = (kKeySide ? p.dO : p.V) + bh * 64;
    const uint32_t sRa = c.base + kOffRa, sRb = c.base + kOffRb;

    // own segment of this row and the envelope over the 32 rows of the warp
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
    float row_lse2 = 0.f, row_D = 0.f;  // query side: this row's LSE (log2 domain) and D
    if (!kKeySide) {
        row_lse2 = p.LSE[bh + orig] * 1.4426950408889634f;
        row_D = p.D[bh + orig];
    }

    // participating tiles of this half, in order
    auto next_tile = [&](int i, TileInfo &t, int &c0, int &c1) -> int {
        for (; i < n_tiles; ++i) {
            t = tile_info(un, i, nA);
            half_cols(un, h, t, c0, c1);
            if (c1 > c0) return i;
        }
        return n_tiles;
    };
    // column tile `t` into stage `st`: rows [0, n16) of both operands, and on the key side the
    // LSE / D of the query columns
    auto load_cols = [&](const TileInfo &t, int st) {
        const int n16 = (t.w + 15) & ~15;
        const uint32_t sCa = c.base + kOffC + st * 2 * kTileBytes;
        load_pair(sCa, sCa + kTileBytes, Ca_bh, Cb_bh, perm, t.k0, n16, t.w - 1, tid);
        if (kKeySide && tid < kTile) {
            float *vec = reinterpret_cast<float *>(__cvta_shared_to_generic(c.base + kOffVec + st * 1024));
            const int o = perm[t.k0 + min(tid, t.w - 1)];
            vec[tid] = p.LSE[bh + o] * 1.4426950408889634f;
            vec[128 + tid] = p.D[bh + o];
        }
    };

    bool failed = false;
    auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
        for (uint32_t it = 0; it < kWaitLimit; ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if (*c.s_abort) return false;
        }
        *c.s_abort = 1;
        atomicOr(p.status + 1, 1);
        return false;
    };

    TileInfo t;
    int c0 = 0, c1 = 0;
    int i = next_tile(0, t, c0, c1);
    // prologue: row operands and the first column tile
    load_pair(sRa, sRb, Ra_bh, Rb_bh, perm, row0, kTile, rows_h - 1, tid);
    if (i < n_tiles) load_cols(t, 0);
    cp_async_commit();

    int n_done = 0;
    while (i < n_tiles) {
        const int st = n_done & 1;
        const uint32_t sCa = c.base + kOffC + st * 2 * kTileBytes, sCb = sCa + kTileBytes;
        TR_T0(t_ld);
        cp_async_wait_all();
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();  // the tile has landed; everybody is done with tensor memory of the previous tile
        TR_ADD(0, t_ld);
        TR_INC(7);
        TR_T0(t_m1);

        if (tid == 0) {
            tc_fence_after();
            const uint32_t idesc = idesc_bf16(128, c1 - c0, 0, 0);
            const uint32_t ra = smem_desc_lo(sRa), rb = smem_desc_lo(sRb);
            const uint32_t ca = smem_desc_lo(sCa + c0 * kRowBytes), cb = smem_desc_lo(sCb + c0 * kRowBytes);
            mma_ss_lean<0>(c.tmem + kTmS + c0, ra, ca, idesc);  // S = Ra Ca^T, K = 64 as four steps of 16
            mma_ss_lean<1>(c.tmem + kTmS + c0, ra + 2, ca + 2, idesc);
            mma_ss_lean<1>(c.tmem + kTmS + c0, ra + 4, ca + 4, idesc);
            mma_ss_lean<1>(c.tmem + kTmS + c0, ra + 6, ca + 6, idesc);
            mma_ss_lean<0>(c.tmem + kTmT + c0, rb, cb, idesc);  // dP = Rb Cb^T
            mma_ss_lean<1>(c.tmem + kTmT + c0, rb + 2, cb + 2, idesc);
            mma_ss_lean<1>(c.tmem + kTmT + c0, rb + 4, cb + 4, idesc);
            mma_ss_lean<1>(c.tmem + kTmT + c0, rb + 6, cb + 6, idesc);
            mma_commit(bar_s);  // also covers the gradient MMAs of the previous tile
        }
        TR_ADD(1, t_m1);
        TR_T0(t_ws);
        const bool ok = wait(bar_s, ph_s);
        ph_s ^= 1;
        if (__syncthreads_or(!ok)) {
            failed = true;
            break;
        }
        tc_fence_after();
        TR_ADD(2, t_ws);
        TR_T0(t_pf);

        // the other stage is free now (its readers completed with the commit above): next tile
        TileInfo tn;
        int n0 = 0, n1 = 0;
        const int i_next = next_tile(i + 1, tn, n0, n1);
        if (i_next < n_tiles) load_cols(tn, st ^ 1);
        cp_async_commit();

        TR_ADD(3, t_pf);
        TR_T0(t_cmp);
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
        const float4 *vec4 = reinterpret_cast<const float4 *>(__cvta_shared_to_generic(c.base + kOffVec + st * 1024));

        const int cb = cq * 32;  // this thread's 32 columns
        if (cb < c1 && cb + 32 > c0) {  // inside the columns the MMAs touch
            uint32_t pk_p[16], pk_ds[16];
            if (cb + 32 <= e_lo_min || cb >= e_hi_max) {
                // no row of the warp has a pair here
#pragma unroll
                for (int e = 0; e < 16; ++e) pk_p[e] = pk_ds[e] = 0u;
            } else {
                uint32_t sv[32], tv[32];
                tmem_ld32(tm + kTmS + cb, sv);
                tmem_ld32(tm + kTmT + cb, tv);
                tc_wait_ld();
                const bool full = cb >= e_lo_max && cb + 32 <= e_hi_min;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float lse2[4], Dv[4];
                    if (kKeySide) {
                        const float4 a = vec4[(cb + e) >> 2], d4 = vec4[32 + ((cb + e) >> 2)];
                        lse2[0] = a.x; lse2[1] = a.y; lse2[2] = a.z; lse2[3] = a.w;
                        Dv[0] = d4.x; Dv[1] = d4.y; Dv[2] = d4.z; Dv[3] = d4.w;
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            lse2[q] = row_lse2;
                            Dv[q] = row_D;
                        }
                    }
                    float pv[4], dsv[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float x = fmaf(__uint_as_float(sv[e + q]), p.scale_log2, -lse2[q]);
                        pv[q] = ex2(x);
                        if (!full && (uint32_t)(cb + e + q - r_lo) >= r_span) pv[q] = 0.f;
                        dsv[q] = pv[q] * (__uint_as_float(tv[e + q]) - Dv[q]);
                    }
                    pk_p[e >> 1] = pack_bf16(pv[0], pv[1]);
                    pk_p[(e >> 1) + 1] = pack_bf16(pv[2], pv[3]);
                    pk_ds[e >> 1] = pack_bf16(dsv[0], dsv[1]);
                    pk_ds[(e >> 1) + 1] = pack_bf16(dsv[2], dsv[3]);
                }
            }
            if (kKeySide) {
                tmem_st16(tm + kTmA1 + (cb >> 1), pk_p);
                tmem_st16(tm + kTmA2 + (cb >> 1), pk_ds);
            } else {
                tmem_st16(tm + kTmA1 + (cb >> 1), pk_ds);
            }
        }
        tc_wait_st();
        tc_fence_before();
        __syncthreads();
        TR_ADD(4, t_cmp);
        TR_T0(t_m2);

        if (tid == 0) {
            tc_fence_after();
            const uint32_t idesc = idesc_bf16(128, 64, 0, 1);  // B = 16 rows of the column tile x 64, MN-major
            const int ks0 = c0 >> 4, ks1 = c1 >> 4;
            for (int ks = ks0; ks < ks1; ++ks) {
                const uint32_t acc = (n_done > 0 || ks > ks0) ? 1u : 0u;
                if (kKeySide) {
                    // dV += P^T dO, dK += dS^T Q
                    mma_ts_lean_flag(c.tmem + kTmAcc1, c.tmem + kTmA1 + ks * 8, smem_desc_lo(sCb + ks * 16 * kRowBytes), idesc, acc);
                    mma_ts_lean_flag(c.tmem + kTmAcc2, c.tmem + kTmA2 + ks * 8, smem_desc_lo(sCa + ks * 16 * kRowBytes), idesc, acc);
                } else {
                    // dQ += dS K
                    mma_ts_lean_flag(c.tmem + kTmAcc1, c.tmem + kTmA1 + ks * 8, smem_desc_lo(sCa + ks * 16 * kRowBytes), idesc, acc);
                }
            }
        }
        TR_ADD(5, t_m2);
        ++n_done;
        i = i_next;
        t = tn;
        c0 = n0;
        c1 = n1;
    }
    cp_async_wait_all();
    if (failed) return;

    // epilogue: wait for the last gradient MMAs, then scatter the rows (or add split partial sums)
    if (tid == 0) mma_commit(bar_fin);
    const bool ok = wait(bar_fin, ph_fin);
    ph_fin ^= 1;
    if (__syncthreads_or(!ok)) return;
    tc_fence_after();
    if (kKeySide || cq < 2) {
        // column quarters 0, 1: the two halves of accumulator 1 (dQ or dV); 2, 3 (key side): of accumulator 2 (dK)
        const int half = cq & 1;
        const uint32_t tacc = tm + (cq < 2 ? kTmAcc1 : kTmAcc2) + 32 * half;
        const float mul = (!kKeySide || cq >= 2) ? p.scale : 1.f;
        __nv_bfloat16 *out = !kKeySide ? p.dQ : (cq < 2 ? p.dV : p.dK);
        const int plane = !kKeySide ? 0 : (cq < 2 ? 2 : 1);
        uint32_t a0[32];
        tmem_ld32(tacc, a0);
        tc_wait_ld();
        if (row_valid) {
            if (un.n_parts == 1) {
                uint4 *dst = reinterpret_cast<uint4 *>(out + (bh + orig) * 64 + 32 * half);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t *src = a0 + 8 * q;
                    dst[q] = make_uint4(pack_bf16(__uint_as_float(src[0]) * mul, __uint_as_float(src[1]) * mul),
                                        pack_bf16(__uint_as_float(src[2]) * mul, __uint_as_float(src[3]) * mul),
                                        pack_bf16(__uint_as_float(src[4]) * mul, __uint_as_float(src[5]) * mul),
                                        pack_bf16(__uint_as_float(src[6]) * mul, __uint_as_float(src[7]) * mul));
                }
            } else {
                // split prefix rows: view position = original position < P
                float *dst = p.acc32 + plane * p.plane + (((size_t)un.b * p.H + un.h) * p.P + orig) * 64 + 32 * half;
#pragma unroll
                for (int e = 0; e < 32; ++e) atomicAdd(dst + e, __uint_as_float(a0[e]) * mul);
            }
        }
    }
    tc_fence_before();
    __syncthreads();  // tensor memory and the row operand tiles are free for the next item
    TR_ADD(6, t_item);
}

// Work items: (unit, half, side), taken from a counter in the order of the plan's unit list
// (largest units first).
__global__ void __launch_bounds__(kThreads, 1) tc_bwd_kernel(const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    Cta c;
    c.base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (c.base - raw);
    c.bars = c.base + kOffBar;
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(sm + kOffBar + 16);
    c.s_abort = (volatile int *)(sm + kOffBar + 20);
    volatile int *s_item = (volatile int *)(sm + kOffBar + 24);
    c.tid = threadIdx.x;
    c.warp = c.tid >> 5;
    c.lane = c.tid & 31;

    if (c.tid == 0) {
        mbar_init(c.bars, 1);
        mbar_init(c.bars + 8, 1);
        *c.s_abort = 0;
        fence_mbar_init();
    }
    if (c.warp == 0) {
        tmem_alloc(smem_u32((const void *)tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    c.tmem = *tmem_slot;

#ifdef MATE_TRACE
    long long tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    c.tr = tr;
    const long long tr_start = clock64();
#endif
    uint32_t ph_s = 0, ph_fin = 0;
    const int n_items = p.n_units * 4;
    while (true) {
        if (c.tid == 0) *s_item = atomicAdd(p.counter, 1);
        __syncthreads();
        const int item = *s_item;
        __syncthreads();
        if (item >= n_items || *c.s_abort) break;
        const FwdUnit un = load_unit(p.units + (item >> 2));
        const int h = item & 1;
        if (item & 2) process_item<true>(p, c, un, h, ph_s, ph_fin);
        else process_item<false>(p, c, un, h, ph_s, ph_fin);
    }

#ifdef MATE_TRACE
    if (c.tid == 0 || c.tid == 255) {
        long long *o = g_trace_bwd + blockIdx.x * 16 + (c.tid == 0 ? 0 : 8);
        for (int i = 0; i < 8; ++i) o[i] = tr[i];
        if (c.tid == 0) o[6] = clock64() - tr_start;  // thread 0: total instead of the item sum
    }
#endif
    // nothing of this CTA may still run on the tensor pipe when tensor memory is freed
    if (*c.s_abort && c.tid == 0) {
        mma_commit(c.bars + 8);
        mbar_wait_bounded(c.bars + 8, ph_fin, kWaitLimit);
    }
    tc_fence_before();
    __syncthreads();
    if (c.warp == 0) tmem_dealloc(c.tmem, 512);
}

bool g_attr_set = false;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

// workspace: [256 B counters][D: B*H*N floats][acc32: 3 planes of B*H*P*64 floats, only with split units]
size_t tc_bwd_workspace(const mate_plan_t *plan) {
    const size_t bhn = (size_t)plan->B * plan->H * plan->N;
    size_t bytes = 256 + align256(bhn * sizeof(float));
    if (plan->n_fwd_slots > 0) bytes += align256(3 * (size_t)plan->B * plan->H * plan->P * 64 * sizeof(float));
    return bytes;
}

int tc_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
           const float *LSE, const void *dO, float scale, void *dQ, void *dK, void *dV, void *workspace,
           cudaStream_t stream) {
    if (plan->n_fwd_units == 0) return MATE_OK;
    if (!g_attr_set) {
        if (cudaFuncSetAttribute(tc_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemBytes) != cudaSuccess)
            return MATE_ERR_CUDA;
        g_attr_set = true;
    }
    const size_t bhn = (size_t)plan->B * plan->H * plan->N;
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
    p.plane = (size_t)plan->B * plan->H * plan->P * 64;
    p.acc32 = plan->n_fwd_slots > 0 ? (float *)(ws + 256 + align256(bhn * sizeof(float))) : nullptr;
    p.rowv = plan->view[0];
    p.colv = plan->view[1];
    p.head_view = plan->head_view_dev;
    p.units = plan->fwd_units_dev;
    p.n_units = plan->n_fwd_units;
    p.N = plan->N;
    p.H = plan->H;
    p.P = plan->P;
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = plan->status_dev;

    if (cudaMemsetAsync(ws, 0, 256, stream) != cudaSuccess) return MATE_ERR_CUDA;
    if (p.acc32 && cudaMemsetAsync(p.acc32, 0, 3 * p.plane * sizeof(float), stream) != cudaSuccess)
        return MATE_ERR_CUDA;
    rowdot_kernel<<<(unsigned)((bhn + 7) / 8), 256, 0, stream>>>((const __nv_bfloat16 *)dO, (const __nv_bfloat16 *)O, D, bhn);
    tc_bwd_kernel<<<plan->n_ctas, kThreads, kSmemBytes, stream>>>(p);
    if (p.acc32) finalize_kernel<<<dim3(plan->n_fwd_units, 16), 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

}  // namespace mate

#ifdef MATE_TRACE
// copies the cycle counters of the last backward launch to the host: [148 CTAs][2 threads][8]
extern "C" int mate_debug_trace_bwd(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, mate::g_trace_bwd, sizeof(long long) * 148 * 16) == cudaSuccess ? 0 : -4;
}
#endif

// Tensor-core forward of multi-view attention (head formula and pattern of Section 3) for bf16,
// d = 64, on sm_100a: tcgen05 MMAs with accumulators in TMEM, operands gathered into 128-byte
// swizzled shared memory in the head's view order (Section 3.1: per-head traversal order).
//
// One CTA (128 threads, thread r = query row r of the tile) walks a list of units (see FwdUnit).
// For every key tile of a unit:
//     S = Q K^T            tcgen05.mma, M = 128, N = tile width rounded to 16, K = 64  -> TMEM
//     online softmax       one thread per row reads its S row from TMEM (two passes: max, then
//                          exp2 / row sum), writes P as bf16 into swizzled shared memory
//     O += P V             tcgen05.mma, M = 128, N = 64, K = tile width; O stays in TMEM and is
//                          rescaled only when a row's running max grows by more than 2^8
// Gather is fused into the loads (each 128-byte row is fetched by its view-order index with
// cp.async), scatter into the epilogue (each thread stores its row at the original position).
// Two CTAs share an SM (256 of 512 TMEM columns and ~98 KB of shared memory each), so one CTA's
// softmax overlaps the other's MMAs.
#include <cuda_bf16.h>

#include "mate_internal.h"
#include "sm100_ptx.cuh"

namespace mate {

namespace {

using namespace ptx;

constexpr int kThreads = 128;
constexpr int kRowBytes = 128;               // 64 bf16
constexpr int kTileBytes = kTile * kRowBytes;  // 16 KB: 128 rows
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffK = kTileBytes;
constexpr uint32_t kOffV = 2 * kTileBytes;   // two stages
constexpr uint32_t kOffP = 4 * kTileBytes;   // 128 x 128 bf16 = two 64-column blocks of 16 KB
constexpr uint32_t kOffBar = 6 * kTileBytes;
constexpr uint32_t kSmemBytes = kOffBar + 64 + 1024;  // + slack for the 1024-byte alignment
constexpr uint32_t kTmemCols = 256;          // S: columns [0,128), O: columns [128,192)
constexpr uint32_t kWaitLimit = 1u << 24;    // polls before a wait gives up
constexpr float kRescaleThreshold = 8.f;     // log2 units

struct Params {
    const __nv_bfloat16 *Q, *K, *V;
    __nv_bfloat16 *O;
    float *LSE;
    ViewPlan rowv, colv;
    const uint8_t *head_view;
    const FwdUnit *units;
    int n_units, N, H;
    float scale_log2;  // scale * log2(e)
    int32_t *status;
};

// Gathers `n_rows` rows (128 B each) of src[(row0 + i)-th view position] into a swizzled tile;
// rows at or beyond `n_load` are zero-filled.  8 threads fetch one row, 16 rows per pass.
__device__ __forceinline__ void load_tile(uint32_t s_tile, const __nv_bfloat16 *src_bh,
                                          const int32_t *perm, int row0, int n_load, int n_rows,
                                          int row_clamp, int tid) {
    const int chunk = tid & 7;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int rr = (tid >> 3) + 16 * i;
        if (rr < n_rows) {
            const bool on = rr < n_load;
            const int t = row0 + min(rr, row_clamp);
            const int src_row = on ? perm[t] : 0;
            const void *src = src_bh + (size_t)src_row * 64 + chunk * 8;
            cp_async16(s_tile + rr * kRowBytes + ((chunk ^ (rr & 7)) << 4), src, on ? 16u : 0u);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 2) tc_fwd_kernel(const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const uint32_t sQ = base + kOffQ, sK = base + kOffK, sP = base + kOffP;
    const uint32_t bar_s = base + kOffBar, bar_pv = bar_s + 8;
    volatile uint32_t *tmem_slot = (volatile uint32_t *)(sm + kOffBar + 16);
    volatile int *s_abort = (volatile int *)(sm + kOffBar + 20);
    int *s_red = (int *)(sm + kOffBar + 32);  // [0..3] lo max per warp, [4..7] hi min per warp

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_pv, 1);
        *s_abort = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32((const void *)tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tS = tmem + ((uint32_t)(warp * 32) << 16);  // this warp's 32 lanes
    const uint32_t tO = tS + 128;
    uint32_t phase_s = 0, phase_pv = 0;

    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (*s_abort) return;
        if (!mbar_wait_bounded(bar, parity, kWaitLimit)) {
            *s_abort = 1;
            atomicOr(p.status + 1, 1);
        }
    };

    for (int u = blockIdx.x; u < p.n_units; u += gridDim.x) {
        const FwdUnit un = p.units[u];
        const ViewPlan &vp = p.head_view[un.h] ? p.colv : p.rowv;
        const int32_t *perm = vp.perm + (size_t)un.b * p.N;
        const size_t bh = ((size_t)un.b * p.H + un.h) * p.N;
        const __nv_bfloat16 *Qbh = p.Q + bh * 64, *Kbh = p.K + bh * 64, *Vbh = p.V + bh * 64;
        const int n_tiles = un.kA_n + un.kB_n;
        const bool row_valid = tid < un.nq;
        const int t_row = un.q0 + min(tid, un.nq - 1);  // rows past nq shadow the last valid row
        const int orig = perm[t_row];

        if (n_tiles == 0) {  // padding rows: O = 0, LSE = -inf
            if (row_valid) {
                uint4 *dst = reinterpret_cast<uint4 *>(p.O + (bh + orig) * 64);
#pragma unroll
                for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
                p.LSE[bh + orig] = -INFINITY;
            }
            continue;
        }

        const int my_lo = vp.seg_lo[(size_t)un.b * p.N + t_row];
        const int my_hi = vp.seg_hi[(size_t)un.b * p.N + t_row];
        {   // block-wide max of lo and min of hi: decides which B tiles need no mask
            int lo_max = my_lo, hi_min = my_hi;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                lo_max = max(lo_max, __shfl_xor_sync(0xffffffffu, lo_max, o));
                hi_min = min(hi_min, __shfl_xor_sync(0xffffffffu, hi_min, o));
            }
            if (lane == 0) {
                s_red[warp] = lo_max;
                s_red[4 + warp] = hi_min;
            }
        }

        auto tile_range = [&](int i, int &k0, int &w) {
            if (i < un.kA_n) {
                k0 = i * kTile;
                w = min(kTile, un.kA_end - k0);
            } else {
                k0 = un.kB0 + (i - un.kA_n) * kTile;
                w = min(kTile, un.kB_end - k0);
            }
        };

        // prologue: Q tile and key tile 0
        load_tile(sQ, Qbh, perm, un.q0, kTile, kTile, un.nq - 1, tid);
        {
            int k0, w;
            tile_range(0, k0, w);
            const int n16 = (w + 15) & ~15;
            load_tile(sK, Kbh, perm, k0, w, n16, kTile, tid);
            load_tile(base + kOffV, Vbh, perm, k0, w, n16, kTile, tid);
        }
        cp_async_commit();

        float m2 = -INFINITY, l = 0.f;  // running max (log2 domain, scaled) and row sum

        for (int i = 0; i < n_tiles; ++i) {
            const int st = i & 1;
            int k0, w;
            tile_range(i, k0, w);
            const int n16 = (w + 15) & ~15;
            const uint32_t sV = base + kOffV + st * kTileBytes;

            cp_async_wait_all();
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();  // tile i (and Q) landed; previous TMEM reads are done

            if (tid == 0) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(128, n16, 0, 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_bf16_ss(tmem, smem_desc_sw128(sQ + ks * 32), smem_desc_sw128(sK + ks * 32),
                                idesc, ks > 0);
                mma_commit(bar_s);
            }
            if (i > 0) {  // P V of the previous tile done: P, the other V stage and O are free
                wait(bar_pv, phase_pv);
                phase_pv ^= 1;
            }
            wait(bar_s, phase_s);
            phase_s ^= 1;
            tc_fence_after();

            if (i + 1 < n_tiles) {  // prefetch the next key tile while this one is in softmax
                int k0n, wn;
                tile_range(i + 1, k0n, wn);
                const int n16n = (wn + 15) & ~15;
                load_tile(sK, Kbh, perm, k0n, wn, n16n, kTile, tid);
                load_tile(base + kOffV + (st ^ 1) * kTileBytes, Vbh, perm, k0n, wn, n16n, kTile, tid);
                cp_async_commit();
            }

            // column window of this row inside the tile: key j = k0 + c counts iff c_lo <= c < c_hi
            int c_lo, c_hi;
            bool full;
            if (i < un.kA_n) {
                c_lo = 0;
                c_hi = un.kA_end - k0;
                full = (w == kTile);
            } else {
                c_lo = my_lo - k0;
                c_hi = my_hi - k0;
                const int lo_max = max(max(s_red[0], s_red[1]), max(s_red[2], s_red[3]));
                const int hi_min = min(min(s_red[4], s_red[5]), min(s_red[6], s_red[7]));
                full = (w == kTile) && (k0 >= lo_max) && (k0 + kTile <= hi_min);
            }
            const uint32_t c_span = (uint32_t)max(c_hi - c_lo, 0);
            const int n_chunks = (n16 + 31) >> 5;

            // pass 1: row max of the raw scores
            float tmax = -INFINITY;
#pragma unroll 1
            for (int ch = 0; ch < n_chunks; ++ch) {
                uint32_t v[32];
                tmem_ld32(tS + ch * 32, v);
                tc_wait_ld();
                if (full) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) tmax = fmaxf(tmax, __uint_as_float(v[e]));
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const bool ok = (uint32_t)(ch * 32 + e - c_lo) < c_span;
                        tmax = fmaxf(tmax, ok ? __uint_as_float(v[e]) : -INFINITY);
                    }
                }
            }
            const float t2 = tmax * p.scale_log2;
            const bool grow = t2 > m2 + kRescaleThreshold;  // also true for the first finite max
            float alpha = 1.f;
            if (grow) {
                alpha = ex2(m2 - t2);  // 0 when m2 = -inf
                m2 = t2;
                l *= alpha;
            }
            if (i > 0 && __any_sync(0xffffffffu, grow)) {
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

            // pass 2: P = exp2(s * scale_log2 - m), row sum, bf16 P into swizzled shared memory
            float lsum = 0.f;
#pragma unroll 1
            for (int ch = 0; ch < n_chunks; ++ch) {
                uint32_t v[32];
                tmem_ld32(tS + ch * 32, v);
                tc_wait_ld();
                uint32_t packed[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float x0 = fmaf(__uint_as_float(v[e]), p.scale_log2, neg_m);
                    float x1 = fmaf(__uint_as_float(v[e + 1]), p.scale_log2, neg_m);
                    if (!full) {
                        if ((uint32_t)(ch * 32 + e - c_lo) >= c_span) x0 = -INFINITY;
                        if ((uint32_t)(ch * 32 + e + 1 - c_lo) >= c_span) x1 = -INFINITY;
                    }
                    const float p0 = ex2(x0), p1 = ex2(x1);
                    lsum += p0 + p1;
                    __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
                    packed[e >> 1] = *reinterpret_cast<uint32_t *>(&b2);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int c8 = ch * 4 + q;  // 16-byte chunk (8 keys) of the P row
                    const uint32_t addr = sP + (c8 >> 3) * kTileBytes + tid * kRowBytes +
                                          (((c8 & 7) ^ (tid & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr),
                                 "r"(packed[4 * q]), "r"(packed[4 * q + 1]), "r"(packed[4 * q + 2]),
                                 "r"(packed[4 * q + 3])
                                 : "memory");
                }
            }
            l += lsum;

            fence_proxy_async();
            tc_fence_before();
            __syncthreads();  // P written, S reads and O rescale finished

            if (tid == 0) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(128, 64, 0, 1);
                const int n_ks = n16 >> 4;
                for (int ks = 0; ks < n_ks; ++ks)
                    mma_bf16_ss(tmem + 128, smem_desc_sw128(sP + (ks >> 2) * kTileBytes + (ks & 3) * 32),
                                smem_desc_sw128(sV + ks * 16 * kRowBytes), idesc, (i > 0) || (ks > 0));
                mma_commit(bar_pv);
            }
        }

        // epilogue: O / l -> bf16, stored at the row's original position (scatter), LSE
        wait(bar_pv, phase_pv);
        phase_pv ^= 1;
        tc_fence_after();
        const float inv_l = 1.f / l;
        uint32_t outw[32];
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {
            uint32_t o[32];
            tmem_ld32(tO + c2 * 32, o);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[e]) * inv_l,
                                                          __uint_as_float(o[e + 1]) * inv_l);
                outw[c2 * 16 + (e >> 1)] = *reinterpret_cast<uint32_t *>(&b2);
            }
        }
        if (row_valid) {
            uint4 *dst = reinterpret_cast<uint4 *>(p.O + (bh + orig) * 64);
#pragma unroll
            for (int c = 0; c < 8; ++c)
                dst[c] = make_uint4(outw[4 * c], outw[4 * c + 1], outw[4 * c + 2], outw[4 * c + 3]);
            p.LSE[bh + orig] = (m2 + log2f(l)) * 0.6931471805599453f;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

int g_num_sms = 0;
bool g_attr_set = false;

}  // namespace

bool tc_supported(int d, int dtype) { return d == 64 && dtype == MATE_BF16; }

size_t tc_fwd_workspace(const mate_plan_t *, int) { return 0; }

int tc_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, float scale, void *O,
           float *LSE, void *, cudaStream_t stream) {
    if (!(scale > 0.f)) return MATE_ERR_UNSUPPORTED;  // the row max is taken before scaling
    if (plan->n_fwd_units == 0) return MATE_OK;
    if (g_num_sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return MATE_ERR_CUDA;
    }
    if (!g_attr_set) {
        if (cudaFuncSetAttribute(tc_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemBytes) != cudaSuccess)
            return MATE_ERR_CUDA;
        g_attr_set = true;
    }
    Params p;
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
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = plan->status_dev;
    const int grid = plan->n_fwd_units < 2 * g_num_sms ? plan->n_fwd_units : 2 * g_num_sms;
    tc_fwd_kernel<<<grid, kThreads, kSmemBytes, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

}  // namespace mate

// SIMT (no tensor core) kernels: one warp per query row (forward, dQ) or per key row (dK/dV).
// fp32 arithmetic whatever the storage type; this is the debug / any-head-dim path and the
// reference the tensor-core kernels were brought up against on the device.
//
// In a head's view order (see mate_plan) the keys of query row t are
//     [0, P)  u  [max(seg_lo[t], P), seg_hi[t])
// which is the attention pattern A of Section 3 for both table rows (own segment plus prefix) and
// prefix rows (seg_lo = 0, seg_hi = n_valid).  The pattern is symmetric, so the queries that
// attend to key t are the same two ranges; dK/dV therefore need no atomics.
#include <cuda_bf16.h>

#include <mutex>

#include "mate_internal.h"

namespace mate {

namespace {

// Built-in scratch of mate_attn_bwd_noalloc: one float per (example, head, position) for the row
// dots D.  It is part of the library image, so every GPU that loads the library holds these
// 4 MiB until the process exits.
constexpr size_t kNoAllocMaxRows = size_t(1) << 20;
static __device__ __align__(256) float g_noalloc_rowdot[kNoAllocMaxRows];

constexpr int kWarpsPerBlock = 4;
constexpr int kMaxD = 128;
constexpr int kAccPerLane = kMaxD / 32;

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f(float &dst, float x) { dst = x; }
__device__ __forceinline__ void from_f(__nv_bfloat16 &dst, float x) { dst = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T>
__device__ __forceinline__ float dot_row(const float *__restrict__ a_smem, const T *__restrict__ row,
                                         int d) {
    float acc = 0.f;
    for (int e = 0; e < d; ++e) acc = fmaf(a_smem[e], to_f(row[e]), acc);
    return acc;
}

struct RowCtx {
    const int32_t *perm, *seg_lo, *seg_hi;
    int n_valid, view;
};

__device__ __forceinline__ RowCtx row_ctx(const ViewPlan &rowv, const ViewPlan &colv,
                                          const uint8_t *head_view, const int32_t *n_valid, int b,
                                          int h, int N) {
    RowCtx c;
    c.view = head_view[h];
    const ViewPlan &vp = c.view ? colv : rowv;
    c.perm = vp.perm + (size_t)b * N;
    c.seg_lo = vp.seg_lo + (size_t)b * N;
    c.seg_hi = vp.seg_hi + (size_t)b * N;
    c.n_valid = n_valid[b];
    return c;
}

// ---------------------------------------------------------------------------------- forward
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_fwd_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                T *__restrict__ O, float *__restrict__ LSE, ViewPlan rowv, ViewPlan colv,
                const uint8_t *__restrict__ head_view, const int32_t *__restrict__ n_valid, int N,
                const int32_t *__restrict__ prefix, int d, float scale, int view_order, TensorRows tr) {
    __shared__ float s_q[kWarpsPerBlock][kMaxD];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * kWarpsPerBlock + warp;
    const int h = blockIdx.y, b = blockIdx.z;
    if (t >= N) return;
    const RowCtx c = row_ctx(rowv, colv, head_view, n_valid, b, h, N);
    const size_t bh = tr.base(b, h);
    const int k = view_order ? t : c.perm[t];  // view order: the tensors are laid out in the head's own order
    T *o_row = O + (bh + k) * d;
    if (t >= c.n_valid) {  // padding query row
        if (!tr.exists(b, k)) return;  // packed layout: beyond the example's end there is no such row
        for (int e = lane; e < d; e += 32) from_f(o_row[e], 0.f);
        if (lane == 0) LSE[bh + k] = -INFINITY;
        return;
    }
    for (int e = lane; e < d; e += 32) s_q[warp][e] = to_f(Q[(bh + k) * d + e]);
    __syncwarp();

    float m = -INFINITY, l = 0.f, acc[kAccPerLane];
#pragma unroll
    for (int i = 0; i < kAccPerLane; ++i) acc[i] = 0.f;

    const int P = min(prefix[b], c.n_valid);  // length of the global block (never reaches into the padding)
    const int lo = max(c.seg_lo[t], P), hi = c.seg_hi[t];
    for (int range = 0; range < 2; ++range) {
        const int j_begin = range ? lo : 0, j_end = range ? hi : P;
        for (int j0 = j_begin; j0 < j_end; j0 += 32) {
            const int j = j0 + lane;
            const bool on = j < j_end;
            const int kj = on ? (view_order ? j : c.perm[j]) : 0;
            float s = on ? scale * dot_row(s_q[warp], K + (bh + kj) * d, d) : -INFINITY;
            const float m_new = fmaxf(m, warp_max(s));
            const float p = on ? expf(s - m_new) : 0.f;
            const float alpha = expf(m - m_new);  // m = -inf on the first step gives 0
            l = l * alpha + warp_sum(p);
            m = m_new;
#pragma unroll
            for (int i = 0; i < kAccPerLane; ++i) acc[i] *= alpha;
            const int n_here = min(32, j_end - j0);
            for (int jj = 0; jj < n_here; ++jj) {
                const float pj = __shfl_sync(0xffffffffu, p, jj);
                const int vj = __shfl_sync(0xffffffffu, kj, jj);
                const T *v_row = V + (bh + vj) * d;
#pragma unroll
                for (int i = 0; i < kAccPerLane; ++i) {
                    const int e = lane + 32 * i;
                    if (e < d) acc[i] = fmaf(pj, to_f(v_row[e]), acc[i]);
                }
            }
        }
    }
    // a valid row attends at least to itself, except in the passes of the row-or-column pattern,
    // where a row may have no key at all: O = 0, LSE = -inf
    const float inv_l = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int i = 0; i < kAccPerLane; ++i) {
        const int e = lane + 32 * i;
        if (e < d) from_f(o_row[e], acc[i] * inv_l);
    }
    if (lane == 0) LSE[bh + k] = m + logf(l);
}

// ---------------------------------------------------------------------------------- backward
// D_k = sum_e dO_ke O_ke, original token order, one warp per row.
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_rowdot_kernel(const T *__restrict__ dO, const T *__restrict__ O, float *__restrict__ D,
                   size_t rows, int d) {
    const size_t r = (size_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    float acc = 0.f;
    for (int e = lane; e < d; e += 32) acc = fmaf(to_f(dO[r * d + e]), to_f(O[r * d + e]), acc);
    acc = warp_sum(acc);
    if (lane == 0) D[r] = acc;
}

// kDKV = false: the warp owns query row t and produces dQ_t = scale * sum_j dS_tj K_j.
// kDKV = true : the warp owns key row t and produces dV_t = sum_k P_kt dO_k and
//               dK_t = scale * sum_k dS_kt Q_k, looping over the queries k that attend to it.
template <typename T, bool kDKV>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_bwd_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                const T *__restrict__ dO, const float *__restrict__ LSE,
                const float *__restrict__ D, T *__restrict__ dQ, T *__restrict__ dK,
                T *__restrict__ dV, ViewPlan rowv, ViewPlan colv,
                const uint8_t *__restrict__ head_view, const int32_t *__restrict__ n_valid, int N,
                const int32_t *__restrict__ prefix, int d, float scale, TensorRows tr) {
    __shared__ float s_a[kWarpsPerBlock][kMaxD];  // own q (dQ) or own k (dK/dV)
    __shared__ float s_b[kWarpsPerBlock][kMaxD];  // own dO (dQ) or own v (dK/dV)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * kWarpsPerBlock + warp;
    const int h = blockIdx.y, b = blockIdx.z;
    if (t >= N) return;
    const RowCtx c = row_ctx(rowv, colv, head_view, n_valid, b, h, N);
    const size_t bh = tr.base(b, h);
    const int own = c.perm[t];
    T *out0 = (kDKV ? dK : dQ) + (bh + own) * d;
    T *out1 = kDKV ? dV + (bh + own) * d : nullptr;
    if (t >= c.n_valid) {
        if (!tr.exists(b, own)) return;  // packed layout: beyond the example's end there is no such row
        for (int e = lane; e < d; e += 32) {
            from_f(out0[e], 0.f);
            if (kDKV) from_f(out1[e], 0.f);
        }
        return;
    }
    const T *a_src = (kDKV ? K : Q) + (bh + own) * d;
    const T *b_src = (kDKV ? V : dO) + (bh + own) * d;
    for (int e = lane; e < d; e += 32) {
        s_a[warp][e] = to_f(a_src[e]);
        s_b[warp][e] = to_f(b_src[e]);
    }
    __syncwarp();
    float own_lse = 0.f, own_D = 0.f;
    if (!kDKV) {
        own_lse = LSE[bh + own];
        own_D = D[bh + own];
    }
    float acc0[kAccPerLane], acc1[kAccPerLane];
#pragma unroll
    for (int i = 0; i < kAccPerLane; ++i) acc0[i] = acc1[i] = 0.f;

    const int P = min(prefix[b], c.n_valid);  // length of the global block (never reaches into the padding)
    const int lo = max(c.seg_lo[t], P), hi = c.seg_hi[t];
    for (int range = 0; range < 2; ++range) {
        const int j_begin = range ? lo : 0, j_end = range ? hi : P;
        for (int j0 = j_begin; j0 < j_end; j0 += 32) {
            const int j = j0 + lane;
            const bool on = j < j_end;
            const int oj = on ? c.perm[j] : 0;  // original index of the other row
            float p = 0.f, ds = 0.f;
            if (on) {
                // dQ: other row is a key  -> s = q_own . k_other, dP = dO_own . v_other
                // dKV: other row is a query -> s = q_other . k_own, dP = dO_other . v_own
                const T *x = (kDKV ? Q : K) + (bh + oj) * d;
                const T *y = (kDKV ? dO : V) + (bh + oj) * d;
                const float s = scale * dot_row(s_a[warp], x, d);
                const float dp = dot_row(s_b[warp], y, d);
                const float lse = kDKV ? LSE[bh + oj] : own_lse;
                const float Dk = kDKV ? D[bh + oj] : own_D;
                p = expf(s - lse);
                ds = p * (dp - Dk);
            }
            const int n_here = min(32, j_end - j0);
            for (int jj = 0; jj < n_here; ++jj) {
                const float pj = __shfl_sync(0xffffffffu, p, jj);
                const float dsj = __shfl_sync(0xffffffffu, ds, jj) * scale;
                const int rj = __shfl_sync(0xffffffffu, oj, jj);
                const T *x = (kDKV ? Q : K) + (bh + rj) * d;   // dK += ds q ; dQ += ds k
                const T *y = dO + (bh + rj) * d;               // dV += p dO
#pragma unroll
                for (int i = 0; i < kAccPerLane; ++i) {
                    const int e = lane + 32 * i;
                    if (e < d) {
                        acc0[i] = fmaf(dsj, to_f(x[e]), acc0[i]);
                        if (kDKV) acc1[i] = fmaf(pj, to_f(y[e]), acc1[i]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kAccPerLane; ++i) {
        const int e = lane + 32 * i;
        if (e < d) {
            from_f(out0[e], acc0[i]);
            if (kDKV) from_f(out1[e], acc1[i]);
        }
    }
}

template <typename T>
int simt_fwd_t(const mate_plan_t *pl, const void *Q, const void *K, const void *V, int d, float scale,
               void *O, float *LSE, int view_order, cudaStream_t st) {
    dim3 grid((pl->N + kWarpsPerBlock - 1) / kWarpsPerBlock, pl->H, pl->B);
    simt_fwd_kernel<T><<<grid, kWarpsPerBlock * 32, 0, st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (T *)O, LSE, pl->view[0], pl->view[1],
        pl->head_view_dev, pl->n_valid_dev, pl->N, pl->global_dev, d, scale, view_order, pl->rows());
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

template <typename T>
int simt_bwd_t(const mate_plan_t *pl, const void *Q, const void *K, const void *V, const void *O,
               const float *LSE, const void *dO, int d, float scale, void *dQ, void *dK, void *dV,
               void *ws, cudaStream_t st) {
    float *D = (float *)ws;
    const size_t rows = pl->n_rows();
    simt_rowdot_kernel<T><<<(unsigned)((rows + kWarpsPerBlock - 1) / kWarpsPerBlock),
                            kWarpsPerBlock * 32, 0, st>>>((const T *)dO, (const T *)O, D, rows, d);
    dim3 grid((pl->N + kWarpsPerBlock - 1) / kWarpsPerBlock, pl->H, pl->B);
    simt_bwd_kernel<T, false><<<grid, kWarpsPerBlock * 32, 0, st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, LSE, D, (T *)dQ, (T *)dK, (T *)dV,
        pl->view[0], pl->view[1], pl->head_view_dev, pl->n_valid_dev, pl->N, pl->global_dev, d, scale, pl->rows());
    simt_bwd_kernel<T, true><<<grid, kWarpsPerBlock * 32, 0, st>>>(
        (const T *)Q, (const T *)K, (const T *)V, (const T *)dO, LSE, D, (T *)dQ, (T *)dK, (T *)dV,
        pl->view[0], pl->view[1], pl->head_view_dev, pl->n_valid_dev, pl->N, pl->global_dev, d, scale, pl->rows());
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

}  // namespace

int simt_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d, int dtype,
             float scale, void *O, float *LSE, unsigned flags, cudaStream_t stream) {
    if (d > kMaxD) return MATE_ERR_UNSUPPORTED;
    const int vo = (flags & MATE_FLAG_VIEW_ORDER) ? 1 : 0;
    return dtype == MATE_F32 ? simt_fwd_t<float>(plan, Q, K, V, d, scale, O, LSE, vo, stream)
                             : simt_fwd_t<__nv_bfloat16>(plan, Q, K, V, d, scale, O, LSE, vo, stream);
}

size_t simt_bwd_workspace(const mate_plan_t *plan) {
    return sizeof(float) * (size_t)plan->B * plan->H * plan->N;
}

int simt_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
             const float *LSE, const void *dO, int d, int dtype, float scale, void *dQ, void *dK,
             void *dV, void *workspace, cudaStream_t stream) {
    if (d > kMaxD) return MATE_ERR_UNSUPPORTED;
    return dtype == MATE_F32
               ? simt_bwd_t<float>(plan, Q, K, V, O, LSE, dO, d, scale, dQ, dK, dV, workspace, stream)
               : simt_bwd_t<__nv_bfloat16>(plan, Q, K, V, O, LSE, dO, d, scale, dQ, dK, dV,
                                           workspace, stream);
}

}  // namespace mate

// Allocation-free backward (see mate.h).  The name g_noalloc_rowdot is only a host-side handle
// here; the address the kernels need comes from cudaGetSymbolAddress, looked up once per device
// with that device current.
extern "C" int mate_attn_bwd_noalloc(const mate_plan_t *plan, const void *Q, const void *K,
                                     const void *V, const void *O, const float *LSE,
                                     const void *dO, int d, int dtype, float scale, void *dQ,
                                     void *dK, void *dV, void *stream) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static float *scratch_of_device[kMaxDevices] = {};

    if (!plan || !Q || !K || !V || !O || !LSE || !dO || !dQ || !dK || !dV) return MATE_ERR_INVALID_ARG;
    if (dtype != MATE_BF16 && dtype != MATE_F32) return MATE_ERR_UNSUPPORTED;
    if (d <= 0 || d % 8 != 0 || d > mate::kMaxD) return MATE_ERR_UNSUPPORTED;
    const void *ptrs[] = {Q, K, V, O, LSE, dO, dQ, dK, dV};
    for (const void *p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) & 15u) return MATE_ERR_ALIGNMENT;
    if (plan->sub[0]) return MATE_ERR_UNSUPPORTED;  // row-or-column plans need the three-pass path
    const size_t rows = (size_t)plan->B * plan->H * plan->N;
    if (rows > mate::kNoAllocMaxRows) return MATE_ERR_TOO_LARGE;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MATE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MATE_ERR_UNSUPPORTED;
    if (dev != plan->device) return MATE_ERR_INVALID_ARG;  // the plan's arrays live on another device
    float *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!scratch_of_device[dev]) {
            float *p = nullptr;
            if (cudaGetSymbolAddress((void **)&p, mate::g_noalloc_rowdot) != cudaSuccess || !p)
                return MATE_ERR_CUDA;
            scratch_of_device[dev] = p;
        }
        scratch = scratch_of_device[dev];
    }
    // every element of D that the backward kernels read is written by the row-dot kernel of the
    // same call first, so nothing in the shared array has to start at zero
    return mate::simt_bwd(plan, Q, K, V, O, LSE, dO, d, dtype, scale, dQ, dK, dV, scratch,
                          (cudaStream_t)stream);
}

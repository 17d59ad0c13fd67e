// Per-cell mean of token logits (cell-selection stage, Section 4.1: S(c) = avg over the tokens t of
// cell c of S(t)).  A cell is the set of table tokens that share a (row id, column id) pair.  In the
// row view of the plan the tokens of one row are contiguous, so one warp takes one row: it reads
// the row's (column id, logit) pairs 32 at a time, coalesced through the view order, and every lane
// accumulates the cells of the columns lane, lane + 32, ... in the order of the tokens (the result
// does not depend on the launch).  HBM-bound by design: every id and logit is read once.
#include "mate_internal.h"

namespace mate {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kColsPerLane = 4;  // columns handled per pass: 32 * kColsPerLane

__global__ void __launch_bounds__(32 * kWarpsPerBlock)
cell_mean_kernel(const float *__restrict__ logits, const int32_t *__restrict__ col_ids, ViewPlan rowv, int N,
                 int n_rows, int n_cols, float *__restrict__ mean, int32_t *__restrict__ count) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);  // row id
    const int b = blockIdx.y;
    if (r >= n_rows) return;
    const int32_t *seg_off = rowv.seg_off + (size_t)b * (rowv.max_id + 2);
    const int32_t *perm = rowv.perm + (size_t)b * N;
    const int lo = seg_off[r], hi = seg_off[r + 1];
    float *out_m = mean + ((size_t)b * n_rows + r) * n_cols;
    int32_t *out_c = count ? count + ((size_t)b * n_rows + r) * n_cols : nullptr;

    for (int c0 = 0; c0 < n_cols; c0 += 32 * kColsPerLane) {
        float sum[kColsPerLane];
        int cnt[kColsPerLane];
#pragma unroll
        for (int q = 0; q < kColsPerLane; ++q) {
            sum[q] = 0.f;
            cnt[q] = 0;
        }
        for (int t0 = lo; t0 < hi; t0 += 32) {
            const int t = t0 + lane;
            int c = -1;
            float x = 0.f;
            if (t < hi) {
                const int orig = perm[t];
                c = col_ids[(size_t)b * N + orig];
                x = logits[(size_t)b * N + orig];
            }
            const int n = min(32, hi - t0);
            for (int j = 0; j < n; ++j) {
                const int cj = __shfl_sync(0xffffffffu, c, j) - c0 - lane;
                const float xj = __shfl_sync(0xffffffffu, x, j);
#pragma unroll
                for (int q = 0; q < kColsPerLane; ++q)
                    if (cj == 32 * q) {
                        sum[q] += xj;
                        ++cnt[q];
                    }
            }
        }
#pragma unroll
        for (int q = 0; q < kColsPerLane; ++q) {
            const int c = c0 + 32 * q + lane;
            if (c < n_cols) {
                out_m[c] = cnt[q] ? sum[q] / (float)cnt[q] : 0.f;
                if (out_c) out_c[c] = cnt[q];
            }
        }
    }
}

}  // namespace
}  // namespace mate

extern "C" int mate_cell_mean(const mate_plan_t *plan, const float *logits, const int32_t *col_ids, float *mean,
                              int32_t *count, void *stream) {
    if (!plan || !logits || !col_ids || !mean) return MATE_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MATE_ERR_CUDA;
    if (dev != plan->device) return MATE_ERR_INVALID_ARG;
    if (plan->T) return MATE_ERR_UNSUPPORTED;  // packed batches: not here
    const int n_rows = plan->view[0].max_id + 1, n_cols = plan->view[1].max_id + 1;
    dim3 grid((n_rows + mate::kWarpsPerBlock - 1) / mate::kWarpsPerBlock, plan->B);
    mate::cell_mean_kernel<<<grid, 32 * mate::kWarpsPerBlock, 0, (cudaStream_t)stream>>>(
        logits, col_ids, plan->view[0], plan->N, n_rows, n_cols, mean, count);
    return cudaGetLastError() == cudaSuccess ? MATE_OK : MATE_ERR_CUDA;
}

// Glue kernels of the head-independent row-or-column pattern (the pattern the paper describes for
// its closest comparison system, Section 2): the attention of a row is computed in three passes over
// disjoint key sets by the ordinary kernels; here their outputs are merged (each pass returns a
// normalised O and the logsumexp of its own keys) and their gradients summed.  HBM-bound,
// element-wise work.
#include <cuda_bf16.h>

#include "mate_internal.h"

namespace mate {
namespace {

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f(float &dst, float x) { dst = x; }
__device__ __forceinline__ void from_f(__nv_bfloat16 &dst, float x) { dst = __float2bfloat16_rn(x); }

// One warp per row.  O <- sum_i w_i O_i with w_i = exp(LSE_i - LSE), LSE = log sum_i exp(LSE_i); a pass
// in which the row has no key returns LSE_i = -inf and weighs 0.  O, LSE hold pass 0 on entry.
template <typename T>
__global__ void merge_kernel(T *__restrict__ O, float *__restrict__ LSE, const T *__restrict__ O1,
                             const float *__restrict__ LSE1, const T *__restrict__ O2, const float *__restrict__ LSE2,
                             size_t rows, int d) {
    const size_t r = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float a = LSE[r], b = LSE1[r], c = LSE2[r];
    const float m = fmaxf(a, fmaxf(b, c));
    if (m == -INFINITY) return;  // padding row: pass 0 has written O = 0, LSE = -inf
    const float wa = __expf(a - m), wb = __expf(b - m), wc = __expf(c - m);
    const float inv = 1.f / (wa + wb + wc);
    for (int e = lane; e < d; e += 32) {
        const size_t i = r * d + e;
        from_f(O[i], (wa * to_f(O[i]) + wb * to_f(O1[i]) + wc * to_f(O2[i])) * inv);
    }
    if (lane == 0) LSE[r] = m + logf(wa + wb + wc);
}

template <typename T>
__global__ void add3_kernel(T *__restrict__ a, const T *__restrict__ b, const T *__restrict__ c, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) from_f(a[i], to_f(a[i]) + to_f(b[i]) + to_f(c[i]));
}

}  // namespace

cudaError_t launch_merge_passes(void *O, float *LSE, const void *O1, const float *LSE1, const void *O2, const float *LSE2,
                                size_t rows, int d, int dtype, cudaStream_t stream) {
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    if (dtype == MATE_F32)
        merge_kernel<float><<<blocks, 256, 0, stream>>>((float *)O, LSE, (const float *)O1, LSE1, (const float *)O2, LSE2,
                                                        rows, d);
    else
        merge_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>((__nv_bfloat16 *)O, LSE, (const __nv_bfloat16 *)O1, LSE1,
                                                                (const __nv_bfloat16 *)O2, LSE2, rows, d);
    return cudaGetLastError();
}

cudaError_t launch_add3(void *a, const void *b, const void *c, size_t n, int dtype, cudaStream_t stream) {
    const unsigned blocks = (unsigned)((n + 255) / 256);
    if (dtype == MATE_F32)
        add3_kernel<float><<<blocks, 256, 0, stream>>>((float *)a, (const float *)b, (const float *)c, n);
    else
        add3_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>((__nv_bfloat16 *)a, (const __nv_bfloat16 *)b,
                                                               (const __nv_bfloat16 *)c, n);
    return cudaGetLastError();
}

}  // namespace mate

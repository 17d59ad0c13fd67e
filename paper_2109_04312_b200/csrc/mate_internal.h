// Internal declarations shared by the libmate translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "mate.h"

namespace mate {

constexpr int kTile = 128;       // key columns per tile and query rows per half of a unit
constexpr int kSchedWords = 8;   // scheduling counters in front of the split-unit counters
constexpr int kUnitRows = 256;   // query rows per unit of the tensor-core kernels (two halves)
// what the key range of a table row is made of (plan kernel step 4 and its host twin)
enum { kBoundsOwn = 0, kBoundsBefore = 1, kBoundsAfter = 2 };
constexpr int kTraceCtas = 256;  // CTAs whose cycle counters a -DMATE_TRACE build keeps

// One unit of work of the tensor-core forward: up to 256 consecutive query rows (view order) of one
// (example, head) -- half 0 = the first 128 rows, half 1 = the rest -- and the key tiles (128 wide)
// they visit, in this order:
//   range A = keys [kA0, kA_end): the prefix block for table rows ([0, P)), a slice of all valid
//             keys for prefix rows.  Key j counts for every row iff j < kA_end.
//   range B = keys [kB0, kB_end): the union of the segments the rows belong to (table rows only).
//             Key j counts for a row iff seg_lo[row] <= j < seg_hi[row]; half h touches only the
//             tiles that meet [lo[h], hi[h]) (min seg_lo / max seg_hi over its rows).
// Prefix rows whose key range is long are split along the keys into n_parts units; each writes an
// un-normalised partial result to the workspace at ws_off (KiB); per group of 32 rows the part
// that finishes last (counted in counters[kSchedWords + 8 * ctr + row / 32]) combines them.
struct FwdUnit {
    int32_t b, h;
    int32_t q0, nq;
    int32_t kA0, kA_end;
    int32_t kB0, kB_end;
    int32_t lo[2], hi[2];
    int32_t n_parts, part;
    int32_t ws_off, ctr;
};
static_assert(sizeof(FwdUnit) == 64, "FwdUnit is read as four 16-byte words");
// bytes of one partial result: 256 rows x (64 fp32 + running max + row sum)
constexpr size_t kPartialBytes = (size_t)kUnitRows * (64 + 2) * sizeof(float);

// Where the rows of example b, head h start in the caller's tensors (in rows of d elements), and how
// far an example reaches.  Padded layout [B, H, N, d]: (b H + h) N, every example N positions long.
// Packed layout [H, T, d] (mate_plan_packed: the examples one behind the other, no padding between
// them): h T + tok_off[b], example b being len[b] positions long; positions at and beyond len[b] of
// the plan's padded view of the example do not exist in the tensors and are never written.
struct TensorRows {
    const int32_t *tok_off = nullptr;  // device [B]; null = padded layout
    const int32_t *len = nullptr;      // device [B]; null = padded layout
    int H = 0, N = 0, T = 0;
#ifdef __CUDACC__
    __device__ __forceinline__ size_t base(int b, int h) const {
        return tok_off ? (size_t)h * T + tok_off[b] : ((size_t)b * H + h) * N;
    }
    __device__ __forceinline__ bool exists(int b, int pos) const { return !len || pos < len[b]; }
#endif
};

struct ViewPlan {
    int32_t *perm = nullptr;      // [B, N]   view position -> original position
    int32_t *inv_perm = nullptr;  // [B, N]
    int32_t *seg_off = nullptr;   // [B, max_id + 2]
    int32_t *seg_lo = nullptr;    // [B, N]   per view position: first key of its own segment (bucketed
                                  //          plans: of the part of it within the adjacent buckets)
    int32_t *seg_hi = nullptr;    // [B, N]   one past the last key (prefix rows: n_valid; padding: 0)
    int32_t *cursor = nullptr;    // [B, max_id + 2] scratch of the counting sort
    int32_t *ident = nullptr;     // [B]      number of leading view positions t with perm[t] = t
    int max_id = 0;
    int n_heads = 0;
};

}  // namespace mate

struct mate_plan_s {
    int B = 0, N = 0, H = 0;
    int device = 0;                      // ordinal of the device the plan's arrays live on
    std::vector<int32_t> prefix;         // |Q| per example (host copy)
    int32_t *prefix_dev = nullptr;       // [B]
    // Length of the global block per example: the positions [0, G) of a head's order that see and are
    // seen by everything.  G = |Q| except for a bucketed plan with a longer global section.  This, not
    // |Q|, is what the attention kernels and the work-lists use; |Q| only decides the order.
    std::vector<int32_t> global;
    int32_t *global_dev = nullptr;       // [B]
    int radius = 0;                      // > 0: bucketed pattern (Section 3.1), buckets of this many positions
    int bounds_mode = 0, group = 1;      // key range of a table row (kBounds*), ids per group
    // row-or-column pattern (mate_plan_sat): this plan is the row pass; sub[0] / sub[1] are the passes
    // over the rest of the token's column in front of / behind its own cell
    mate_plan_s *sub[2] = {nullptr, nullptr};
    int32_t *pair_ids_dev = nullptr;     // ids of the sub-plans (owned by the main plan)
    // packed layout (mate_plan_packed): start and length of every example on the common token axis
    int T = 0;                           // total tokens; 0 = padded layout
    int32_t *tok_off_dev = nullptr, *len_dev = nullptr;  // [B] each (one allocation, owned by the plan)
    mate::TensorRows rows() const {
        mate::TensorRows r;
        r.tok_off = tok_off_dev;
        r.len = len_dev;
        r.H = H;
        r.N = N;
        r.T = T;
        return r;
    }
    size_t n_rows() const { return T ? (size_t)H * T : (size_t)B * H * N; }  // rows of a [.., d] tensor
    std::vector<uint8_t> head_view;      // host copy
    uint8_t *head_view_dev = nullptr;    // [H]
    mate::ViewPlan view[2];
    int32_t *n_valid_dev = nullptr;      // [B]
    std::vector<int32_t> n_valid;        // host copy
    std::vector<int64_t> pairs;          // [B, 2] unmasked pairs per example and view
    int32_t *status_dev = nullptr;       // device status word(s): [0] = id validation, [1] = kernel timeouts
    void *dev_block = nullptr;           // one allocation backing all device arrays above
    void *work_block = nullptr;          // one allocation backing the work-lists below
    // tensor-core forward work-list: units by decreasing cost; the CTAs of the persistent kernel
    // take them in this order through a shared counter
    mate::FwdUnit *fwd_units_dev = nullptr;
    // [kSchedWords + 8 * n_fwd_slots]: [0] next unit, [1] CTAs finished, then the arrival counters of
    // the split units.  Zero between launches (the kernel resets what it counted), which is why
    // two forward calls on one plan must not overlap on the GPU.
    int32_t *fwd_counters_dev = nullptr;
    int n_fwd_units = 0;
    int n_fwd_slots = 0;                  // split units (prefix rows cut along the keys)
    int n_ctas = 0;                       // CTAs of the persistent kernel (SMs of the plan's device)
    size_t fwd_ws_bytes = 0;              // partial results of the split units
    std::vector<mate::FwdUnit> fwd_units; // host copy
    // tensor-core backward work-list: the same units with no prefix unit split
    mate::FwdUnit *bwd_units_dev = nullptr;
    int n_bwd_units = 0;
    std::vector<mate::FwdUnit> bwd_units;
};

namespace mate {

// Raises a kernel's dynamic shared-memory limit once per device.  cudaFuncSetAttribute acts on the
// device that is current when it is called, so the "already done" flags are kept per device ordinal
// (under a mutex: host threads may drive different devices at the same time).
struct SmemAttrOnce {
    static constexpr int kMaxDevices = 64;
    std::mutex mu;
    bool done[kMaxDevices] = {};
    // returns MATE_OK or MATE_ERR_CUDA; `device` is the current device
    int ensure(const void *kernel, int bytes, int device) {
        std::lock_guard<std::mutex> lock(mu);
        if (device >= 0 && device < kMaxDevices && done[device]) return MATE_OK;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
            return MATE_ERR_CUDA;
        if (device >= 0 && device < kMaxDevices) done[device] = true;
        return MATE_OK;
    }
};

// plan kernels (mate_plan_kernels.cu)
cudaError_t launch_plan_kernels(const int32_t *row_ids, const int32_t *col_ids, int B, int N,
                                const int32_t *prefix /* device [B] */, const int32_t *global_len /* device [B] */,
                                int radius, int bounds_mode, int group,
                                const ViewPlan &rowv, const ViewPlan &colv, int32_t *n_valid, int32_t *status,
                                cudaStream_t stream);
cudaError_t launch_unpack_ids(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *tok_off,
                              const int32_t *len, int32_t *rows_out, int32_t *cols_out, cudaStream_t stream);
cudaError_t launch_pair_ids(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix,
                            int n_row_ids, int32_t *out, cudaStream_t stream);

// row-or-column pattern (mate_sat.cu): merge of the passes' outputs, sum of their gradients
cudaError_t launch_merge_passes(void *O, float *LSE, const void *O1, const float *LSE1, const void *O2, const float *LSE2,
                                size_t rows, int d, int dtype, cudaStream_t stream);
cudaError_t launch_add3(void *a, const void *b, const void *c, size_t n, int dtype, cudaStream_t stream);

// SIMT kernels (mate_simt.cu)
int simt_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d, int dtype,
             float scale, void *O, float *LSE, unsigned flags, cudaStream_t stream);
size_t simt_bwd_workspace(const mate_plan_t *plan);
int simt_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
             const float *LSE, const void *dO, int d, int dtype, float scale, void *dQ, void *dK,
             void *dV, void *workspace, cudaStream_t stream);

// tensor-core kernels (mate_fwd_tc.cu / mate_bwd_tc.cu)
bool tc_supported(int d, int dtype);
int tc_fwd_ctas_per_sm();  // CTAs of the forward kernel per SM (the grid is this times the plan's SM count)
size_t tc_fwd_workspace(const mate_plan_t *plan, int d);
size_t tc_bwd_workspace(const mate_plan_t *plan);
int tc_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
           const float *LSE, const void *dO, float scale, void *dQ, void *dK, void *dV, void *workspace,
           cudaStream_t stream);
int tc_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, float scale, void *O,
           float *LSE, void *workspace, unsigned flags, cudaStream_t stream);

}  // namespace mate

// Optional cycle counters (compile with -DMATE_TRACE): clock64() time spent in marked regions of
// the tensor-core kernels, per CTA and role, in a local array `tr`.  Profiling aid only; compiled
// out of the library.
#ifdef MATE_TRACE
#define TR_T0(var) const long long var = clock64()
#define TR_ADD(cat, var) tr[cat] += clock64() - (var)
#define TR_INC(cat) tr[cat] += 1
#else
#define TR_T0(var)
#define TR_ADD(cat, var)
#define TR_INC(cat)
#endif

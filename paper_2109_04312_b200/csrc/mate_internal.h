// Internal declarations shared by the libmate translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "mate.h"

namespace mate {

constexpr int kTile = 128;  // query rows and key columns per tile of the tensor-core kernels

// One unit of forward work for the tensor-core kernel: up to 128 consecutive query rows (view
// order) of one (example, head) and the key tiles they visit.  Key tiles are up to 128 wide.
//   range A = keys [0, kA_end): the prefix block for table rows (kA_end = P), every valid key for
//             prefix rows (kA_end = n_valid).  Inside it a key j counts iff j < kA_end.
//   range B = keys [kB0, kB_end): the union of the segments the query rows belong to (table rows
//             only, kB0 >= P).  Inside it key j counts for a row iff seg_lo[row] <= j < seg_hi[row].
struct FwdUnit {
    int32_t b, h;
    int32_t q0, nq;        // first query row (view order) and number of rows (<= 128)
    int32_t kA_end, kA_n;  // range A: end key and number of 128-key tiles
    int32_t kB0, kB_end;   // range B: first and end key
    int32_t kB_n;          // range B: number of tiles
    int32_t part, n_parts; // split-key bookkeeping: this unit is part `part` of `n_parts`
    int32_t slot;          // partial-result slot in the workspace when n_parts > 1, else -1
    int32_t cost;          // key tiles visited (sort key, largest first)
    int32_t pad_[3];
};
static_assert(sizeof(FwdUnit) == 64, "FwdUnit is read as four 16-byte words");

struct ViewPlan {
    int32_t *perm = nullptr;      // [B, N]   view position -> original position
    int32_t *inv_perm = nullptr;  // [B, N]
    int32_t *seg_off = nullptr;   // [B, max_id + 2]
    int32_t *seg_lo = nullptr;    // [B, N]   per view position: first key of its own segment
    int32_t *seg_hi = nullptr;    // [B, N]   one past the last key (prefix rows: n_valid; padding: 0)
    int32_t *cursor = nullptr;    // [B, max_id + 2] scratch of the counting sort
    int max_id = 0;
    int n_heads = 0;
};

}  // namespace mate

struct mate_plan_s {
    int B = 0, N = 0, P = 0, H = 0;
    std::vector<uint8_t> head_view;      // host copy
    uint8_t *head_view_dev = nullptr;    // [H]
    mate::ViewPlan view[2];
    int32_t *n_valid_dev = nullptr;      // [B]
    std::vector<int32_t> n_valid;        // host copy
    std::vector<int64_t> pairs;          // [B, 2] unmasked pairs per example and view
    int32_t *status_dev = nullptr;       // device status word(s): [0] = id validation, [1] = kernel timeouts
    void *dev_block = nullptr;           // one allocation backing all device arrays above
    // tensor-core forward work-list
    mate::FwdUnit *fwd_units_dev = nullptr;
    int n_fwd_units = 0;
    int n_fwd_slots = 0;                 // partial-result slots (split prefix rows)
    std::vector<mate::FwdUnit> fwd_units; // host copy (combine pass bookkeeping)
    mate::FwdUnit *bwd_units_dev = nullptr;
    int n_bwd_units = 0;
    int n_bwd_slots = 0;
};

namespace mate {

// plan kernels (mate_plan_kernels.cu)
cudaError_t launch_plan_kernels(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int P,
                                const ViewPlan &rowv, const ViewPlan &colv, int32_t *n_valid,
                                int32_t *status, cudaStream_t stream);

// SIMT kernels (mate_simt.cu)
int simt_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d, int dtype,
             float scale, void *O, float *LSE, cudaStream_t stream);
size_t simt_bwd_workspace(const mate_plan_t *plan);
int simt_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, const void *O,
             const float *LSE, const void *dO, int d, int dtype, float scale, void *dQ, void *dK,
             void *dV, void *workspace, cudaStream_t stream);

// tensor-core kernels (mate_fwd_tc.cu / mate_bwd_tc.cu)
bool tc_supported(int d, int dtype);
size_t tc_fwd_workspace(const mate_plan_t *plan, int d);
int tc_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, float scale, void *O,
           float *LSE, void *workspace, cudaStream_t stream);

}  // namespace mate

// Per-view token order (Section 3.1: every head traverses the table in its own row order or
// column order, which depends on the input but not on chance): a stable counting sort of the
// positions by (prefix, table id, padding).  One CTA per (example, view); integer work only.
#include "mate_internal.h"

namespace mate {

namespace {

constexpr int kPlanThreads = 1024;
constexpr int kPlanWarps = kPlanThreads / 32;
constexpr int kSmemIds = 2048;    // id tables up to this many entries live in shared memory ...
constexpr int kSmemHist = 8192;   // ... and so do the per-slice tables of the scatter (slices x ids entries)

__device__ __forceinline__ int warp_inclusive_scan(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t *__restrict__ row_ids, const int32_t *__restrict__ col_ids, int N,
            const int32_t *__restrict__ prefix, const int32_t *__restrict__ global_len, int radius, int bounds_mode,
            int group,
            ViewPlan rowv, ViewPlan colv, int32_t *__restrict__ n_valid_out,
            int32_t *__restrict__ status) {
    __shared__ int32_t s_tot[kSmemIds];
    __shared__ int32_t s_hist[kSmemHist];
    __shared__ int s_n_valid;

    const int b = blockIdx.x, view = blockIdx.y;
    const int P = prefix[b];  // |Q| of this example
    const ViewPlan &vp = view ? colv : rowv;
    const int32_t *ids = (view ? col_ids : row_ids) + (size_t)b * N;
    const int32_t *oth = (view ? row_ids : col_ids) + (size_t)b * N;
    const int S = vp.max_id + 2;  // one slot per id and one behind them, which counts the padding
    int32_t *seg_off = vp.seg_off + (size_t)b * S;
    int32_t *perm = vp.perm + (size_t)b * N;
    int32_t *inv_perm = vp.inv_perm + (size_t)b * N;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // The positions are cut into W slices of L consecutive positions (a multiple of 32), one warp
    // per slice in the scatter; every slice has its own table of S cursors.  With one slice the
    // table is the id table itself (shared memory, or global memory when there are many ids).
    const int W = (S <= kSmemIds) ? max(1, min(kPlanWarps, kSmemHist / S)) : 1;
    const int L = ((N + W - 1) / W + 31) & ~31;
    volatile int32_t *tot = (S <= kSmemIds) ? s_tot : (vp.cursor + (size_t)b * S);
    volatile int32_t *hist = (W > 1) ? s_hist : tot;

    for (int i = tid; i < S; i += kPlanThreads) tot[i] = 0;
    if (W > 1)
        for (int i = tid; i < W * S; i += kPlanThreads) hist[i] = 0;
    __syncthreads();

    // A position is a table token iff it lies behind the prefix and both ids are valid; anything
    // else behind the prefix is treated as padding so that every later index stays in range even
    // when the input breaks the conventions (which is reported through `status`).
    auto is_table = [&](int k) {
        int id = ids[k];
        return k >= P && id >= 0 && id <= vp.max_id && oth[k] >= 0;
    };

    // 1. validate + per-slice histogram of the table ids (padding counts under the last slot)
    bool bad = false;
    for (int k = tid; k < N; k += kPlanThreads) {
        int id = ids[k], o = oth[k];
        int slot = -1;
        if (k < P) {
            bad |= (id != 0) | (o != 0);
        } else if (id < 0) {
            bad |= (o >= 0);
            slot = S - 1;
        } else if (o < 0 || id > vp.max_id) {
            bad = true;
            slot = S - 1;
        } else {
            slot = id;
        }
        if (slot >= 0) atomicAdd((int *)&hist[(k / L) * S + slot], 1);
    }
    if (bad) atomicOr(status, 1);
    __syncthreads();
    if (W > 1) {
        for (int i = tid; i < S; i += kPlanThreads) {
            int sum = 0;
            for (int w = 0; w < W; ++w) sum += hist[w * S + i];
            tot[i] = sum;
        }
        __syncthreads();
    }

    // 2. exclusive scan of the id counts -> segment offsets (warp 0, 32 entries per step); the
    //    padding slot is left out of the sums and so receives the number of valid positions
    if (warp == 0) {
        int carry = P;
        for (int base = 0; base < S; base += 32) {
            int i = base + lane;
            int c = (i < S - 1) ? tot[i] : 0;
            int incl = warp_inclusive_scan(c, lane);
            int excl = carry + incl - c;
            if (i < S) {
                seg_off[i] = excl;
                tot[i] = excl;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            s_n_valid = carry;
            if (view == 0) n_valid_out[b] = carry;
        }
    }
    __syncthreads();
    const int n_valid = s_n_valid;
    if (W > 1) {  // cursor of (slice, id): the id's offset plus what the slices in front hold of it
        for (int i = tid; i < S; i += kPlanThreads) {
            int run = tot[i];
            for (int w = 0; w < W; ++w) {
                const int c = hist[w * S + i];
                hist[w * S + i] = run;
                run += c;
            }
        }
        __syncthreads();
    }

    // 3. stable scatter: one warp per slice walks its positions in order, 32 at a time; lanes
    //    holding the same id are ranked by lane, so equal ids keep their original order
    if (warp < W) {
        volatile int32_t *cur = hist + warp * S;
        const int k_end = min(N, (warp + 1) * L);
        for (int base = warp * L; base < k_end; base += 32) {
            int k = base + lane;
            bool in = k < N;
            bool table = in && is_table(k);
            bool padding = in && !table && k >= P;
            int slot = table ? ids[k] : S - 1;
            bool counted = table || padding;
            int key = counted ? slot : (int)0x80000000 + lane;
            unsigned grp = __match_any_sync(0xffffffffu, key);
            int rank = __popc(grp & ((1u << lane) - 1u));
            int cnt = __popc(grp);
            int basep = 0;
            if (counted) basep = cur[slot];
            __syncwarp();
            if (counted && rank == 0) cur[slot] = basep + cnt;
            __syncwarp();
            int pos = counted ? basep + rank : k;  // prefix tokens keep their positions
            if (in) {
                perm[pos] = k;
                inv_perm[k] = pos;
            }
        }
    }
    __syncthreads();

    // 3b. how many leading positions of the order are in place (perm[t] = t for every t below): rows
    //     there are contiguous in the caller's tensors, which lets the attention kernels fetch whole
    //     tiles with one bulk tensor copy instead of row-by-row gathers
    {
        __shared__ int s_ident;
        if (tid == 0) s_ident = N;
        __syncthreads();
        int first_moved = N;
        for (int t = tid; t < N; t += kPlanThreads)
            if (perm[t] != t) first_moved = min(first_moved, t);
        if (first_moved < N) atomicMin(&s_ident, first_moved);
        __syncthreads();
        if (tid == 0) vp.ident[b] = s_ident;
    }

    // 4. per view position: its key range.  Normally its own segment; for the passes of the
    //    row-or-column pattern, whose ids are (column, row) pairs in groups of `group` ids per
    //    column, the segments of its group in front of / behind its own.  With a radius (the bucketed form of
    //    Section 3.1: the order behind the prefix is cut into buckets of `radius` positions and a
    //    token sees its own bucket and the two next to it) the range is clipped to those buckets.
    int32_t *seg_lo = vp.seg_lo + (size_t)b * N, *seg_hi = vp.seg_hi + (size_t)b * N;
    const int G = global_len[b];  // the first G positions of the order see and are seen by everything (G >= P)
    for (int t = tid; t < N; t += kPlanThreads) {
        int lo = 0, hi = 0;
        if (t < min(G, n_valid)) {
            hi = n_valid;
        } else if (t < n_valid) {
            int id = ids[perm[t]];
            lo = seg_off[id];
            hi = seg_off[id + 1];
            if (bounds_mode == kBoundsBefore) {  // the segments of the same group in front of the own one
                hi = lo;
                lo = seg_off[id / group * group];
            } else if (bounds_mode == kBoundsAfter) {  // ... behind the own one
                lo = hi;
                hi = seg_off[min((id / group + 1) * group, vp.max_id + 1)];
            }
            if (radius > 0) {
                const long long bk = (t - G) / radius;
                const long long w0 = G + (bk - 1) * radius, w1 = G + (bk + 2) * radius;
                lo = (int)max((long long)lo, w0);
                hi = (int)min((long long)hi, w1);
            }
            lo = max(lo, G);  // keys in front of G belong to the global block
            hi = max(hi, lo);
        }
        seg_lo[t] = lo;
        seg_hi[t] = hi;
    }
}

}  // namespace

cudaError_t launch_plan_kernels(const int32_t *row_ids, const int32_t *col_ids, int B, int N,
                                const int32_t *prefix, const int32_t *global_len, int radius, int bounds_mode, int group,
                                const ViewPlan &rowv, const ViewPlan &colv, int32_t *n_valid, int32_t *status,
                                cudaStream_t stream) {
    dim3 grid(B, 2);
    plan_kernel<<<grid, kPlanThreads, 0, stream>>>(row_ids, col_ids, N, prefix, global_len, radius, bounds_mode,
                                                   max(group, 1), rowv, colv, n_valid, status);
    return cudaGetLastError();
}

namespace {
// packed ids (examples one behind the other) -> one padded row of N ids per example, -1 behind its end
__global__ void unpack_ids_kernel(const int32_t *__restrict__ row_ids, const int32_t *__restrict__ col_ids, size_t n, int N,
                                  const int32_t *__restrict__ tok_off, const int32_t *__restrict__ len,
                                  int32_t *__restrict__ rows_out, int32_t *__restrict__ cols_out) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int b = (int)(i / N), k = (int)(i % N);
    const bool in = k < len[b];
    rows_out[i] = in ? row_ids[tok_off[b] + k] : -1;
    cols_out[i] = in ? col_ids[tok_off[b] + k] : -1;
}

// ids of the two extra passes of the row-or-column pattern: (column, row) pairs as one id,
// column-major, for table tokens; -1 (treated as padding by those passes) for everything else
__global__ void pair_ids_kernel(const int32_t *__restrict__ row_ids, const int32_t *__restrict__ col_ids, size_t n,
                                int N, const int32_t *__restrict__ prefix, int n_row_ids, int32_t *__restrict__ out) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int b = (int)(i / N), k = (int)(i % N);
    const int r = row_ids[i], c = col_ids[i];
    out[i] = (k >= prefix[b] && r >= 0 && c >= 0) ? c * n_row_ids + r : -1;
}
}  // namespace

cudaError_t launch_unpack_ids(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *tok_off,
                              const int32_t *len, int32_t *rows_out, int32_t *cols_out, cudaStream_t stream) {
    const size_t n = (size_t)B * N;
    unpack_ids_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(row_ids, col_ids, n, N, tok_off, len, rows_out,
                                                                       cols_out);
    return cudaGetLastError();
}

cudaError_t launch_pair_ids(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix,
                            int n_row_ids, int32_t *out, cudaStream_t stream) {
    const size_t n = (size_t)B * N;
    pair_ids_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(row_ids, col_ids, n, N, prefix, n_row_ids, out);
    return cudaGetLastError();
}

}  // namespace mate

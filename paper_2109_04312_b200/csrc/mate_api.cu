// C ABI of libmate: argument checks, the plan object, and dispatch to the kernels.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <new>

#include "mate_internal.h"

using mate::FwdUnit;
using mate::kTile;
using mate::ViewPlan;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Carves the plan's device arrays out of one allocation.
struct Carver {
    char *base;
    size_t off = 0;
    explicit Carver(char *b) : base(b) {}
    template <typename T>
    T *take(size_t n) {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

void carve(mate_plan_t *pl, char *base, size_t *total) {
    Carver c(base);
    const size_t BN = (size_t)pl->B * pl->N;
    for (int v = 0; v < 2; ++v) {
        ViewPlan &vp = pl->view[v];
        const size_t S = (size_t)pl->B * (vp.max_id + 2);
        vp.perm = c.take<int32_t>(BN);
        vp.inv_perm = c.take<int32_t>(BN);
        vp.seg_lo = c.take<int32_t>(BN);
        vp.seg_hi = c.take<int32_t>(BN);
        vp.seg_off = c.take<int32_t>(S);
        vp.cursor = c.take<int32_t>(S);
        vp.ident = c.take<int32_t>(pl->B);
    }
    pl->n_valid_dev = c.take<int32_t>(pl->B);
    pl->prefix_dev = c.take<int32_t>(pl->B);
    pl->global_dev = c.take<int32_t>(pl->B);
    pl->status_dev = c.take<int32_t>(4);
    pl->head_view_dev = c.take<uint8_t>(pl->H);
    *total = align_up(c.off, 256);
}

// Work-list of the tensor-core forward, built on the host from the segment offsets, then spread
// over the CTAs of a persistent kernel so that every CTA gets about the same amount of softmax
// work (longest-processing-time-first: units by decreasing cost, each to the least loaded CTA).
//
// Cost model: the exponentials are the inner limit of the kernel, and a warp (32 query rows)
// evaluates them 32 key columns at a time, so the cost of a unit is the number of (warp, 32-column
// chunk) pairs it visits plus a constant per half for loading Q and storing O.
constexpr int kChunk = 32;
constexpr int kCostPerHalf = 12;

struct UnitCost {
    FwdUnit u;
    int64_t cost;
};

// Column range of one table row (view position t) of one (example, view): its segment, clipped to the
// three adjacent buckets when the plan is bucketed.  The same arithmetic as step 4 of the plan kernel.
struct RowBounds {
    const int32_t *so;
    int S, P, radius;  // P: length of the global block (bucket origin; no range reaches in front of it)
    int mode = mate::kBoundsOwn, group = 1;
    int seg_of(int t) const { return (int)(std::upper_bound(so, so + S, t) - so) - 1; }
    int lo(int t) const {
        const int id = seg_of(t);
        int l = so[id];
        if (mode == mate::kBoundsBefore) l = so[id / group * group];
        if (mode == mate::kBoundsAfter) l = so[id + 1];
        if (radius <= 0) return std::max(l, P);
        const int64_t bk = (t - P) / radius;
        return (int)std::max<int64_t>(std::max(l, P), P + (bk - 1) * radius);
    }
    int hi(int t) const {
        const int id = seg_of(t);
        int h = so[id + 1];
        if (mode == mate::kBoundsBefore) h = so[id];
        if (mode == mate::kBoundsAfter) h = so[std::min((id / group + 1) * group, S - 1)];
        if (radius > 0) {
            const int64_t bk = (t - P) / radius;
            h = (int)std::min<int64_t>(h, P + (bk + 2) * radius);
        }
        return std::max(h, lo(t));
    }
};

int64_t half_cost(const FwdUnit &u, int h, const RowBounds &rb) {
    const int rows = std::min(kTile, u.nq - h * kTile);
    if (rows <= 0) return 0;
    int64_t c = kCostPerHalf;
    const int n_warps = ceil_div(rows, 32);
    c += (int64_t)n_warps * ceil_div(std::max(u.kA_end - u.kA0, 0), kChunk);
    if (u.kB_end > u.kB0) {
        for (int w = 0; w < n_warps; ++w) {
            const int t0 = u.q0 + h * kTile + w * 32;
            const int t1 = std::min(t0 + 32, u.q0 + h * kTile + rows) - 1;
            c += ceil_div(rb.hi(t1) - rb.lo(t0), kChunk) + 1;  // + 1: chunks are aligned to the tile, not to lo
        }
    }
    return c;
}

// Units of all (example, head) pairs.  share = 0: no unit is split (the backward's list: its work
// items are halves of units per side, fine enough as they are).  share > 0 (a CTA's share of the
// total cost): a prefix-row unit, whose columns are all valid positions, that costs more than 1.3
// shares is cut along the columns into parts of about 0.75 shares, to be combined in the kernel.
void make_units(mate_plan_t *pl, const std::vector<std::vector<int32_t>> &seg_off_host, int64_t share,
                std::vector<UnitCost> &all, int *n_slots, size_t *ws_bytes, int64_t *total_cost) {
    const int N = pl->N;
    all.clear();
    *n_slots = 0;
    *ws_bytes = 0;
    *total_cost = 0;
    for (int v = 0; v < 2; ++v) {
        const ViewPlan &vp = pl->view[v];
        if (vp.n_heads == 0) continue;
        const int S = vp.max_id + 2;
        for (int b = 0; b < pl->B; ++b) {
            const int32_t *so = seg_off_host[v].data() + (size_t)b * S;
            const int nv = pl->n_valid[b];
            const int P = std::min(pl->global[b], nv);  // rows and keys in front of it are global
            const RowBounds rb{so, S, P, pl->radius, pl->bounds_mode, pl->group};
            std::vector<UnitCost> proto;  // units of one (example, view); copied per head below
            for (int q0 = 0; q0 < P; q0 += mate::kUnitRows) {  // prefix rows: every valid key
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(mate::kUnitRows, P - q0);
                u.kA_end = nv;
                const int n_tiles = ceil_div(nv, kTile);
                const int64_t whole = half_cost(u, 0, rb) + half_cost(u, 1, rb);
                int want = 1;
                if (share > 0 && 10 * whole > 13 * share)
                    want = (int)std::min<int64_t>(n_tiles, (4 * whole + 3 * share - 1) / (3 * share));
                const int per = ceil_div(n_tiles, want);
                const int n_parts = ceil_div(n_tiles, per);  // every part holds at least one tile
                for (int part = 0; part < n_parts; ++part) {
                    FwdUnit w = u;
                    w.kA0 = part * per * kTile;
                    w.kA_end = std::min(nv, (part + 1) * per * kTile);
                    w.n_parts = n_parts;
                    w.part = part;
                    proto.push_back({w, 0});
                }
            }
            for (int q0 = P; q0 < nv; q0 += mate::kUnitRows) {  // table rows: prefix + own segments
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(mate::kUnitRows, nv - q0);
                u.kA0 = 0;
                u.kA_end = P;
                u.kB0 = rb.lo(q0);   // lo and hi do not decrease along the rows
                u.kB_end = rb.hi(q0 + u.nq - 1);
                for (int h = 0; h < 2; ++h) {
                    const int r0 = q0 + h * kTile, r1 = std::min(q0 + u.nq, r0 + kTile) - 1;
                    if (r1 < r0) continue;
                    u.lo[h] = rb.lo(r0);
                    u.hi[h] = rb.hi(r1);
                }
                u.n_parts = 1;
                proto.push_back({u, 0});
            }
            for (int q0 = nv; q0 < N; q0 += mate::kUnitRows) {  // padding rows: no key at all
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(mate::kUnitRows, N - q0);
                u.n_parts = 1;
                proto.push_back({u, 0});
            }
            for (auto &pc : proto) pc.cost = half_cost(pc.u, 0, rb) + half_cost(pc.u, 1, rb);
            for (int h = 0; h < pl->H; ++h) {
                if (pl->head_view[h] != v) continue;
                int slot = -1;
                for (UnitCost pc : proto) {
                    pc.u.b = b;
                    pc.u.h = h;
                    pc.u.ctr = -1;
                    if (pc.u.n_parts > 1) {
                        if (pc.u.part == 0) slot = (*n_slots)++;
                        pc.u.ctr = slot;
                        pc.u.ws_off = (int32_t)((*ws_bytes + pc.u.part * mate::kPartialBytes) >> 10);
                        if (pc.u.part == pc.u.n_parts - 1) *ws_bytes += pc.u.n_parts * mate::kPartialBytes;
                    }
                    *total_cost += pc.cost;
                    all.push_back(pc);
                }
            }
        }
    }
    // longest first: the CTAs of the persistent kernels take work from the head of the list as they
    // become free (a shared counter), so the order is the whole schedule
    std::stable_sort(all.begin(), all.end(), [](const UnitCost &a, const UnitCost &b) { return a.cost > b.cost; });
}

int build_units(mate_plan_t *pl, const std::vector<std::vector<int32_t>> &seg_off_host) {
    static_assert(mate::kPartialBytes % 1024 == 0, "ws_off counts KiB");
    const int n_ctas = std::max(pl->n_ctas, 1);
    std::vector<UnitCost> all;
    int n_slots = 0;
    size_t ws_bytes = 0;
    int64_t total_cost = 0;
    // backward: unsplit list; its total cost also gives the share of a CTA
    make_units(pl, seg_off_host, 0, all, &n_slots, &ws_bytes, &total_cost);
    pl->bwd_units.clear();
    for (const UnitCost &uc : all) pl->bwd_units.push_back(uc.u);
    pl->n_bwd_units = (int)pl->bwd_units.size();
    // forward: long prefix units split; the forward kernel runs several CTAs per SM
    const int64_t share = std::max<int64_t>(total_cost / ((int64_t)n_ctas * mate::tc_fwd_ctas_per_sm()), 1);
    make_units(pl, seg_off_host, share, all, &n_slots, &ws_bytes, &total_cost);
    pl->fwd_units.clear();
    for (const UnitCost &uc : all) pl->fwd_units.push_back(uc.u);
    pl->n_fwd_units = (int)pl->fwd_units.size();
    pl->n_fwd_slots = n_slots;
    pl->fwd_ws_bytes = ws_bytes;
    if (getenv("MATE_LOG"))
        fprintf(stderr, "[mate] work-lists: forward %d units (%d split), backward %d units, %d CTAs, cost total %lld "
                        "(%.1f per CTA, largest forward unit %lld), forward workspace %zu bytes\n",
                pl->n_fwd_units, pl->n_fwd_slots, pl->n_bwd_units, n_ctas, (long long)total_cost,
                (double)total_cost / n_ctas, all.empty() ? 0ll : (long long)all.front().cost, pl->fwd_ws_bytes);

    // device copy: units, CTA offsets, arrival counters (zeroed once; the kernel resets them)
    Carver c(nullptr);
    c.take<FwdUnit>(pl->n_fwd_units);
    c.take<FwdUnit>(pl->n_bwd_units);
    c.take<int32_t>(mate::kSchedWords + 8 * (size_t)pl->n_fwd_slots);
    const size_t bytes = align_up(c.off, 256);
    if (cudaMalloc(&pl->work_block, bytes) != cudaSuccess) {
        cudaGetLastError();
        return MATE_ERR_NOMEM;
    }
    Carver d((char *)pl->work_block);
    pl->fwd_units_dev = d.take<FwdUnit>(pl->n_fwd_units);
    pl->bwd_units_dev = d.take<FwdUnit>(pl->n_bwd_units);
    pl->fwd_counters_dev = d.take<int32_t>(mate::kSchedWords + 8 * (size_t)pl->n_fwd_slots);
    return MATE_OK;
}

}  // namespace

extern "C" {

const char *mate_status_string(int status) {
    switch (status) {
        case MATE_OK: return "ok";
        case MATE_ERR_INVALID_ARG: return "invalid argument";
        case MATE_ERR_UNSUPPORTED: return "unsupported head dim, dtype or implementation";
        case MATE_ERR_ALIGNMENT: return "tensor pointer not 16-byte aligned";
        case MATE_ERR_CUDA: return "CUDA runtime error";
        case MATE_ERR_TIMEOUT: return "bounded device wait expired";
        case MATE_ERR_NOMEM: return "out of memory";
        case MATE_ERR_WORKSPACE: return "workspace missing or too small";
        case MATE_ERR_TOO_LARGE: return "B*H*N exceeds the built-in scratch of mate_attn_bwd_noalloc";
        default: return "unknown status";
    }
}

int mate_plan_destroy(mate_plan_t *plan) {
    if (!plan) return MATE_OK;
    for (int s = 0; s < 2; ++s) mate_plan_destroy(plan->sub[s]);
    if (plan->pair_ids_dev) cudaFree(plan->pair_ids_dev);
    if (plan->tok_off_dev) cudaFree(plan->tok_off_dev);
    if (plan->dev_block) cudaFree(plan->dev_block);
    if (plan->work_block) cudaFree(plan->work_block);
    delete plan;
    return MATE_OK;
}

int mate_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len,
              const uint8_t *head_view, int H, int max_row_id, int max_col_id, void *stream,
              mate_plan_t **out) {
    return mate_plan_bucketed(row_ids, col_ids, B, N, prefix_len, head_view, H, max_row_id, max_col_id, 0,
                              stream, out);
}

int mate_plan_bucketed(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len,
                       const uint8_t *head_view, int H, int max_row_id, int max_col_id, int radius,
                       void *stream, mate_plan_t **out) {
    if (out) *out = nullptr;
    if (B <= 0) return MATE_ERR_INVALID_ARG;
    const std::vector<int32_t> prefix((size_t)B, prefix_len);
    return mate_plan_varlen(row_ids, col_ids, B, N, prefix.data(), head_view, H, max_row_id, max_col_id, radius,
                            stream, out);
}

static int build_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                      const int32_t *global_len, const uint8_t *head_view, int H, int max_row_id, int max_col_id,
                      int radius, int bounds_mode, int group, void *stream, mate_plan_t **out);

int mate_plan_varlen(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                     const uint8_t *head_view, int H, int max_row_id, int max_col_id, int radius,
                     void *stream, mate_plan_t **out) {
    return build_plan(row_ids, col_ids, B, N, prefix_len, nullptr, head_view, H, max_row_id, max_col_id, radius,
                      mate::kBoundsOwn, 1, stream, out);
}

int mate_plan_bucketed_global(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                              const int32_t *global_len, const uint8_t *head_view, int H, int max_row_id,
                              int max_col_id, int radius, void *stream, mate_plan_t **out) {
    if (out) *out = nullptr;
    if (!global_len || !prefix_len || B <= 0 || radius <= 0) return MATE_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b)
        if (global_len[b] < prefix_len[b] || global_len[b] > N) return MATE_ERR_INVALID_ARG;
    return build_plan(row_ids, col_ids, B, N, prefix_len, global_len, head_view, H, max_row_id, max_col_id, radius,
                      mate::kBoundsOwn, 1, stream, out);
}

/* Packed batches: the examples lie one behind the other on a common token axis.  The plan itself is the
 * padded one over N = the longest example (small integer arrays); what changes is where the kernels
 * find an example's rows in the tensors, and that positions behind an example's end do not exist. */
int mate_plan_packed(const int32_t *row_ids, const int32_t *col_ids, int B, const int32_t *cu_seqlens,
                     const int32_t *prefix_len, const uint8_t *head_view, int H, int max_row_id, int max_col_id,
                     void *stream, mate_plan_t **out) {
    if (out) *out = nullptr;
    if (!row_ids || !col_ids || !cu_seqlens || !prefix_len || !head_view || !out || B <= 0 || H <= 0)
        return MATE_ERR_INVALID_ARG;
    if (cu_seqlens[0] != 0) return MATE_ERR_INVALID_ARG;
    int n_max = 1;
    std::vector<int32_t> off_len((size_t)2 * B);
    for (int b = 0; b < B; ++b) {
        const int len = cu_seqlens[b + 1] - cu_seqlens[b];
        if (len < 0 || prefix_len[b] < 0 || prefix_len[b] > len) return MATE_ERR_INVALID_ARG;
        n_max = std::max(n_max, len);
        off_len[b] = cu_seqlens[b];
        off_len[B + b] = len;
    }
    const int T = cu_seqlens[B];
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *off_dev = nullptr, *ids = nullptr;
    const size_t BN = (size_t)B * n_max;
    if (cudaMalloc(&off_dev, sizeof(int32_t) * 2 * B) != cudaSuccess || cudaMalloc(&ids, sizeof(int32_t) * 2 * BN) != cudaSuccess) {
        cudaGetLastError();
        if (off_dev) cudaFree(off_dev);
        return MATE_ERR_NOMEM;
    }
    bool ok = cudaMemcpyAsync(off_dev, off_len.data(), sizeof(int32_t) * 2 * B, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && mate::launch_unpack_ids(row_ids, col_ids, B, n_max, off_dev, off_dev + B, ids, ids + BN, st) == cudaSuccess;
    mate_plan_t *pl = nullptr;
    int rc = ok ? build_plan(ids, ids + BN, B, n_max, prefix_len, nullptr, head_view, H, max_row_id, max_col_id, 0,
                             mate::kBoundsOwn, 1, stream, &pl)
                : MATE_ERR_CUDA;
    cudaFree(ids);  // build_plan has waited for its kernels
    if (rc != MATE_OK) {
        cudaFree(off_dev);
        return rc;
    }
    pl->T = T;
    pl->tok_off_dev = off_dev;
    pl->len_dev = off_dev + B;
    *out = pl;
    return MATE_OK;
}

/* The head-independent pattern: three passes over plans the ordinary kernels can run (see mate.h).
 *   main plan  every head a row head: prefix rows against everything, table rows against the prefix
 *              and their own row (which holds their own cell)
 *   sub[0]     ids = (column, row) pairs, column-major, prefix treated as padding: table rows against
 *              the cells of their column in front of their own cell
 *   sub[1]     the same behind their own cell
 * The three key sets of a row are disjoint and their union is the pattern. */
int mate_plan_sat(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len, int H,
                  int max_row_id, int max_col_id, void *stream, mate_plan_t **out) {
    if (out) *out = nullptr;
    if (!out || B <= 0 || H <= 0 || max_row_id < 0 || max_col_id < 0) return MATE_ERR_INVALID_ARG;
    if ((long long)(max_row_id + 1) * (max_col_id + 1) > (1ll << 28)) return MATE_ERR_UNSUPPORTED;
    const std::vector<int32_t> prefix((size_t)B, prefix_len), zero((size_t)B, 0);
    const std::vector<uint8_t> rows_only((size_t)H, 0), cols_only((size_t)H, 1);
    mate_plan_t *pl = nullptr;
    int rc = build_plan(row_ids, col_ids, B, N, prefix.data(), nullptr, rows_only.data(), H, max_row_id, max_col_id, 0,
                        mate::kBoundsOwn, 1, stream, &pl);
    if (rc != MATE_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const int n_row_ids = max_row_id + 1, max_pair = n_row_ids * (max_col_id + 1) - 1;
    bool ok = cudaMalloc(&pl->pair_ids_dev, sizeof(int32_t) * (size_t)B * N) == cudaSuccess;
    ok = ok && mate::launch_pair_ids(row_ids, col_ids, B, N, pl->prefix_dev, n_row_ids, pl->pair_ids_dev, st) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        mate_plan_destroy(pl);
        return MATE_ERR_NOMEM;
    }
    for (int s = 0; s < 2 && rc == MATE_OK; ++s)
        rc = build_plan(pl->pair_ids_dev, pl->pair_ids_dev, B, N, zero.data(), nullptr, cols_only.data(), H, max_pair, max_pair, 0,
                        s == 0 ? mate::kBoundsBefore : mate::kBoundsAfter, n_row_ids, stream, &pl->sub[s]);
    if (rc != MATE_OK) {
        mate_plan_destroy(pl);
        return rc;
    }
    *out = pl;
    return MATE_OK;
}

static int build_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                      const int32_t *global_len, const uint8_t *head_view, int H, int max_row_id, int max_col_id,
                      int radius, int bounds_mode, int group, void *stream, mate_plan_t **out) {
    if (out) *out = nullptr;
    if (radius < 0) return MATE_ERR_INVALID_ARG;
    if (!row_ids || !col_ids || !head_view || !out || !prefix_len) return MATE_ERR_INVALID_ARG;
    if (B <= 0 || N <= 0 || H <= 0) return MATE_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b)
        if (prefix_len[b] < 0 || prefix_len[b] > N) return MATE_ERR_INVALID_ARG;
    if (max_row_id < 0 || max_col_id < 0) return MATE_ERR_INVALID_ARG;
    if ((long long)B * N > (1ll << 30) || max_row_id > (1 << 28) || max_col_id > (1 << 28))
        return MATE_ERR_UNSUPPORTED;
    for (int h = 0; h < H; ++h)
        if (head_view[h] > 1) return MATE_ERR_INVALID_ARG;

    cudaStream_t st = (cudaStream_t)stream;
    mate_plan_t *pl = new (std::nothrow) mate_plan_t();
    if (!pl) return MATE_ERR_NOMEM;
    pl->B = B;
    pl->N = N;
    pl->prefix.assign(prefix_len, prefix_len + B);
    if (global_len) pl->global.assign(global_len, global_len + B);
    else pl->global = pl->prefix;
    pl->H = H;
    pl->radius = radius;
    pl->bounds_mode = bounds_mode;
    pl->group = std::max(group, 1);
    pl->head_view.assign(head_view, head_view + H);
    pl->view[0].max_id = max_row_id;
    pl->view[1].max_id = max_col_id;
    for (int h = 0; h < H; ++h) pl->view[head_view[h]].n_heads++;

    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&pl->n_ctas, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            delete pl;
            return MATE_ERR_CUDA;
        }
        pl->device = dev;
    }
    size_t total = 0;
    carve(pl, nullptr, &total);
    if (cudaMalloc(&pl->dev_block, total) != cudaSuccess) {
        cudaGetLastError();
        delete pl;
        return MATE_ERR_NOMEM;
    }
    carve(pl, (char *)pl->dev_block, &total);

    int rc = MATE_OK;
    int32_t status_host[4] = {0, 0, 0, 0};
    std::vector<std::vector<int32_t>> seg_off_host(2);
    pl->n_valid.resize(B);
    bool ok = cudaMemsetAsync(pl->status_dev, 0, 4 * sizeof(int32_t), st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(pl->head_view_dev, pl->head_view.data(), H, cudaMemcpyHostToDevice,
                               st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(pl->prefix_dev, pl->prefix.data(), B * sizeof(int32_t), cudaMemcpyHostToDevice,
                               st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(pl->global_dev, pl->global.data(), B * sizeof(int32_t), cudaMemcpyHostToDevice,
                               st) == cudaSuccess;
    ok = ok && mate::launch_plan_kernels(row_ids, col_ids, B, N, pl->prefix_dev, pl->global_dev, radius, bounds_mode, pl->group, pl->view[0], pl->view[1],
                                         pl->n_valid_dev, pl->status_dev, st) == cudaSuccess;
    for (int v = 0; v < 2 && ok; ++v) {
        seg_off_host[v].resize((size_t)B * (pl->view[v].max_id + 2));
        ok = cudaMemcpyAsync(seg_off_host[v].data(), pl->view[v].seg_off,
                             seg_off_host[v].size() * sizeof(int32_t), cudaMemcpyDeviceToHost,
                             st) == cudaSuccess;
    }
    ok = ok && cudaMemcpyAsync(pl->n_valid.data(), pl->n_valid_dev, B * sizeof(int32_t),
                               cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(status_host, pl->status_dev, sizeof(status_host),
                               cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) rc = MATE_ERR_CUDA;
    if (rc == MATE_OK && status_host[0] != 0) rc = MATE_ERR_INVALID_ARG;
    if (rc != MATE_OK) {
        mate_plan_destroy(pl);
        return rc;
    }

    // unmasked pairs per (example, view): P * n_valid + sum_s L_s (L_s + P); a bucketed plan counts,
    // row by row, the prefix and the clipped part of the segment
    pl->pairs.assign((size_t)B * 2, 0);
    for (int v = 0; v < 2; ++v) {
        const int S = pl->view[v].max_id + 2;
        for (int b = 0; b < B; ++b) {
            const int32_t *so = seg_off_host[v].data() + (size_t)b * S;
            const int P = std::min(pl->global[b], pl->n_valid[b]);
            int64_t c = (int64_t)P * pl->n_valid[b];
            if (radius > 0 || pl->bounds_mode != mate::kBoundsOwn || P != pl->prefix[b]) {
                const RowBounds rb{so, S, P, radius, pl->bounds_mode, pl->group};
                for (int t = P; t < pl->n_valid[b]; ++t) c += P + rb.hi(t) - rb.lo(t);
            } else {
                for (int s = 0; s + 1 < S; ++s) {
                    const int64_t L = so[s + 1] - so[s];
                    c += L * (L + P);
                }
            }
            pl->pairs[(size_t)b * 2 + v] = c;
        }
    }

    rc = build_units(pl, seg_off_host);
    if (rc != MATE_OK) {
        mate_plan_destroy(pl);
        return rc;
    }
    bool up = cudaMemsetAsync(pl->fwd_counters_dev, 0,
                              sizeof(int32_t) * (mate::kSchedWords + 8 * (size_t)pl->n_fwd_slots), st) == cudaSuccess;
    if (pl->n_fwd_units > 0)
        up = up && cudaMemcpyAsync(pl->fwd_units_dev, pl->fwd_units.data(), sizeof(FwdUnit) * pl->n_fwd_units,
                                   cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (pl->n_bwd_units > 0)
        up = up && cudaMemcpyAsync(pl->bwd_units_dev, pl->bwd_units.data(), sizeof(FwdUnit) * pl->n_bwd_units,
                                   cudaMemcpyHostToDevice, st) == cudaSuccess;
    up = up && cudaStreamSynchronize(st) == cudaSuccess;
    if (!up) {
        mate_plan_destroy(pl);
        return MATE_ERR_CUDA;
    }
    *out = pl;
    return MATE_OK;
}

int mate_plan_get(const mate_plan_t *plan, int view, int32_t *perm, int32_t *inv_perm,
                  int32_t *seg_off) {
    if (!plan || view < 0 || view > 1) return MATE_ERR_INVALID_ARG;
    const ViewPlan &vp = plan->view[view];
    const size_t BN = (size_t)plan->B * plan->N * sizeof(int32_t);
    bool ok = true;
    if (perm) ok = ok && cudaMemcpy(perm, vp.perm, BN, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (inv_perm) ok = ok && cudaMemcpy(inv_perm, vp.inv_perm, BN, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (seg_off)
        ok = ok && cudaMemcpy(seg_off, vp.seg_off, (size_t)plan->B * (vp.max_id + 2) * sizeof(int32_t),
                              cudaMemcpyDeviceToHost) == cudaSuccess;
    return ok ? MATE_OK : MATE_ERR_CUDA;
}

int mate_plan_useful_pairs(const mate_plan_t *plan, int64_t *pairs) {
    if (!plan || !pairs) return MATE_ERR_INVALID_ARG;
    for (int b = 0; b < plan->B; ++b)
        for (int h = 0; h < plan->H; ++h) {
            int64_t c = plan->pairs[(size_t)b * 2 + plan->head_view[h]];
            for (int s = 0; s < 2; ++s)
                if (plan->sub[s]) c += plan->sub[s]->pairs[(size_t)b * 2 + 1];
            pairs[(size_t)b * plan->H + h] = c;
        }
    return MATE_OK;
}

int mate_plan_status(const mate_plan_t *plan, void *stream) {
    if (!plan) return MATE_ERR_INVALID_ARG;
    for (int s = 0; s < 2; ++s)
        if (plan->sub[s]) {
            const int rc = mate_plan_status(plan->sub[s], stream);
            if (rc != MATE_OK) return rc;
        }
    cudaStream_t st = (cudaStream_t)stream;
    int32_t s[4] = {0, 0, 0, 0};
    if (cudaMemcpyAsync(s, plan->status_dev, sizeof(s), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(plan->status_dev + 1, 0, 2 * sizeof(int32_t), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return MATE_ERR_CUDA;
    if (s[1] != 0) {
        if (getenv("MATE_LOG"))
            fprintf(stderr, "[mate] a bounded wait expired: barrier slot %d, parity %d, warp %d\n", (s[2] >> 8) & 0xff,
                    (s[2] >> 7) & 1, s[2] & 0x7f);
        // a kernel that gave up may have left the scheduling and arrival counters half way
        if (cudaMemsetAsync(plan->fwd_counters_dev, 0,
                            sizeof(int32_t) * (mate::kSchedWords + 8 * (size_t)plan->n_fwd_slots), st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return MATE_ERR_CUDA;
        return MATE_ERR_TIMEOUT;
    }
    return MATE_OK;
}

// The plan's arrays, its CTA count and the kernels' per-device set-up belong to the device the plan
// was made on: a call with another device current is refused before anything is launched.
static int check_device(const mate_plan_t *plan) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MATE_ERR_CUDA;
    return dev == plan->device ? MATE_OK : MATE_ERR_INVALID_ARG;
}

static int check_common(const mate_plan_t *plan, int d, int dtype, unsigned flags, bool *use_tc) {
    if (!plan) return MATE_ERR_INVALID_ARG;
    if (dtype != MATE_BF16 && dtype != MATE_F32) return MATE_ERR_UNSUPPORTED;
    if (d <= 0 || d % 8 != 0 || d > 128) return MATE_ERR_UNSUPPORTED;
    const unsigned impl = flags & 3u;
    constexpr unsigned kLoaderBits = MATE_FLAG_BULK_TILES | MATE_FLAG_GATHER_TILES;
    if (impl == 3u || (flags & ~(3u | MATE_FLAG_VIEW_ORDER | kLoaderBits)) || (flags & kLoaderBits) == kLoaderBits)
        return MATE_ERR_INVALID_ARG;
    const bool tc_ok = mate::tc_supported(d, dtype);
    if (impl == MATE_IMPL_TCGEN05 && !tc_ok) return MATE_ERR_UNSUPPORTED;
    *use_tc = (impl == MATE_IMPL_TCGEN05) || (impl == MATE_IMPL_AUTO && tc_ok);
    return MATE_OK;
}

// Scratch of one pass (the ordinary kernels) and of a whole call.  For a row-or-column plan the call
// holds, behind the passes' own scratch (the passes run one after the other and share it), the
// outputs of the two extra passes: forward 2 x (O + LSE), backward 2 x (dQ, dK, dV).
static size_t pass_fwd_bytes(const mate_plan_t *plan, int d, bool use_tc) {
    size_t n = use_tc ? mate::tc_fwd_workspace(plan, d) : 0;
    for (int s = 0; s < 2; ++s)
        if (plan->sub[s]) n = std::max(n, use_tc ? mate::tc_fwd_workspace(plan->sub[s], d) : (size_t)0);
    return align_up(n, 256);
}
static size_t pass_bwd_bytes(const mate_plan_t *plan, bool use_tc) {
    return align_up(use_tc ? mate::tc_bwd_workspace(plan) : mate::simt_bwd_workspace(plan), 256);
}
static size_t elem_bytes(int dtype) { return dtype == MATE_F32 ? 4 : 2; }

int mate_attn_workspace_bytes(const mate_plan_t *plan, int d, int dtype, unsigned flags,
                              size_t *fwd_bytes, size_t *bwd_bytes) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    const size_t rows = plan->n_rows();
    size_t f = pass_fwd_bytes(plan, d, use_tc), b = pass_bwd_bytes(plan, use_tc);
    if (plan->sub[0]) {
        f += 2 * (align_up(rows * d * elem_bytes(dtype), 256) + align_up(rows * sizeof(float), 256));
        b += 6 * align_up(rows * d * elem_bytes(dtype), 256);
    }
    if (fwd_bytes) *fwd_bytes = f;
    if (bwd_bytes) *bwd_bytes = b;
    return MATE_OK;
}

static int fwd_pass(const mate_plan_t *plan, bool use_tc, const void *Q, const void *K, const void *V, int d, int dtype,
                    float scale, void *O, float *LSE, void *ws, unsigned flags, cudaStream_t st) {
    if (use_tc) return mate::tc_fwd(plan, Q, K, V, scale, O, LSE, ws, flags, st);
    return mate::simt_fwd(plan, Q, K, V, d, dtype, scale, O, LSE, flags, st);
}

int mate_attn_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d,
                  int dtype, float scale, void *O, float *LSE, void *workspace,
                  size_t workspace_bytes, unsigned flags, void *stream) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    if ((rc = check_device(plan)) != MATE_OK) return rc;
    if (!Q || !K || !V || !O || !LSE) return MATE_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE))
        return MATE_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    // the tensor-core forward takes the row maximum before scaling, which needs scale > 0
    if (use_tc && !(scale > 0.f)) {
        if ((flags & 3u) == MATE_IMPL_TCGEN05) return MATE_ERR_UNSUPPORTED;
        use_tc = false;
    }
    size_t need = 0;
    mate_attn_workspace_bytes(plan, d, dtype, use_tc ? MATE_IMPL_TCGEN05 : MATE_IMPL_SIMT, &need, nullptr);
    if (need > 0 && (!workspace || workspace_bytes < need)) return MATE_ERR_WORKSPACE;
    if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MATE_ERR_ALIGNMENT;
    if ((flags & MATE_FLAG_VIEW_ORDER) && (plan->sub[0] || plan->T)) return MATE_ERR_UNSUPPORTED;
    rc = fwd_pass(plan, use_tc, Q, K, V, d, dtype, scale, O, LSE, workspace, flags, st);
    if (rc != MATE_OK || !plan->sub[0]) return rc;
    // row-or-column pattern: the two passes over the rest of the column, then the merge
    const size_t rows = plan->n_rows();
    const size_t o_bytes = align_up(rows * d * elem_bytes(dtype), 256), l_bytes = align_up(rows * sizeof(float), 256);
    char *w = (char *)workspace + pass_fwd_bytes(plan, d, use_tc);
    void *Os[2];
    float *Ls[2];
    for (int s = 0; s < 2; ++s) {
        Os[s] = w;
        Ls[s] = (float *)(w + o_bytes);
        w += o_bytes + l_bytes;
        rc = fwd_pass(plan->sub[s], use_tc, Q, K, V, d, dtype, scale, Os[s], Ls[s], workspace, flags, st);
        if (rc != MATE_OK) return rc;
    }
    return mate::launch_merge_passes(O, LSE, Os[0], Ls[0], Os[1], Ls[1], rows, d, dtype, st) == cudaSuccess ? MATE_OK
                                                                                                           : MATE_ERR_CUDA;
}

static int bwd_pass(const mate_plan_t *plan, bool use_tc, const void *Q, const void *K, const void *V, const void *O,
                    const float *LSE, const void *dO, int d, int dtype, float scale, void *dQ, void *dK, void *dV, void *ws,
                    cudaStream_t st) {
    if (use_tc) return mate::tc_bwd(plan, Q, K, V, O, LSE, dO, scale, dQ, dK, dV, ws, st);
    return mate::simt_bwd(plan, Q, K, V, O, LSE, dO, d, dtype, scale, dQ, dK, dV, ws, st);
}

int mate_attn_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V,
                  const void *O, const float *LSE, const void *dO, int d, int dtype, float scale,
                  void *dQ, void *dK, void *dV, void *workspace, size_t workspace_bytes,
                  unsigned flags, void *stream) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    if ((rc = check_device(plan)) != MATE_OK) return rc;
    if (!Q || !K || !V || !O || !LSE || !dO || !dQ || !dK || !dV) return MATE_ERR_INVALID_ARG;
    if (flags & MATE_FLAG_VIEW_ORDER) return MATE_ERR_UNSUPPORTED;  // forward only
    const void *ptrs[] = {Q, K, V, O, LSE, dO, dQ, dK, dV};
    for (const void *p : ptrs)
        if (!aligned16(p)) return MATE_ERR_ALIGNMENT;
    size_t need = 0;
    mate_attn_workspace_bytes(plan, d, dtype, use_tc ? MATE_IMPL_TCGEN05 : MATE_IMPL_SIMT, nullptr, &need);
    if (!workspace || workspace_bytes < need) return MATE_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MATE_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    rc = bwd_pass(plan, use_tc, Q, K, V, O, LSE, dO, d, dtype, scale, dQ, dK, dV, workspace, st);
    if (rc != MATE_OK || !plan->sub[0]) return rc;
    // Row-or-column pattern.  With the final O and LSE every pass computes the gradient of its own
    // pairs.  The two column passes are each other's transpose (keys in front of / behind the own
    // cell), and the kernels take a plan's key ranges for the query side and for the key side alike;
    // run on both plans and summed, every pair is still counted once on each side.
    const size_t n = plan->n_rows() * d;
    const size_t g_bytes = align_up(n * elem_bytes(dtype), 256);
    char *w = (char *)workspace + pass_bwd_bytes(plan, use_tc);
    void *g[2][3];
    for (int s = 0; s < 2; ++s) {
        for (int i = 0; i < 3; ++i, w += g_bytes) g[s][i] = w;
        rc = bwd_pass(plan->sub[s], use_tc, Q, K, V, O, LSE, dO, d, dtype, scale, g[s][0], g[s][1], g[s][2], workspace, st);
        if (rc != MATE_OK) return rc;
    }
    void *outs[3] = {dQ, dK, dV};
    for (int i = 0; i < 3; ++i)
        if (mate::launch_add3(outs[i], g[0][i], g[1][i], n, dtype, st) != cudaSuccess) return MATE_ERR_CUDA;
    return MATE_OK;
}

}  // extern "C"

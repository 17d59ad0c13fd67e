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

void carve(mate_plan_t *pl, char *base, size_t *total, int max_units) {
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
    }
    pl->n_valid_dev = c.take<int32_t>(pl->B);
    pl->status_dev = c.take<int32_t>(4);
    pl->head_view_dev = c.take<uint8_t>(pl->H);
    pl->fwd_units_dev = c.take<FwdUnit>(max_units);
    pl->bwd_units_dev = c.take<FwdUnit>(max_units);
    *total = align_up(c.off, 256);
}

// Tile work-list of the tensor-core kernels, built on the host from the segment offsets.
// `symmetric` units are reused by the backward kernels (the pattern is symmetric, so the key tiles
// a query tile visits are also the query tiles a key tile is visited by).
void build_units(mate_plan_t *pl, const std::vector<std::vector<int32_t>> &seg_off_host) {
    std::vector<FwdUnit> units;
    const int P = pl->P, N = pl->N;
    for (int v = 0; v < 2; ++v) {
        const ViewPlan &vp = pl->view[v];
        if (vp.n_heads == 0) continue;
        const int S = vp.max_id + 2;
        for (int b = 0; b < pl->B; ++b) {
            const int32_t *so = seg_off_host[v].data() + (size_t)b * S;
            const int nv = pl->n_valid[b];
            std::vector<FwdUnit> tiles;
            auto seg_of = [&](int t) {  // segment index s with so[s] <= t < so[s+1]
                return (int)(std::upper_bound(so, so + S, t) - so) - 1;
            };
            for (int q0 = 0; q0 < P; q0 += kTile) {
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(kTile, P - q0);
                u.kA_end = nv;
                u.kA_n = ceil_div(nv, kTile);
                tiles.push_back(u);
            }
            for (int q0 = P; q0 < nv; q0 += kTile) {
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(kTile, nv - q0);
                const int lo_first = so[seg_of(q0)];
                const int hi_last = so[seg_of(q0 + u.nq - 1) + 1];
                u.kA_end = P;
                u.kA_n = ceil_div(P, kTile);
                u.kB0 = lo_first;
                u.kB_end = hi_last;
                u.kB_n = ceil_div(hi_last - lo_first, kTile);
                tiles.push_back(u);
            }
            for (int q0 = nv; q0 < N; q0 += kTile) {
                FwdUnit u{};
                u.q0 = q0;
                u.nq = std::min(kTile, N - q0);
                tiles.push_back(u);
            }
            for (int h = 0; h < pl->H; ++h) {
                if (pl->head_view[h] != v) continue;
                for (FwdUnit u : tiles) {
                    u.b = b;
                    u.h = h;
                    u.part = 0;
                    u.n_parts = 1;
                    u.slot = -1;
                    u.cost = u.kA_n + u.kB_n;
                    units.push_back(u);
                }
            }
        }
    }
    std::stable_sort(units.begin(), units.end(),
                     [](const FwdUnit &a, const FwdUnit &b) { return a.cost > b.cost; });
    pl->fwd_units = std::move(units);
    pl->n_fwd_units = (int)pl->fwd_units.size();
    pl->n_fwd_slots = 0;
}

int max_units_bound(int B, int N, int P, int H) {
    // per (b, h): prefix tiles + table tiles + padding tiles, each at most ceil(.../128) + 1
    const int per = ceil_div(P, kTile) + 2 * (ceil_div(N, kTile) + 1);
    return B * H * per;
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
    if (plan->dev_block) cudaFree(plan->dev_block);
    delete plan;
    return MATE_OK;
}

int mate_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len,
              const uint8_t *head_view, int H, int max_row_id, int max_col_id, void *stream,
              mate_plan_t **out) {
    if (out) *out = nullptr;
    if (!row_ids || !col_ids || !head_view || !out) return MATE_ERR_INVALID_ARG;
    if (B <= 0 || N <= 0 || H <= 0 || prefix_len < 0 || prefix_len > N) return MATE_ERR_INVALID_ARG;
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
    pl->P = prefix_len;
    pl->H = H;
    pl->head_view.assign(head_view, head_view + H);
    pl->view[0].max_id = max_row_id;
    pl->view[1].max_id = max_col_id;
    for (int h = 0; h < H; ++h) pl->view[head_view[h]].n_heads++;

    const int max_units = max_units_bound(B, N, prefix_len, H);
    size_t total = 0;
    carve(pl, nullptr, &total, max_units);
    if (cudaMalloc(&pl->dev_block, total) != cudaSuccess) {
        cudaGetLastError();
        delete pl;
        return MATE_ERR_NOMEM;
    }
    carve(pl, (char *)pl->dev_block, &total, max_units);

    int rc = MATE_OK;
    int32_t status_host[4] = {0, 0, 0, 0};
    std::vector<std::vector<int32_t>> seg_off_host(2);
    pl->n_valid.resize(B);
    bool ok = cudaMemsetAsync(pl->status_dev, 0, 4 * sizeof(int32_t), st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(pl->head_view_dev, pl->head_view.data(), H, cudaMemcpyHostToDevice,
                               st) == cudaSuccess;
    ok = ok && mate::launch_plan_kernels(row_ids, col_ids, B, N, prefix_len, pl->view[0], pl->view[1],
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

    // unmasked pairs per (example, view): P * n_valid + sum_s L_s (L_s + P)
    pl->pairs.assign((size_t)B * 2, 0);
    for (int v = 0; v < 2; ++v) {
        const int S = pl->view[v].max_id + 2;
        for (int b = 0; b < B; ++b) {
            const int32_t *so = seg_off_host[v].data() + (size_t)b * S;
            int64_t c = (int64_t)prefix_len * pl->n_valid[b];
            for (int s = 0; s + 1 < S; ++s) {
                const int64_t L = so[s + 1] - so[s];
                c += L * (L + prefix_len);
            }
            pl->pairs[(size_t)b * 2 + v] = c;
        }
    }

    build_units(pl, seg_off_host);
    if (pl->n_fwd_units > max_units) {  // cannot happen; guards the device array
        mate_plan_destroy(pl);
        return MATE_ERR_INVALID_ARG;
    }
    if (pl->n_fwd_units > 0 &&
        (cudaMemcpyAsync(pl->fwd_units_dev, pl->fwd_units.data(),
                         sizeof(FwdUnit) * pl->n_fwd_units, cudaMemcpyHostToDevice, st) != cudaSuccess ||
         cudaStreamSynchronize(st) != cudaSuccess)) {
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
        for (int h = 0; h < plan->H; ++h)
            pairs[(size_t)b * plan->H + h] = plan->pairs[(size_t)b * 2 + plan->head_view[h]];
    return MATE_OK;
}

int mate_plan_status(const mate_plan_t *plan, void *stream) {
    if (!plan) return MATE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t s[4] = {0, 0, 0, 0};
    if (cudaMemcpyAsync(s, plan->status_dev, sizeof(s), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(plan->status_dev + 1, 0, sizeof(int32_t), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return MATE_ERR_CUDA;
    return s[1] != 0 ? MATE_ERR_TIMEOUT : MATE_OK;
}

static int check_common(const mate_plan_t *plan, int d, int dtype, unsigned flags, bool *use_tc) {
    if (!plan) return MATE_ERR_INVALID_ARG;
    if (dtype != MATE_BF16 && dtype != MATE_F32) return MATE_ERR_UNSUPPORTED;
    if (d <= 0 || d % 8 != 0 || d > 128) return MATE_ERR_UNSUPPORTED;
    const unsigned impl = flags & 3u;
    if (impl == 3u) return MATE_ERR_INVALID_ARG;
    const bool tc_ok = mate::tc_supported(d, dtype);
    if (impl == MATE_IMPL_TCGEN05 && !tc_ok) return MATE_ERR_UNSUPPORTED;
    *use_tc = (impl == MATE_IMPL_TCGEN05) || (impl == MATE_IMPL_AUTO && tc_ok);
    return MATE_OK;
}

int mate_attn_workspace_bytes(const mate_plan_t *plan, int d, int dtype, unsigned flags,
                              size_t *fwd_bytes, size_t *bwd_bytes) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    if (fwd_bytes) *fwd_bytes = use_tc ? mate::tc_fwd_workspace(plan, d) : 0;
    if (bwd_bytes) *bwd_bytes = mate::simt_bwd_workspace(plan);
    return MATE_OK;
}

int mate_attn_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d,
                  int dtype, float scale, void *O, float *LSE, void *workspace,
                  size_t workspace_bytes, unsigned flags, void *stream) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    if (!Q || !K || !V || !O || !LSE) return MATE_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE))
        return MATE_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    if (use_tc) {
        const size_t need = mate::tc_fwd_workspace(plan, d);
        if (need > 0 && (!workspace || workspace_bytes < need)) return MATE_ERR_WORKSPACE;
        if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 255u)) return MATE_ERR_ALIGNMENT;
        return mate::tc_fwd(plan, Q, K, V, scale, O, LSE, workspace, st);
    }
    return mate::simt_fwd(plan, Q, K, V, d, dtype, scale, O, LSE, st);
}

int mate_attn_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V,
                  const void *O, const float *LSE, const void *dO, int d, int dtype, float scale,
                  void *dQ, void *dK, void *dV, void *workspace, size_t workspace_bytes,
                  unsigned flags, void *stream) {
    bool use_tc = false;
    int rc = check_common(plan, d, dtype, flags, &use_tc);
    if (rc != MATE_OK) return rc;
    if (!Q || !K || !V || !O || !LSE || !dO || !dQ || !dK || !dV) return MATE_ERR_INVALID_ARG;
    const void *ptrs[] = {Q, K, V, O, LSE, dO, dQ, dK, dV};
    for (const void *p : ptrs)
        if (!aligned16(p)) return MATE_ERR_ALIGNMENT;
    const size_t need = mate::simt_bwd_workspace(plan);
    if (!workspace || workspace_bytes < need) return MATE_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MATE_ERR_ALIGNMENT;
    return mate::simt_bwd(plan, Q, K, V, O, LSE, dO, d, dtype, scale, dQ, dK, dV, workspace,
                          (cudaStream_t)stream);
}

}  // extern "C"

/*
 * CPU oracle for multi-view (row / column / prefix) attention -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 restatement of the definition in Section 3 of the paper (the sparse head
 * formula and the attention pattern A^i_k).  It builds the explicit N x N boolean mask and runs
 * masked softmax attention and its analytic backward with per-element loops.  Nothing here is
 * blocked, fused or reordered; the CUDA library shares no code with this file and never calls it.
 * Only the tests, the smoke check and the benchmark's cpu_baseline leg may load it.
 *
 * Conventions the paper leaves open (each is a reading, none is printed in the paper):
 *   - Q (the query set) is the first P positions; their row and column ids are 0 (Section 3).
 *   - padding = negative id; padding keys are excluded for every query ("all positions (except
 *     padding)", Section 3); padding queries give O = 0, LSE = -inf and zero gradients.
 *   - masking removes a key from the softmax support (the gather form of the head formula).
 *   - the softmax scale is an argument (the head formula has none, Appendix D divides by
 *     sqrt(embedding_size)).
 *   - a table token whose id is 0 is an ordinary table token (segment 0), not a prefix token.
 * Parity of these conventions is unpinned by the paper; every arithmetic function below is pinned
 * by closed forms, brute force and finite differences in the CPU test-suite.
 *
 * A radius argument > 0 selects the bucketed approximation of Section 3.1 / Appendix D: in a
 * head's own order the first G positions (G >= P, the global section) attend and are attended by
 * everything, the positions behind them are cut into buckets of `radius`, and such a token keeps,
 * of A^i_k, the global section and the keys whose bucket is its own or adjacent.  Pinned by a token-by-token construction of those sets, by the paper's
 * statement that a radius covering the longest row / column gives back the exact pattern, and by
 * brute-force attention over the sets.  radius = 0 is the exact pattern.
 *
 * head_view may also name, per head, the head-independent pattern the paper describes for its
 * closest comparison system (Section 2: attention restricted to the same row and the same column):
 * value 2, see oracle_mask_sat.  Pinned by token-by-token sets and by "row pattern OR column
 * pattern".
 *
 * oracle_cell_mean is the mean-pooling of token logits per table cell of Section 4.1,
 * S(c) = avg over the tokens t of cell c of S(t); pinned by a hand-worked example and per-cell loops.
 *
 * Layouts: Q, K, V, dO, O, dQ, dK, dV are double [B][H][N][d]; LSE is double [B][H][N];
 * row_ids / col_ids are int32 [B][N]; head_view is uint8 [H] (0 = row head, 1 = column head,
 * 2 = row-or-column).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Attention pattern A^i_k of Section 3 as an explicit matrix for one example and one view:
 *   M[k][j] = 1  iff  j is in A_k.
 *   k in Q            -> every position (except padding)
 *   row head, k not Q -> Q union {j : r_j = r_k}
 *   col head, k not Q -> Q union {j : c_j = c_k}
 * Padding rows attend to nothing.  view: 0 = row, 1 = column. */
void oracle_mask(const int32_t *row_ids, const int32_t *col_ids, int N, int P, int view,
                 uint8_t *M) {
    const int32_t *id = view == 0 ? row_ids : col_ids;
    for (int k = 0; k < N; ++k) {
        int k_valid = id[k] >= 0;
        int k_in_Q = k < P;
        for (int j = 0; j < N; ++j) {
            int j_valid = id[j] >= 0;
            int j_in_Q = j < P;
            int in_A;
            if (k_in_Q)
                in_A = 1;                                  /* {1..n} */
            else
                in_A = j_in_Q || (!j_in_Q && id[j] == id[k]); /* Q u {j : id_j = id_k} */
            M[(size_t)k * N + j] = (uint8_t)(k_valid && j_valid && in_A);
        }
    }
}

/* The head-independent pattern the paper describes for its closest comparison system (Section 2,
 * related work: an attention mask restricting attention to tokens of the same row and of the same
 * column): a table token attends the query/text prefix and every table token that shares its row
 * OR its column; prefix tokens attend everything; padding as above.  One pattern for all heads. */
void oracle_mask_sat(const int32_t *row_ids, const int32_t *col_ids, int N, int P, uint8_t *M) {
    for (int k = 0; k < N; ++k) {
        int k_valid = row_ids[k] >= 0 && col_ids[k] >= 0;
        int k_in_Q = k < P;
        for (int j = 0; j < N; ++j) {
            int j_valid = row_ids[j] >= 0 && col_ids[j] >= 0;
            int j_in_Q = j < P;
            int in_A = k_in_Q || j_in_Q || row_ids[j] == row_ids[k] || col_ids[j] == col_ids[k];
            M[(size_t)k * N + j] = (uint8_t)(k_valid && j_valid && in_A);
        }
    }
}

void oracle_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int P, int view,
                 int max_id, int32_t *perm, int32_t *inv_perm, int32_t *seg_off);

/* Bucketed pattern (Section 3.1, Appendix D).  Every head orders the tokens its own way
 * (oracle_plan).  The first G positions of that order are the global section: they attend every
 * position and every position attends them (G >= P: the prefix, and, when G is larger, the table
 * tokens that come first in the head's order; Appendix A.2 uses G = 116).  The positions behind it
 * are cut into buckets of `radius`; such a token attends the global section and, within A_k, the
 * tokens of its own bucket and of the two adjacent buckets.  radius <= 0: the exact pattern (G is
 * then without effect); G < P is read as G = P. */
void oracle_mask_bucketed(const int32_t *row_ids, const int32_t *col_ids, int N, int P, int view,
                          int radius, int G, uint8_t *M) {
    oracle_mask(row_ids, col_ids, N, P, view, M);
    if (radius <= 0) return;
    if (G < P) G = P;
    const int32_t *id = view == 0 ? row_ids : col_ids;
    int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    int32_t seg[2];
    oracle_plan(row_ids, col_ids, 1, N, P, view, 0, perm, pos, seg);
    for (int k = 0; k < N; ++k)
        for (int j = 0; j < N; ++j) {
            if (id[k] < 0 || id[j] < 0) continue; /* padding stays excluded */
            if (pos[k] < G || pos[j] < G) {
                M[(size_t)k * N + j] = 1; /* to and from the global section */
            } else {
                int bucket_k = (pos[k] - G) / radius, bucket_j = (pos[j] - G) / radius;
                if (abs(bucket_k - bucket_j) > 1) M[(size_t)k * N + j] = 0;
            }
        }
    free(perm);
    free(pos);
}

/* Mask of one pattern id as used in head_view: 0 = row head, 1 = column head (both Section 3, or
 * their bucketed form when radius > 0), 2 = the head-independent row-OR-column pattern. */
static void mask_of_pattern(const int32_t *row_ids, const int32_t *col_ids, int N, int P, int pattern,
                            int radius, int G, uint8_t *M) {
    if (pattern == 2)
        oracle_mask_sat(row_ids, col_ids, N, P, M);
    else
        oracle_mask_bucketed(row_ids, col_ids, N, P, pattern, radius, G, M);
}

/* Number of unmasked (query, key) pairs per (b, h): popcount of the mask. out: int64 [B][H]. */
void oracle_useful_pairs(const int32_t *row_ids, const int32_t *col_ids, int B, int H, int N, int P,
                         const uint8_t *head_view, int radius, int G, int64_t *out) {
    uint8_t *M = (uint8_t *)malloc((size_t)N * N);
    for (int b = 0; b < B; ++b)
        for (int view = 0; view < 3; ++view) {
            mask_of_pattern(row_ids + (size_t)b * N, col_ids + (size_t)b * N, N, P, view, radius, G, M);
            int64_t c = 0;
            for (size_t i = 0; i < (size_t)N * N; ++i) c += M[i];
            for (int h = 0; h < H; ++h)
                if (head_view[h] == view) out[(size_t)b * H + h] = c;
        }
    free(M);
}

/* Forward of one query row k: softmax over the support {j : M[k][j]} of scale * q_k . k_j,
 * output = sum_j prob_j v_j (the head formula of Section 3 after the projections).
 * Returns LSE_k = m_k + ln Z_k, writes O_k (length d).  s is scratch of length N. */
static double fwd_row(const double *q, const double *K, const double *V, const uint8_t *Mk, int N,
                      int d, double scale, double *s, double *o) {
    double m = -INFINITY;
    for (int j = 0; j < N; ++j) {
        if (!Mk[j]) continue;
        double acc = 0.0;
        for (int e = 0; e < d; ++e) acc += q[e] * K[(size_t)j * d + e];
        s[j] = scale * acc;
        if (s[j] > m) m = s[j];
    }
    for (int e = 0; e < d; ++e) o[e] = 0.0;
    if (m == -INFINITY) return -INFINITY; /* empty support: padding row */
    double Z = 0.0;
    for (int j = 0; j < N; ++j)
        if (Mk[j]) Z += exp(s[j] - m);
    for (int j = 0; j < N; ++j) {
        if (!Mk[j]) continue;
        double p = exp(s[j] - m) / Z;
        for (int e = 0; e < d; ++e) o[e] += p * V[(size_t)j * d + e];
    }
    return m + log(Z);
}

int oracle_fwd(const double *Q, const double *K, const double *V, const int32_t *row_ids,
               const int32_t *col_ids, int B, int H, int N, int d, int P, const uint8_t *head_view,
               double scale, int radius, int G, double *O, double *LSE) {
    uint8_t *M[3];
    for (int v = 0; v < 3; ++v) M[v] = (uint8_t *)malloc((size_t)N * N);
    if (!M[0] || !M[1] || !M[2]) return -1;
    for (int b = 0; b < B; ++b) {
        for (int view = 0; view < 3; ++view)
            mask_of_pattern(row_ids + (size_t)b * N, col_ids + (size_t)b * N, N, P, view, radius, G, M[view]);
#pragma omp parallel
        {
            double *s = (double *)malloc(sizeof(double) * (size_t)N);
#pragma omp for collapse(2) schedule(dynamic, 16)
            for (int h = 0; h < H; ++h)
                for (int k = 0; k < N; ++k) {
                    size_t bh = (size_t)b * H + h;
                    const uint8_t *Mk = M[head_view[h]] + (size_t)k * N;
                    LSE[bh * N + k] = fwd_row(Q + (bh * N + k) * d, K + bh * N * d, V + bh * N * d,
                                              Mk, N, d, scale, s, O + (bh * N + k) * d);
                }
            free(s);
        }
    }
    for (int v = 0; v < 3; ++v) free(M[v]);
    return 0;
}

/* Analytic backward of the forward above.  With P_kj = exp(s_kj - LSE_k) on the mask, else 0:
 *   D_k   = sum_e dO_ke O_ke
 *   dV_j  = sum_k P_kj dO_k
 *   dP_kj = dO_k . V_j
 *   dS_kj = P_kj (dP_kj - D_k)
 *   dQ_k  = scale * sum_j dS_kj K_j
 *   dK_j  = scale * sum_k dS_kj Q_k
 * O and LSE are recomputed here from Q, K, V, so the result depends on no forward output. */
int oracle_bwd(const double *Q, const double *K, const double *V, const double *dO,
               const int32_t *row_ids, const int32_t *col_ids, int B, int H, int N, int d, int P,
               const uint8_t *head_view, double scale, int radius, int G, double *dQ, double *dK, double *dV) {
    uint8_t *M[3];
    for (int v = 0; v < 3; ++v) M[v] = (uint8_t *)malloc((size_t)N * N);
    double *LSE = (double *)malloc(sizeof(double) * (size_t)H * N);
    double *D = (double *)malloc(sizeof(double) * (size_t)H * N);
    if (!M[0] || !M[1] || !M[2] || !LSE || !D) return -1;
    for (int b = 0; b < B; ++b) {
        for (int view = 0; view < 3; ++view)
            mask_of_pattern(row_ids + (size_t)b * N, col_ids + (size_t)b * N, N, P, view, radius, G, M[view]);
        /* pass 1, one query row at a time: LSE_k, D_k, dQ_k */
#pragma omp parallel
        {
            double *s = (double *)malloc(sizeof(double) * (size_t)N);
            double *o = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for collapse(2) schedule(dynamic, 16)
            for (int h = 0; h < H; ++h)
                for (int k = 0; k < N; ++k) {
                    size_t bh = (size_t)b * H + h;
                    const uint8_t *Mk = M[head_view[h]] + (size_t)k * N;
                    const double *q = Q + (bh * N + k) * d;
                    const double *Kh = K + bh * N * d, *Vh = V + bh * N * d;
                    const double *dOk = dO + (bh * N + k) * d;
                    double *dQk = dQ + (bh * N + k) * d;
                    double lse = fwd_row(q, Kh, Vh, Mk, N, d, scale, s, o);
                    double Dk = 0.0;
                    for (int e = 0; e < d; ++e) Dk += dOk[e] * o[e];
                    LSE[(size_t)h * N + k] = lse;
                    D[(size_t)h * N + k] = Dk;
                    for (int e = 0; e < d; ++e) dQk[e] = 0.0;
                    for (int j = 0; j < N; ++j) {
                        if (!Mk[j]) continue;
                        double Pkj = exp(s[j] - lse);
                        double dP = 0.0;
                        for (int e = 0; e < d; ++e) dP += dOk[e] * Vh[(size_t)j * d + e];
                        double dS = Pkj * (dP - Dk);
                        for (int e = 0; e < d; ++e) dQk[e] += scale * dS * Kh[(size_t)j * d + e];
                    }
                }
            free(s);
            free(o);
        }
        /* pass 2, one key row at a time: dV_j, dK_j (sums over the queries k with M[k][j]) */
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
        for (int h = 0; h < H; ++h)
            for (int j = 0; j < N; ++j) {
                size_t bh = (size_t)b * H + h;
                const uint8_t *Mv = M[head_view[h]];
                const double *Qh = Q + bh * N * d, *dOh = dO + bh * N * d;
                const double *kj = K + (bh * N + j) * d, *vj = V + (bh * N + j) * d;
                double *dKj = dK + (bh * N + j) * d, *dVj = dV + (bh * N + j) * d;
                for (int e = 0; e < d; ++e) dKj[e] = dVj[e] = 0.0;
                for (int k = 0; k < N; ++k) {
                    if (!Mv[(size_t)k * N + j]) continue;
                    const double *q = Qh + (size_t)k * d, *dOk = dOh + (size_t)k * d;
                    double acc = 0.0, dP = 0.0;
                    for (int e = 0; e < d; ++e) acc += q[e] * kj[e];
                    for (int e = 0; e < d; ++e) dP += dOk[e] * vj[e];
                    double Pkj = exp(scale * acc - LSE[(size_t)h * N + k]);
                    double dS = Pkj * (dP - D[(size_t)h * N + k]);
                    for (int e = 0; e < d; ++e) {
                        dVj[e] += Pkj * dOk[e];
                        dKj[e] += scale * dS * q[e];
                    }
                }
            }
    }
    for (int v = 0; v < 3; ++v) free(M[v]);
    free(LSE);
    free(D);
    return 0;
}

/* Per-view token order (Section 3.1: a row-order or column-order traversal, data dependent but
 * deterministic).  Sort key: (0, 0) for prefix tokens, (1, id) for valid table tokens, (2, 0) for
 * padding; ties keep the original order, which makes the order unique. */
typedef struct {
    int32_t cls, id, pos;
} sort_key_t;

static int cmp_key(const void *a, const void *b) {
    const sort_key_t *x = (const sort_key_t *)a, *y = (const sort_key_t *)b;
    if (x->cls != y->cls) return x->cls < y->cls ? -1 : 1;
    if (x->id != y->id) return x->id < y->id ? -1 : 1;
    return x->pos < y->pos ? -1 : (x->pos > y->pos);
}

/* perm[b][t] = original index of the token at position t of the view order; inv_perm is its
 * inverse; seg_off[b][i] = P + #{valid table tokens with id < i}, i = 0 .. max_id + 1, so the
 * tokens with id s sit at view positions [seg_off[s], seg_off[s+1]). */
void oracle_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int P, int view,
                 int max_id, int32_t *perm, int32_t *inv_perm, int32_t *seg_off) {
    sort_key_t *keys = (sort_key_t *)malloc(sizeof(sort_key_t) * (size_t)N);
    for (int b = 0; b < B; ++b) {
        const int32_t *id = (view == 0 ? row_ids : col_ids) + (size_t)b * N;
        for (int k = 0; k < N; ++k) {
            keys[k].pos = k;
            if (k < P) {
                keys[k].cls = 0;
                keys[k].id = 0;
            } else if (id[k] >= 0) {
                keys[k].cls = 1;
                keys[k].id = id[k];
            } else {
                keys[k].cls = 2;
                keys[k].id = 0;
            }
        }
        qsort(keys, (size_t)N, sizeof(sort_key_t), cmp_key); /* total order: pos breaks ties */
        for (int t = 0; t < N; ++t) {
            perm[(size_t)b * N + t] = keys[t].pos;
            inv_perm[(size_t)b * N + keys[t].pos] = t;
        }
        for (int i = 0; i <= max_id + 1; ++i) {
            int32_t c = 0;
            for (int k = P; k < N; ++k)
                if (id[k] >= 0 && id[k] < i) ++c;
            seg_off[(size_t)b * (max_id + 2) + i] = P + c;
        }
    }
    free(keys);
}

/* Mean-pooling of per-token logits over the tokens of each table cell (Section 4.1:
 * S(c) = avg_{t in c} S(t)).  A cell is the set of table tokens (positions >= P with valid ids)
 * that share a (row id, column id) pair.  mean: double [B][max_row_id+1][max_col_id+1], count:
 * int32 of the same shape; a pair that no token carries gets count 0 and mean 0. */
void oracle_cell_mean(const double *logits, const int32_t *row_ids, const int32_t *col_ids, int B, int N,
                      int P, int max_row_id, int max_col_id, double *mean, int32_t *count) {
    const int R = max_row_id + 1, Cn = max_col_id + 1;
    for (int b = 0; b < B; ++b)
        for (int r = 0; r < R; ++r)
            for (int c = 0; c < Cn; ++c) {
                double sum = 0.0;
                int32_t n = 0;
                for (int t = P; t < N; ++t)
                    if (row_ids[(size_t)b * N + t] == r && col_ids[(size_t)b * N + t] == c) {
                        sum += logits[(size_t)b * N + t];
                        ++n;
                    }
                mean[((size_t)b * R + r) * Cn + c] = n ? sum / n : 0.0;
                count[((size_t)b * R + r) * Cn + c] = n;
            }
}

/*
 * libmate -- multi-view (row head / column head / global prefix) sparse self-attention for
 * flattened tables, hand-written CUDA for sm_100a.
 *
 * The operation is the one defined in Section 3 of "MATE: Multi-view Attention for Table
 * Transformer Efficiency": for head i and token position k the output is a softmax-weighted sum of
 * the values of the positions in the attention pattern A^i_k,
 *     k in Q (the query/text prefix)  ->  A = every position (except padding)
 *     row head,    k not in Q         ->  A = Q  u  { j : r_j = r_k }
 *     column head, k not in Q         ->  A = Q  u  { j : c_j = c_k }
 * applied after the Q/K/V projections (Q, K, V are inputs here).  Section 3.1's observation that
 * every head may traverse the tokens in its own data-dependent, deterministic order is what
 * mate_plan pre-computes: in a head's view order each table token's keys are one contiguous
 * segment plus the prefix block.
 *
 * Conventions (the paper leaves them open):
 *   - Q is the first prefix_len positions; their row and column ids must be 0.
 *   - a negative id marks padding (both arrays must agree).  Padding keys are never attended;
 *     padding query rows return O = 0, LSE = -inf and zero gradients; values stored at padding
 *     positions are ignored.
 *   - a table token whose id is 0 is an ordinary table token (segment 0).
 *   - masking removes a key from the softmax support; `scale` multiplies q.k before the softmax.
 *   - LSE is the natural-log logsumexp of the scaled scores over A.
 *
 * All tensor pointers are DEVICE pointers unless a comment says "host".  The library never keeps
 * or frees caller memory.  Every call returns a status (0 = MATE_OK, negative = error); nothing
 * throws across this boundary.  Calls taking a `stream` (a cudaStream_t passed as void*) enqueue
 * work on it and return without waiting, except mate_plan, which waits for its own kernels.
 */
#ifndef MATE_H_
#define MATE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mate_plan_s mate_plan_t;

enum {
    MATE_OK = 0,
    MATE_ERR_INVALID_ARG = -1, /* null pointer, bad size, ids that break the conventions above     */
    MATE_ERR_UNSUPPORTED = -2, /* head dim / dtype / implementation not available for these sizes   */
    MATE_ERR_ALIGNMENT = -3,   /* a tensor pointer is not 16-byte aligned                           */
    MATE_ERR_CUDA = -4,        /* a CUDA runtime call failed (the CUDA error is left in place)      */
    MATE_ERR_TIMEOUT = -5,     /* a bounded wait inside a kernel expired (see mate_plan_status)     */
    MATE_ERR_NOMEM = -6,       /* host or device allocation failed                                  */
    MATE_ERR_WORKSPACE = -7,   /* workspace pointer null or smaller than mate_attn_workspace_bytes  */
    MATE_ERR_TOO_LARGE = -8    /* problem exceeds the built-in scratch of mate_attn_bwd_noalloc      */
};

enum { MATE_BF16 = 0, MATE_F32 = 1 };          /* element type of Q, K, V, O, dO, dQ, dK, dV */
enum { MATE_VIEW_ROW = 0, MATE_VIEW_COL = 1 }; /* entries of head_view                      */

/* flags for mate_attn_fwd / mate_attn_bwd: which implementation runs.
 *   AUTO     tensor-core (tcgen05) kernels when dtype = bf16 and d = 64, otherwise the SIMT kernels
 *   SIMT     one-warp-per-row fp32-arithmetic kernels (any dtype, d <= 128): the debug path
 *   TCGEN05  tensor-core kernels or MATE_ERR_UNSUPPORTED */
enum { MATE_IMPL_AUTO = 0, MATE_IMPL_SIMT = 1, MATE_IMPL_TCGEN05 = 2 };

/* further flag bits (or-ed to the implementation choice):
 *   VIEW_ORDER   (mate_attn_fwd only) Q, K, V are laid out, head by head, in that head's own order
 *                (row b, h, t of a tensor holds the token at position t of the order mate_plan computed
 *                for the head's view), and O and LSE are returned in the same order: what a producer
 *                that writes its projections through the plan's order provides (Section 3.1: the
 *                reordering can be folded into the neighbouring steps).  No gather, no scatter; the
 *                tensor-core kernel then fetches every full K/V tile with bulk tensor copies.  Not for
 *                mate_plan_sat plans and not for mate_attn_bwd (MATE_ERR_UNSUPPORTED).
 *   BULK_TILES   the tensor-core forward fetches the K/V tiles that are contiguous in the tensors -- the
 *                prefix block of every head and, for a row-major table, every tile of the row view --
 *                with bulk tensor copies (one per tile and matrix) instead of row-by-row gathers.  Same
 *                results bit for bit.  This is the default wherever the driver provides tensor maps,
 *                so the bit only states it.
 *   GATHER_TILES every K/V tile is gathered row by row.  (Timed back to back on sequences of 512 to
 *                8192 positions, bulk copies are 2-3 % faster on two workloads, equal on one and
 *                0.6 % slower on one.)  Both bits together: MATE_ERR_INVALID_ARG. */
enum { MATE_FLAG_VIEW_ORDER = 4, MATE_FLAG_BULK_TILES = 8, MATE_FLAG_GATHER_TILES = 16 };

const char *mate_status_string(int status);

/* Pre-computes, for both views, the per-head token order of Section 3.1 (Figure 2): a stable
 * counting sort of the positions by (prefix, table id, padding), i.e. the row-order / column-order
 * traversal of the table, together with the segment offsets and the tile work-lists the attention
 * kernels walk.  Integer work; the result is unique (ties keep the original order).
 *
 *   row_ids, col_ids  device int32 [B, N]
 *   prefix_len        |Q|, 0 <= prefix_len <= N
 *   head_view         HOST uint8 [H], MATE_VIEW_ROW or MATE_VIEW_COL per head (any mix, one view
 *                     may have no head)
 *   max_row_id, max_col_id   inclusive upper bounds of the non-negative ids
 *   out               receives a plan owned by the library; free it with mate_plan_destroy
 *
 * The plan can be reused for any number of forward/backward calls, layers and head dims, on the
 * device that was current when it was made (calls with another device current return
 * MATE_ERR_INVALID_ARG).  It also holds a few scheduling counters of the tensor-core forward, so
 * calls that use ONE plan -- mate_attn_fwd, mate_plan_status -- must not overlap on the GPU: put
 * them on one stream or order them with events.  Work that should overlap (two streams) needs one
 * plan per stream; mate_attn_bwd keeps its counters in its workspace and only needs separate
 * workspaces.  Runs its kernels on `stream` and waits for them (it allocates device memory, so call
 * it outside a stream capture).  Ids that break the conventions give MATE_ERR_INVALID_ARG and no
 * plan. */
int mate_plan(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len,
              const uint8_t *head_view, int H, int max_row_id, int max_col_id, void *stream,
              mate_plan_t **out);

/* The same plan for the bucketed, approximate form of the pattern (Section 3.1 and Appendix D: a
 * global section G, which here is the prefix, and a local section cut into buckets of R positions
 * of each head's own order; the paper uses R = 42).  In a head's order the positions behind the
 * prefix form buckets of `radius` consecutive positions; a table token attends the prefix and,
 * of its own row / column, only the keys in its own bucket and the two adjacent ones.  Prefix
 * tokens still attend every non-padding position.  The order (perm, inv_perm, seg_off) is that
 * of mate_plan; only the key ranges, the work-lists and the pair counts differ.  The pattern
 * stays symmetric, so the forward and the backward calls take such a plan unchanged.  A radius
 * at least as long as the longest row / column segment gives back the exact pattern, as the
 * paper notes; radius = 0 means exactly that (mate_plan); radius < 0 is MATE_ERR_INVALID_ARG.
 * All other arguments, ownership and errors as for mate_plan. */
int mate_plan_bucketed(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len,
                       const uint8_t *head_view, int H, int max_row_id, int max_col_id, int radius,
                       void *stream, mate_plan_t **out);

/* The bucketed form with a global section that may be longer than the prefix (Section 3.1: the first
 * G tokens of a head's order attend to and from everything, with G at least the length of the
 * question; Appendix A.2 uses G = 116, R = 42): the first global_len[b] positions of each head's
 * own order -- the prefix and, beyond it, the table tokens that come first in that order -- see
 * every non-padding position and are seen by all of them; the positions behind are cut into
 * buckets of `radius`, counted from global_len[b], and attend the global section plus, of their own
 * row / column, their own bucket and the two adjacent ones.  prefix_len and global_len are HOST
 * int32 [B] arrays with prefix_len[b] <= global_len[b] <= N; radius > 0.  global_len = prefix_len
 * is mate_plan_varlen.  All other arguments, ownership and errors as for mate_plan. */
int mate_plan_bucketed_global(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                              const int32_t *global_len, const uint8_t *head_view, int H, int max_row_id,
                              int max_col_id, int radius, void *stream, mate_plan_t **out);

/* The same with one prefix length per example (the paper's inputs are a question or a passage of
 * varying length followed by the table, Section 3 and Section 5; its formula takes the set Q per
 * example).  prefix_len is a HOST int32 [B] array, 0 <= prefix_len[b] <= N; examples of different
 * total length are padded at the tail with negative ids as for mate_plan.  radius as for
 * mate_plan_bucketed (0 = the exact pattern).  mate_plan and mate_plan_bucketed are this call with
 * B equal entries.  All other arguments, ownership and errors as for mate_plan. */
int mate_plan_varlen(const int32_t *row_ids, const int32_t *col_ids, int B, int N, const int32_t *prefix_len,
                     const uint8_t *head_view, int H, int max_row_id, int max_col_id, int radius,
                     void *stream, mate_plan_t **out);

/* Packed batches: examples of different length stored one behind the other, without padding
 * (the paper's inputs are a question or a passage followed by a table of any size, Section 3 and
 * Section 5; the attention of one example never reaches another).  row_ids, col_ids: DEVICE int32
 * [T], example b owning the tokens cu_seqlens[b] .. cu_seqlens[b + 1] - 1; cu_seqlens: HOST int32
 * [B + 1], cu_seqlens[0] = 0, non-decreasing, cu_seqlens[B] = T; prefix_len: HOST int32 [B],
 * 0 <= prefix_len[b] <= length of example b.  Negative ids inside an example still mark padding.
 * With such a plan every tensor of mate_attn_fwd / mate_attn_bwd / mate_attn_bwd_noalloc is
 * [H, T, d] (LSE [H, T]) in place of [B, H, N, d] ([B, H, N]); the plan's N (mate_plan_get,
 * mate_attn_workspace_bytes) is the longest example.  The exact pattern only; MATE_FLAG_VIEW_ORDER
 * and mate_cell_mean return MATE_ERR_UNSUPPORTED.  Ownership and errors as for mate_plan. */
int mate_plan_packed(const int32_t *row_ids, const int32_t *col_ids, int B, const int32_t *cu_seqlens,
                     const int32_t *prefix_len, const uint8_t *head_view, int H, int max_row_id, int max_col_id,
                     void *stream, mate_plan_t **out);

/* Plan of the head-independent pattern that the paper describes for its closest comparison system
 * (Section 2, related work: attention restricted to the tokens of the same row and of the same
 * column; one pattern for all heads): a table token attends the prefix and every table token that
 * shares its row id OR its column id; prefix tokens attend every non-padding position; padding as
 * for mate_plan.  The pattern is evaluated exactly, in three passes of the ordinary kernels over
 * disjoint key sets -- (prefix and own row), (rest of the own column in front of the own cell),
 * (rest of the column behind it) -- whose outputs are merged through their logsumexps and whose
 * gradients are summed; mate_attn_workspace_bytes accounts for the passes' intermediate results.
 * The returned plan is used with mate_attn_fwd / mate_attn_bwd like any other (all H heads share
 * the pattern); mate_plan_get returns the row / column orders of mate_plan; mate_plan_useful_pairs
 * counts the pattern's pairs.  mate_attn_bwd_noalloc does not take such a plan
 * (MATE_ERR_UNSUPPORTED).  Arguments, ownership and errors as for mate_plan;
 * (max_row_id + 1) * (max_col_id + 1) must not exceed 2^28. */
int mate_plan_sat(const int32_t *row_ids, const int32_t *col_ids, int B, int N, int prefix_len, int H,
                  int max_row_id, int max_col_id, void *stream, mate_plan_t **out);

/* Copies one view's order to HOST arrays (any pointer may be null to skip it):
 *   perm      int32 [B, N]          perm[b][t] = original position of the t-th token of the view
 *   inv_perm  int32 [B, N]          inverse of perm
 *   seg_off   int32 [B, max_id+2]   tokens with id s occupy view positions [seg_off[s], seg_off[s+1]);
 *                                   seg_off[0] = prefix_len (of the example), seg_off[max_id+1] = number of
 *                                   non-padding tokens */
int mate_plan_get(const mate_plan_t *plan, int view, int32_t *perm, int32_t *inv_perm,
                  int32_t *seg_off);

/* Number of unmasked (query, key) pairs per example and head (the O(ng + nb) count of Table 1):
 * HOST int64 [B, H].  Forward work is 4*d flops per pair, backward 10*d. */
int mate_plan_useful_pairs(const mate_plan_t *plan, int64_t *pairs);

/* Waits for `stream` and returns MATE_ERR_TIMEOUT if any kernel that used this plan gave up on a
 * bounded wait since the last call (its outputs are then undefined), MATE_ERR_CUDA if the stream
 * reports an error, else MATE_OK. */
int mate_plan_status(const mate_plan_t *plan, void *stream);

/* Test hook (the paper has no counterpart): launches a one-thread kernel that waits, with the
 * bounded helper the attention kernels use and a limit of a few tries (a few microseconds each), on a
 * barrier that nothing arrives on; the wait gives up, the kernel raises the plan's time-out word as
 * the attention kernels would, and returns.  The next mate_plan_status on the plan then reports
 * MATE_ERR_TIMEOUT once, and the plan stays usable.  Lets the time-out path be exercised without
 * making any real kernel wait in vain. */
int mate_debug_expire_wait(const mate_plan_t *plan, void *stream);

int mate_plan_destroy(mate_plan_t *plan);

/* Scratch sizes (bytes) the caller must provide to mate_attn_fwd / mate_attn_bwd for head dim d,
 * element type dtype and implementation `flags`.  Either size may be 0. */
int mate_attn_workspace_bytes(const mate_plan_t *plan, int d, int dtype, unsigned flags,
                              size_t *fwd_bytes, size_t *bwd_bytes);

/* Forward: the head formula of Section 3 for every (b, h, k).
 *   Q, K, V   [B, H, N, d] contiguous, dtype elements, 16-byte aligned
 *   O         [B, H, N, d] same type, fully overwritten, original token order
 *   LSE       float32 [B, H, N]
 *   workspace device scratch of at least fwd_bytes (may be null when that is 0), 256-byte aligned;
 *             contents are undefined afterwards; concurrent calls need separate workspaces AND
 *             separate plans (see mate_plan)
 *   scale     any finite value.  The tensor-core kernels need scale > 0; with MATE_IMPL_AUTO other
 *             values run on the SIMT kernels, with MATE_IMPL_TCGEN05 they give MATE_ERR_UNSUPPORTED
 * d must be a multiple of 8 and at most 128.  Asynchronous on `stream`. */
int mate_attn_fwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V, int d,
                  int dtype, float scale, void *O, float *LSE, void *workspace,
                  size_t workspace_bytes, unsigned flags, void *stream);

/* Backward of mate_attn_fwd (derived from the Section 3 head formula; the paper states no
 * backward): given O and LSE of the forward call and dO, writes dQ, dK, dV (fully overwritten,
 * no accumulation into previous contents).  Same layouts, types and rules as the forward. */
int mate_attn_bwd(const mate_plan_t *plan, const void *Q, const void *K, const void *V,
                  const void *O, const float *LSE, const void *dO, int d, int dtype, float scale,
                  void *dQ, void *dK, void *dV, void *workspace, size_t workspace_bytes,
                  unsigned flags, void *stream);

/* Per-cell mean of token scores (cell-selection stage, Section 4.1: the score of a cell is the
 * mean of the scores of its tokens, S(c) = avg_{t in c} S(t)).  A cell is the set of table tokens
 * (positions behind the prefix, non-negative ids) that share a (row id, column id) pair.
 *   logits   float32 [B, N], one score per token (prefix and padding positions are ignored)
 *   col_ids  the int32 [B, N] column ids the plan was made from
 *   mean     float32 [B, max_row_id + 1, max_col_id + 1], fully overwritten; 0 where no token
 *            carries the pair
 *   count    int32, same shape, tokens per cell; may be null
 * Uses the row view of the plan (a row's tokens are contiguous there).  The sum of a cell runs
 * over its tokens in original order, so the result is the same on every launch.  Asynchronous on
 * `stream`; no workspace. */
int mate_cell_mean(const mate_plan_t *plan, const float *logits, const int32_t *col_ids, float *mean,
                   int32_t *count, void *stream);

/* Backward for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving or training loop whose
 * framework has handed all device memory to its own pool, a latency-critical section where the
 * device-wide synchronisation of cudaMalloc/cudaFree is not acceptable, or a plug-in that gets
 * tensors but no allocator.  Such a caller cannot create the workspace mate_attn_bwd asks for.
 *
 * Same arguments, results and rules as mate_attn_bwd with flags = MATE_IMPL_SIMT, minus the
 * workspace: the scratch (one float per (example, head, position)) lives in a 4 MiB array that is
 * part of the library itself, so every GPU that loads libmate holds it until the process exits.
 * The call makes no cudaMalloc, cudaFree or other allocating call.
 *
 *   limit       B * H * N <= 1,048,576; larger problems return MATE_ERR_TOO_LARGE and launch nothing
 *   first call  the first call on each device looks up the array's device address (with that
 *               device current); make that first call outside any stream capture
 *   sharing     all calls on a device use the same array.  Its contents are left over from the
 *               previous call; the kernels overwrite every element they later read, so nothing
 *               depends on them.  Two calls that overlap on the GPU (different streams) race on
 *               the array: serialise them.
 * The plan is an input like the tensors; create it ahead of time with mate_plan. */
int mate_attn_bwd_noalloc(const mate_plan_t *plan, const void *Q, const void *K, const void *V,
                          const void *O, const float *LSE, const void *dO, int d, int dtype,
                          float scale, void *dQ, void *dK, void *dV, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MATE_H_ */

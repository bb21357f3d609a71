/*
 * csp.h -- C interface of the B200 (sm_100a) library for the scoring-and-compaction pass of
 * Cross-Self Pruning (CSP), the KV-cache pruning method of "Cross-Self KV Cache Pruning for
 * Efficient Vision-Language Inference".
 *
 * One call handles one layer: every sequence b < batch and every KV head h < n_kv_heads is an
 * independent unit.  For each unit the path is
 *
 *   score    logits of the last W queries against every cached key (Eq. 5), each row normalised
 *            by n-softmax over all keys it can see (Eq. 7), the last R key columns dropped
 *            (Section 3.2, "A[-O:, :-R]"), rows averaged over the query heads of the KV group,
 *            then summed over the query axis separately for queries with the same modality
 *            label as the key (intra, "self") and a different one (inter, "cross") (Eq. 1);
 *   select   a top-K over each of the two score vectors (Eq. 2), the two masks combined (Eq. 3),
 *            the kept positions listed in ascending order followed by the last R positions;
 *   compact  K, V and the labels gathered by that list (Eq. 4).
 *
 * Algorithm 1 is `csp_prune_layer`; a cache shorter than its budget T is passed through.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless its name ends in `_host`.  The caller owns every
 *    buffer.  The library never allocates or frees device memory and, except for
 *    csp_device_status and csp_prune_layer_host, never synchronises: work is enqueued on the
 *    given CUDA stream (a cudaStream_t passed as void*; NULL is the default stream).
 *  - Inputs are read-only.  Outputs must not overlap inputs or each other, with one exception:
 *    compaction in place (k_out the very tensor k and v_out the very tensor v), see csp_compact.
 *  - Host threads: entry points may be called from several host threads at once, on the same or on
 *    different devices, as long as calls that can overlap on the GPU use different workspaces and
 *    outputs.  What the library remembers between calls (per-device launch settings) is synchronised
 *    internally.  csp_prune_layer_static is the exception: all its calls share one scratch array.
 *  - Tensors are described by a base pointer and ELEMENT strides; the innermost (head_dim)
 *    axis is contiguous.  Base pointers and row starts must be 16-byte aligned (every stride
 *    times the element size a multiple of 16 bytes).
 *  - Errors the host can see (null pointer, unsupported shape, misalignment, workspace too
 *    small, wrong GPU) are returned at once and nothing is enqueued.  Conditions only the
 *    device can see are OR-ed into a status word at the start of the workspace
 *    (CSP_DEV_* bits) and read back with csp_device_status; kernels never trap and every wait
 *    inside them is bounded.
 *  - Labels: modality[b, (h,) t] is a small integer; 0 is text, anything else is visual;
 *    "intra" means equal labels.  After a prune the labels differ per head, so they carry a
 *    head stride (0 when all heads of a sequence share one row of labels).
 */
#ifndef CSP_H
#define CSP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CSP_OK = 0,
    CSP_ERR_INVALID_ARG = 1,  /* null pointer, negative size */
    CSP_ERR_UNSUPPORTED = 2,  /* shape, dtype, stride or mode this build has no kernel for */
    CSP_ERR_WORKSPACE = 3,    /* workspace missing or smaller than csp_workspace_bytes */
    CSP_ERR_ARCH = 4,         /* the current device is not compute capability 10.x */
    CSP_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed (launch, copy, descriptor) */
    CSP_ERR_TIMEOUT = 6       /* a bounded wait inside a kernel expired (from csp_device_status) */
} csp_status;

typedef enum { CSP_F32 = 0, CSP_BF16 = 1 } csp_dtype;

/* Eq. 3 prints M = M^s AND M^c; Sections 3.2 and 5.1 describe the kept set as both selections
 * together, with overlap saving budget.  OR is the default reading, AND the printed one. */
typedef enum { CSP_COMBINE_OR = 0, CSP_COMBINE_AND = 1 } csp_combine;

/* SEGMENTED: four budgets per sequence, a top-K of the intra score and of the inter score among
 * the text keys and among the visual keys.  GLOBAL: the paper's literal K^s and K^c over all keys.
 * OVERALL: the comparison arm of the paper's ablation ("Influence of n-softmax"): one budget per
 * sequence, a single top-K on the overall selection function s + c (fp32 sum), no split. */
typedef enum { CSP_SELECT_SEGMENTED = 0, CSP_SELECT_GLOBAL = 1, CSP_SELECT_OVERALL = 2 } csp_select_mode;

/* PER_KV: one selection per KV head from the mean over its query-head group.
 * MEAN_ALL: one selection per sequence from the mean over every head (Section 3.2). */
typedef enum { CSP_HEADS_PER_KV = 0, CSP_HEADS_MEAN_ALL = 1 } csp_head_reduce;

/* bits of the device status word */
enum {
    CSP_DEV_K_CLAMPED = 1,  /* a budget exceeded its candidate count (or was negative) and was clamped */
    CSP_DEV_CAPACITY = 2,   /* a unit's kept rows did not fit out_capacity; its n_out is -1 */
    CSP_DEV_TIMEOUT = 4,    /* a bounded wait expired; outputs of that call are not valid */
    CSP_DEV_BAD_LEN = 8     /* a sequence length was negative or above max_len; unit skipped, n_out -1 */
};

typedef struct {
    void* ptr;
    int64_t stride_b, stride_h, stride_t; /* in elements; the head_dim axis has stride 1 */
} csp_tensor;

typedef struct {
    int32_t batch;        /* B  sequences                                                     */
    int32_t n_q_heads;    /* H_q, a multiple of n_kv_heads; group size G = H_q / H_kv <= 8     */
    int32_t n_kv_heads;   /* H_kv                                                             */
    int32_t head_dim;     /* d; row bytes d*sizeof(elem) must be 128, 256 or 512               */
    int32_t window;       /* W (the paper's O): 1..32 last queries are the observation window */
    int32_t recent;       /* R: last R keys are always kept and never scored                  */
    int32_t max_len;      /* padded key length of k, v, modality and the score vectors        */
    int32_t out_capacity; /* rows per head available in keep_idx, k_out, v_out, mod_out       */
    int32_t dtype;        /* csp_dtype: element type of q_win, k, v, k_out, v_out             */
    float n;              /* the n of n-softmax (Eq. 7); the paper uses 1; 0 gives softmax    */
    float scale;          /* logit scale; 0 means 1/sqrt(head_dim) (Eq. 5)                    */
    int32_t combine;      /* csp_combine                                                      */
    int32_t select_mode;  /* csp_select_mode                                                  */
    int32_t head_reduce;  /* csp_head_reduce; MEAN_ALL requires shared labels (mod_stride_h == 0) */
} csp_params;

/* Bytes of scratch that csp_score (MEAN_ALL) and csp_prune_layer need; also holds the status
 * word.  The first 256 bytes must be zero before first use (csp_workspace_reset). */
size_t csp_workspace_bytes(const csp_params* p);

/* Enqueue the zeroing of the workspace's status area. */
csp_status csp_workspace_reset(void* workspace, void* cuda_stream);

/*
 * Eq. 5, Eq. 7, the window/recent trim and Eq. 1.
 *   q_win      [B, H_q, W, d]      queries of the last W positions (position L_b-W+w), read-only
 *   k          [B, H_kv, max_len, d] cached keys; rows >= L_b are ignored
 *   modality   labels, uint8, element (b,h,t) at modality[b*mod_stride_b + h*mod_stride_h + t]
 *   seq_lens   [B] int32: L_b.  A sequence with L_b < W or L_b < R is skipped here (and passed
 *              through unchanged by csp_select)
 *   lse_or_null [B, H_q, W] fp32: natural log of sum_t exp(logit) over the keys each window row
 *              sees, if an upstream attention kernel has it; NULL makes the library compute it
 *   score_self, score_cross [B, H_kv, max_len] fp32 outputs; entries t >= L_b - R are not written
 * A query at position p sees keys t <= p.  The n-softmax denominator runs over ALL visible keys,
 * including the last R; only then are those columns dropped.
 */
csp_status csp_score(const csp_params* p, csp_tensor q_win, csp_tensor k,
                     const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                     const int32_t* seq_lens, const float* lse_or_null,
                     float* score_self, float* score_cross,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Eq. 2, Eq. 3 and the index list of Eq. 4.
 *   budgets    int32. SEGMENTED: [B,4] = k_self_text, k_self_visual, k_cross_text, k_cross_visual.
 *              GLOBAL: [B,2] = k_self, k_cross.  OVERALL: [B,1] = k.  Each is clamped to
 *              [0, candidates] (flagged).
 *   total_budget_or_null [B] int32 = T of Algorithm 1: a sequence with L_b < T keeps everything.
 *   keep_idx   [B, H_kv, out_capacity] int32: kept positions ascending, then L_b-R .. L_b-1
 *   n_out      [B, H_kv] int32: length of that list; -1 if it would exceed out_capacity (flagged,
 *              keep_idx of that unit untouched)
 * Order of a top-K: higher score first; among equal scores the lower position wins (-0 == +0).
 * Scores must not be NaN.
 */
csp_status csp_select(const csp_params* p, const float* score_self, const float* score_cross,
                      const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                      const int32_t* seq_lens, const int32_t* budgets,
                      const int32_t* total_budget_or_null,
                      int32_t* keep_idx, int32_t* n_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Eq. 4: k_out[b,h,j,:] = k[b,h,keep_idx[b,h,j],:] for j < n_out[b,h]; same for v and the labels.
 *   k_out, v_out [B, H_kv, out_capacity, d] (strided); mod_out [B, H_kv, out_capacity] dense, may
 *   be NULL.  Rows j >= n_out are left as they were; units with n_out <= 0 are skipped; an n_out above
 *   out_capacity copies the first out_capacity rows only (csp_prune_layer also raises CSP_DEV_CAPACITY;
 *   csp_compact has no status word).  Entries of keep_idx outside [0, max_len) copy nothing.
 * In place (the iteration of Algorithm 1 without a second cache buffer): k_out may be the very tensor k
 * and v_out the very tensor v (same pointer and strides, both or neither; CSP_ERR_UNSUPPORTED otherwise).
 * keep_idx is ascending with keep_idx[j] >= j, as csp_select writes it, so rows only move down; mod_out
 * stays a separate array.  Any other overlap between inputs and outputs is not detected and not allowed.
 */
csp_status csp_compact(const csp_params* p, csp_tensor k, csp_tensor v,
                       const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                       const int32_t* keep_idx, const int32_t* n_out,
                       csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, void* cuda_stream);

/*
 * csp_select followed by csp_compact on the same stream (Eq. 2-4), for a caller that already has the two score
 * vectors (from csp_score, or carried along by csp_decode_step).  Same arguments, results and flags as the two
 * calls; keep_idx may be NULL, in which case the list lives in the workspace.  With at least one unit per SM
 * and max_len in (1024, 4096] (up to 8192 with two units per SM and out_capacity >= max_len / 12), a second (not in-place) output buffer and contiguous output rows
 * (stride_t == head_dim), both steps run in one persistent kernel in which the selection of later units overlaps
 * the copy of earlier ones; otherwise as two kernels.  The results do not depend on which.
 */
csp_status csp_select_compact(const csp_params* p, const float* score_self, const float* score_cross,
                              csp_tensor k, csp_tensor v,
                              const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                              const int32_t* seq_lens, const int32_t* budgets,
                              const int32_t* total_budget_or_null,
                              csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                              int32_t* keep_idx_or_null,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 1, one invocation for one layer: csp_score, then csp_select_compact, on one stream.
 * score_self / score_cross / keep_idx may be NULL, in which case they live in the
 * workspace; n_out is required.
 */
csp_status csp_prune_layer(const csp_params* p, csp_tensor q_win, csp_tensor k, csp_tensor v,
                           const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                           const int32_t* seq_lens, const int32_t* budgets,
                           const int32_t* total_budget_or_null, const float* lse_or_null,
                           csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                           float* score_self_or_null, float* score_cross_or_null,
                           int32_t* keep_idx_or_null,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * A paged cache: K and V rows live in fixed-size pages of a pool instead of one dense run per sequence, and a
 * table says which page holds which stretch of a sequence (the layout serving engines use so that caches can grow
 * and shrink without copying).  Algorithm 1's loop prunes such a cache again and again; pruning it where it lies
 * frees whole pages at the end of every sequence.
 *   pool tensors  k_pool, v_pool [n_pages, H_kv, page_rows, d]: stride_b is the page stride
 *   page_table    [B, max_pages] int32 device: rows [i page_rows, (i+1) page_rows) of sequence b are page
 *                 page_table[b, i]; entries beyond a sequence's length are not read.  A page number outside
 *                 [0, n_pages) never faults: its rows score as zeros and are not copied, and the call is
 *                 flagged CSP_DEV_BAD_LEN.
 *   page_rows     a multiple of 128; max_pages * page_rows >= max_len
 * Labels, scores and keep_idx stay dense arrays over logical positions.
 */
typedef struct {
    const int32_t* page_table;
    int32_t max_pages, page_rows, n_pages;
} csp_pages;

/*
 * csp_prune_layer on a paged cache (Algorithm 1; Eq. 1-5, 7 unchanged, only the addressing differs).
 *   k_out, v_out  either dense [B, H_kv, out_capacity, d], or the pools themselves (same pointers and strides):
 *                 then the kept rows move down inside each sequence's own pages (logical row j goes to page
 *                 page_table[b, j / page_rows]), and pages past n_out rows can be returned to the pool.
 * bf16 caches, CSP_HEADS_PER_KV.  Everything else as for csp_prune_layer.
 */
csp_status csp_prune_layer_paged(const csp_params* p, csp_tensor q_win, csp_tensor k_pool, csp_tensor v_pool,
                                 const csp_pages* pages,
                                 const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                                 const int32_t* seq_lens, const int32_t* budgets,
                                 const int32_t* total_budget_or_null, const float* lse_or_null,
                                 csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                                 float* score_self_or_null, float* score_cross_or_null,
                                 int32_t* keep_idx_or_null,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of scratch that csp_decode_attn needs (status word + per-split partial results).  The first
 * 256 bytes must be zero before first use (csp_workspace_reset). */
size_t csp_decode_workspace_bytes(const csp_params* p);

/*
 * Section 3.3, Eq. 6-7: attention of ONE new query per head over a pruned cache, normalised with the
 * n-softmax, whose constant n stands for the exponential mass of the rows that pruning removed:
 *   out[b,hq,:] = sum_{t < n_rows[b,hkv]} e^{o_t} / (n + sum_j e^{o_j}) v[b,hkv,t,:],
 *   o_t = scale <q[b,hq,:], k[b,hkv,t,:]>,  hkv = hq / (H_q / H_kv).
 *   q       [B, H_q, d] (stride_b, stride_h; stride_t is not used), bf16
 *   k, v    [B, H_kv, out_capacity, d] bf16: the k_out / v_out of csp_prune_layer (or any cache of that
 *           layout); p->out_capacity is the row capacity, p->max_len / window / recent are not used
 *   n_rows  [B, H_kv] int32 device: valid rows per head (the n_out of the prune); values outside
 *           [0, out_capacity] are clamped and flagged CSP_DEV_BAD_LEN; 0 rows give a zero vector
 *   out     [B, H_q, d] fp32, dense
 * bf16 caches with head_dim 64 or 128 only (CSP_ERR_UNSUPPORTED otherwise).  Nothing is allocated; the
 * caller owns the workspace; the work is enqueued on the stream.
 */
csp_status csp_decode_attn(const csp_params* p, csp_tensor q, csp_tensor k, csp_tensor v,
                           const int32_t* n_rows, float* out,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The measurement behind the method (Section 1, the figure on the gap between self- and cross-attention): the
 * window's attention weights, per query head and not averaged, collected in two histograms, one for pairs whose
 * query and key carry the same modality label (intra) and one for the others (inter), and the Jensen-Shannon
 * divergence between the two.  Which weights: A[g,w,t] of Eq. 7 for window row w and every candidate key
 * t < L_b - R that the row sees, i.e. exactly the entries that Eq. 1 sums.  Bin j of CSP_HIST_BINS covers
 * log2(A) in [CSP_HIST_LO + j CSP_HIST_WIDTH, CSP_HIST_LO + (j + 1) CSP_HIST_WIDTH); smaller weights (and zeros)
 * count in bin 0.  The paper shows a kernel density estimate; the half-octave bins are this library's choice.
 *   hist   [B, H_kv, 2, CSP_HIST_BINS] uint32 (0: intra, 1: inter); cleared and filled by the call
 *   js_or_null     [B, H_kv] fp32: 1/2 KL(P || M) + 1/2 KL(Q || M) in nats, M = (P + Q) / 2, P and Q the two
 *                  histograms of the unit normalised to sum 1; NaN when either is empty
 *   js_all_or_null [1] fp32: the same for the histograms summed over all units of the call (one layer's figure
 *                  when the call is one layer)
 * Other arguments as for csp_score; workspace of csp_workspace_bytes (it also receives the scores).  bf16 caches,
 * CSP_HEADS_PER_KV only.  A diagnostic, several times slower than csp_score: every weight is binned.
 */
#define CSP_HIST_BINS 64
#define CSP_HIST_LO (-32.0f)
#define CSP_HIST_WIDTH 0.5f
csp_status csp_weight_histogram(const csp_params* p, csp_tensor q_win, csp_tensor k,
                                const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                                const int32_t* seq_lens, const float* lse_or_null,
                                uint32_t* hist, float* js_or_null, float* js_all_or_null,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * csp_decode_attn over a paged cache (Section 3.3, Eq. 6-7; only the addressing differs): k_pool, v_pool and pages as
 * for csp_prune_layer_paged, e.g. the pools a prune in place has just compacted.  p->out_capacity is the logical row
 * capacity per head (at most max_pages * page_rows); n_rows [B, H_kv] counts logical rows.  A page number outside
 * the pool is flagged CSP_DEV_BAD_LEN; its rows read as zeros.  Workspace: csp_decode_workspace_bytes.
 */
csp_status csp_decode_attn_paged(const csp_params* p, csp_tensor q, csp_tensor k_pool, csp_tensor v_pool,
                                 const csp_pages* pages, const int32_t* n_rows, float* out,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of scratch that csp_decode_step needs: those of csp_decode_attn plus one row of logits per query head
 * and unit.  The first 256 bytes must be zero before first use (csp_workspace_reset). */
size_t csp_decode_step_workspace_bytes(const csp_params* p);

/*
 * Algorithm 1's iteration loop, one appended token: csp_decode_attn for the new token's query, and the scores
 * of Eq. 1 carried along, so that the next prune needs no pass over the cache of its own.  The query of the
 * token at position pos sees exactly the n_rows = pos + 1 rows the cache holds at that step, its own included, so
 * its n-softmax weights (Eq. 7) are row pos of the attention matrix and are final.  They are averaged over the
 * query heads of the KV group and added to the intra sum of the rows that carry the query's label and to the
 * inter sum of the others (Eq. 1).  After the last W steps before a prune, started with first_step != 0, the two
 * arrays hold what csp_score would compute on that cache with those W queries as the observation window;
 * csp_select and csp_compact then finish the prune (Eq. 2-4).
 *   q, k, v, n_rows, out   as for csp_decode_attn; the new token's K and V rows are already in the cache
 *   modality     labels of the cached rows, element (b,h,t) at modality[b*mod_stride_b + h*mod_stride_h + t]
 *   query_label  [B] uint8: label of each sequence's new token
 *   first_step   != 0 starts a new window: all out_capacity slots of every unit are overwritten (rows that are
 *                appended later in the window start from zero); 0 adds to the slots t < n_rows
 *   acc_self, acc_cross  [B, H_kv, out_capacity] fp32, the layout of csp_select's score vectors with
 *                max_len = out_capacity
 * bf16 caches with head_dim 64 or 128.  Nothing is allocated; the caller owns the workspace.
 */
csp_status csp_decode_step(const csp_params* p, csp_tensor q, csp_tensor k, csp_tensor v, const int32_t* n_rows,
                           const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                           const uint8_t* query_label, int32_t first_step, float* out, float* acc_self,
                           float* acc_cross, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Bytes of device staging that csp_prune_layer_host needs for these parameters. */
size_t csp_host_staging_bytes(const csp_params* p);

/*
 * Algorithm 1 for a caller whose cache lives in HOST memory (pinned memory makes the copies
 * asynchronous): copies the dense inputs into `staging` (device, caller-owned,
 * >= csp_host_staging_bytes), runs csp_prune_layer there, copies k_out, v_out, mod_out, n_out
 * back and waits for the stream.  All *_host tensors are dense: q [B,H_q,W,d],
 * k, v [B,H_kv,max_len,d], modality [B,max_len] (mod_per_head == 0) or [B,H_kv,max_len],
 * outputs [B,H_kv,out_capacity,(d)].  dev_status_host (may be NULL) receives the status word.
 * Only the kept rows of V are needed (Eq. 4): when v_host is page-locked memory the device can address, they are
 * read from it directly by the compaction kernel and V is never copied as a whole; otherwise V is staged in full.
 */
csp_status csp_prune_layer_host(const csp_params* p, const void* q_host, const void* k_host,
                                const void* v_host, const uint8_t* modality_host, int mod_per_head,
                                const int32_t* seq_lens_host, const int32_t* budgets_host,
                                const int32_t* total_budget_host_or_null,
                                void* k_out_host, void* v_out_host, uint8_t* mod_out_host,
                                int32_t* n_out_host, int32_t* dev_status_host,
                                void* staging, size_t staging_bytes, void* cuda_stream);

/*
 * No counterpart in the paper: a convenience of this library.  Algorithm 1 exactly as
 * csp_prune_layer computes it, for callers that have no way to obtain scratch memory: code that runs
 * after a serving engine has claimed all device memory for its own pool, plug-ins that are handed
 * tensors but no allocator, or latency-critical loops where a cudaMalloc (which stalls the device)
 * is not acceptable.  The scratch (status word, score vectors, index list) is a fixed array inside
 * the library, csp_static_workspace_limit() bytes (8 MiB) on every GPU that loads it, held until
 * the process exits.  The call allocates and frees nothing.
 *   - Shapes whose csp_workspace_bytes exceeds the limit are refused with CSP_ERR_WORKSPACE and
 *     nothing is enqueued (8 MiB covers e.g. 32 KV heads x 4096 positions; use csp_prune_layer with
 *     your own workspace beyond that).
 *   - Arguments are checked as in csp_prune_layer before anything else happens; a call that returns an
 *     error has enqueued nothing.
 *   - The first call on a device looks up the array's device address; make that first call
 *     outside any stream capture.  The address is kept for the life of the process (a cudaDeviceReset
 *     in between is not supported).
 *   - All calls share the one array, which still holds the previous call's contents; the status
 *     area is cleared on the stream at the start of every call.  Two calls whose GPU work can
 *     overlap (different streams, several host threads) race on it: serialise them.
 *   - dev_status_out_or_null: DEVICE pointer to one int32 that receives the CSP_DEV_* status word
 *     of this call (copied on the stream); per-unit failures also show as n_out == -1.
 * Inputs, outputs and all other rules are those of csp_prune_layer.
 */
csp_status csp_prune_layer_static(const csp_params* p, csp_tensor q_win, csp_tensor k, csp_tensor v,
                                  const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                                  const int32_t* seq_lens, const int32_t* budgets,
                                  const int32_t* total_budget_or_null, const float* lse_or_null,
                                  csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                                  int32_t* dev_status_out_or_null, void* cuda_stream);

/* Size in bytes of the built-in scratch array used by csp_prune_layer_static. */
size_t csp_static_workspace_limit(void);

/*
 * No counterpart in the paper: a measuring aid.  With G >= 3 query heads per KV head the scoring kernel (Eq. 5,
 * Eq. 7) is bound by exponentials, not by memory, so its roofline needs this GPU's exponential rate.  Enqueues a
 * registers-only kernel (two CTAs of 1024 threads per SM, eight independent chains per thread) that evaluates
 * *exponentials_host_out base-2 exponentials in total; the caller times it with events on the stream.
 *   fma_pipe    0: ex2.approx.ftz.f32 on the special-function unit (what the scoring kernels issue);
 *               1: the two-wide FMA-pipe evaluation the G >= 3 kernels use for one pair in eight;
 *               2: ex2.approx.f16x2, two half-precision exponentials per instruction (measured for comparison; no
 *                  kernel uses it: a half-precision argument is too coarse for the row sums)
 *   iterations  1 .. 2^20 loop trips (8 exponentials per thread and trip; 16 in mode 2)
 *   sink        device array that receives one float per thread (keeps the loop alive); may be NULL
 */
csp_status csp_probe_ex2_rate(int32_t fma_pipe, int32_t iterations, float* sink, size_t sink_elems,
                              int64_t* exponentials_host_out, void* cuda_stream);

/* Waits for the stream, copies the status word to *host_out (may be NULL), clears it, and returns
 * CSP_ERR_TIMEOUT if CSP_DEV_TIMEOUT was set, else CSP_OK. */
csp_status csp_device_status(void* workspace, void* cuda_stream, int32_t* host_out);

const char* csp_status_string(csp_status s);

#ifdef __cplusplus
}
#endif
#endif

/*
 * CPU oracle for the Cross-Self Pruning (CSP) scoring-and-compaction pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, double-precision
 * restatement of what the paper defines (Eq. 1-4, Eq. 5, Eq. 7, Algorithm 1).
 * It also holds the plain definition of decode attention with the n-softmax
 * normaliser (Section 3.3) and of a decode step that carries the scores of Eq. 1 along
 * (Algorithm 1's iteration loop).  It exists to check the CUDA library and to be timed as a CPU baseline.  It
 * shares no code with the CUDA library and must never be called from it.
 *
 * Every function has at least one independent pin in the CPU test-suite
 * (closed forms, library softmax on a padded row, full-matrix brute force,
 * numpy stable sort); none is "parity unpinned".
 *
 * All tensors are dense and contiguous:
 *   q        [B, Hq,  W,       d]   element type given by orc_params.dtype
 *   k, v     [B, Hkv, max_len, d]
 *   modality [B, max_len]           when mod_per_head == 0
 *            [B, Hkv, max_len]      when mod_per_head != 0
 *   seq_lens [B]
 * bf16 elements are passed as their 16 raw bits and widened exactly to double.
 */
#ifndef CSP_ORACLE_H
#define CSP_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_COMBINE_OR = 0, ORC_COMBINE_AND = 1 };
enum { ORC_SELECT_SEGMENTED = 0, ORC_SELECT_GLOBAL = 1, ORC_SELECT_OVERALL = 2 };
enum { ORC_HEADS_PER_KV = 0, ORC_HEADS_MEAN_ALL = 1 };

/* per-unit flag bits written by orc_select / orc_prune_layer */
enum { ORC_FLAG_K_CLAMPED = 1, ORC_FLAG_CAPACITY = 2, ORC_FLAG_IDENTITY = 4 };

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim;
    int32_t window, recent, max_len, out_capacity;
    int32_t dtype;
    int32_t combine, select_mode, head_reduce;
    double n;      /* the n of n-softmax (Eq. 7); the paper uses 1 */
    double scale;  /* <= 0 means 1/sqrt(head_dim) (Eq. 5) */
} orc_params;

/* Eq. 7: a[i] = exp(o[i]) / (n + sum_j exp(o[j])), j over the `len` kept logits. */
void orc_nsoftmax(const double* o, int64_t len, double n, double* a);

/* Eq. 5 + Eq. 7 + window/recent trim + Eq. 1 for every (b, kv head).
 * score_self/score_cross: [B, Hkv, max_len] doubles; entries t >= L_b - R are set to 0.
 * row_mass (optional, may be NULL): [B, Hq, W] = sum over ALL visible keys of A (incl. recent).
 * lse (optional, may be NULL): [B, Hq, W] natural-log of sum_t exp(o) supplied by the caller,
 * used in place of the oracle's own row sum.  Returns 0, or -1 on a bad argument. */
int orc_score(const orc_params* p, const void* q, const void* k,
              const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
              const double* lse, double* score_self, double* score_cross, double* row_mass);

/* Eq. 2 on one score vector: mark the k best candidates (cand[t] != 0, t < n_keys).
 * Order: higher score first, lower index first among equal scores.  k is clamped to the
 * candidate count.  mask[t] is set to 1 for winners and left untouched otherwise.
 * kth / knext receive the k-th and (k+1)-th best scores (NaN where absent).
 * Returns the number selected. */
int orc_topk(const float* score, const uint8_t* cand, int64_t n_keys, int64_t k,
             uint8_t* mask, float* kth, float* knext);

/* Eq. 2 + Eq. 3 + the index list of Eq. 4 for every (b, kv head), from fp32 scores.
 * budgets: SEGMENTED [B,4] = k_self_text, k_self_visual, k_cross_text, k_cross_visual
 *          GLOBAL    [B,2] = k_self, k_cross
 * total_budget (optional): [B] = T of Algorithm 1 (L_b < T keeps everything).
 * keep_idx [B,Hkv,out_capacity] ascending kept positions followed by the last R positions;
 * n_out [B,Hkv] (-1 when the list would not fit out_capacity); flags [B,Hkv];
 * margins (optional) [B,Hkv,4,2] = k-th and (k+1)-th score of each top-k problem
 * (problem order as in `budgets`; GLOBAL uses the first two). */
int orc_select(const orc_params* p, const float* score_self, const float* score_cross,
               const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
               const int32_t* budgets, const int32_t* total_budget,
               int32_t* keep_idx, int32_t* n_out, int32_t* flags, float* margins);

/* Eq. 4: row gather of K, V and the modality labels by keep_idx. */
int orc_compact(const orc_params* p, const void* k, const void* v,
                const uint8_t* modality, int mod_per_head,
                const int32_t* keep_idx, const int32_t* n_out,
                void* k_out, void* v_out, uint8_t* mod_out);

/* Algorithm 1, one invocation: score (rounded to fp32) -> select -> compact. */
int orc_prune_layer(const orc_params* p, const void* q, const void* k, const void* v,
                    const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
                    const int32_t* budgets, const int32_t* total_budget, const double* lse,
                    float* score_self, float* score_cross,
                    int32_t* keep_idx, int32_t* n_out, int32_t* flags, float* margins,
                    void* k_out, void* v_out, uint8_t* mod_out);

/* Attention of one new query per head over a pruned cache, with the n-softmax of Eq. 7 as the
 * normaliser (Section 3.3: the denominator keeps the constant n for the mass that pruning removed):
 *   o_t = scale <q[b,hq,:], k[b,hkv,t,:]>,  t < n_rows[b,hkv]   (hkv = hq / (Hq / Hkv))
 *   out[b,hq,:] = sum_t  e^{o_t} / (n + sum_j e^{o_j})  v[b,hkv,t,:]
 * q: [B, Hq, d]; k, v: [B, Hkv, out_capacity, d]; n_rows: [B, Hkv] (rows beyond it are ignored);
 * out: [B, Hq, d] doubles.  A head with no rows gives a zero vector.  Returns 0, or -1 on a bad
 * argument (n_rows outside [0, out_capacity]). */
int orc_decode_attn(const orc_params* p, const void* q, const void* k, const void* v,
                    const int32_t* n_rows, double* out);

/* One decode step of Algorithm 1's iteration loop: orc_decode_attn for the new token's query, and the same
 * n-softmax weights added to running intra / inter score vectors.  The query of the token at position p sees
 * exactly the rows the cache holds at that step (rows 0..p, its own included), so its weights are row p of the
 * attention matrix and never change afterwards: summed over the last W steps they are the scores of Eq. 1 for
 * the window made of those W queries, without another pass over the cache.
 *   a_g[t]       = e^{o_{g,t}} / (n + sum_j e^{o_{g,j}})            (Eq. 7, query head g of the KV group)
 *   acc_self[t] += (1/G) sum_g a_g[t]   if modality[b,hkv,t] == query_label[b]   (intra, Eq. 1)
 *   acc_cross[t]+= (1/G) sum_g a_g[t]   otherwise                                 (inter, Eq. 1)
 * modality: [B, Hkv, out_capacity] labels of the cached rows (per head: after a prune heads differ);
 * query_label: [B]; acc_self, acc_cross: [B, Hkv, out_capacity] doubles; a step adds to t < n_rows[b,hkv];
 * first != 0 starts a new window: all out_capacity slots of a unit are cleared first (rows appended later
 * in the window then start from zero).  Returns 0 or -1. */
int orc_decode_step(const orc_params* p, const void* q, const void* k, const void* v, const int32_t* n_rows,
                    const uint8_t* modality, const uint8_t* query_label, int first,
                    double* out, double* acc_self, double* acc_cross);

/* Diagnostic behind the method's motivation (Section 1, the figure on the distribution gap): the attention
 * weights of the observation window, per query head and not averaged, split into intra-modality pairs (query
 * and key carry the same label) and inter-modality pairs, each collected in a histogram of log2(weight), and the
 * Jensen-Shannon divergence between the two normalised histograms.
 *   weights: A[g,w,t] of Eq. 7 for window row w (position L-W+w), candidate keys t < L-R with t <= L-W+w
 *   bin j of ORC_HIST_BINS covers log2(A) in [ORC_HIST_LO + j ORC_HIST_WIDTH, ORC_HIST_LO + (j+1) ORC_HIST_WIDTH);
 *   values below the first bin (and exact zeros) go to bin 0, values above the last to the last
 *   hist [B,Hkv,2,ORC_HIST_BINS] int64 counts (0: intra, 1: inter)
 *   near (optional) [B,Hkv,2,ORC_HIST_BINS]: how many weights lie within near_eps (in log2 units) of the lower
 *        edge of bin j, i.e. could fall on either side of it in another precision
 *   js   (optional) [B,Hkv]: orc_js_divergence of the unit's two histograms
 *   js_all (optional) [1]: the same for the histograms summed over all units of the call
 * The paper plots a kernel density estimate; the binning (half-octave bins from 2^-32 to 1) is this
 * library's choice and is stated wherever the result is reported. */
enum { ORC_HIST_BINS = 64 };
#define ORC_HIST_LO (-32.0)
#define ORC_HIST_WIDTH 0.5
int orc_weight_histogram(const orc_params* p, const void* q, const void* k,
                         const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
                         int64_t* hist, int64_t* near, double near_eps, double* js, double* js_all);

/* Jensen-Shannon divergence, in nats, between two histograms normalised to sum 1:
 * 1/2 KL(P || M) + 1/2 KL(Q || M), M = (P + Q) / 2, 0 log 0 = 0.  NaN if either histogram is empty. */
double orc_js_divergence(const int64_t* hist_p, const int64_t* hist_q, int bins);

/* number of OpenMP threads the unit loops will use */
int orc_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif

/*
 * CPU oracle for the CSP scoring-and-compaction pass -- TEST INFRASTRUCTURE ONLY.
 * See csp_oracle.h for the contract.  Double precision, plain loops, no blocking,
 * no fusion: each function follows the paper's own order of steps so that it can be
 * checked against the equations by eye.  OpenMP is used only across independent
 * (sequence, KV head) units.
 */
#include "csp_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* exact widening of one stored element to double */
static double load_elem(const void* base, int64_t i, int dtype) {
    if (dtype == ORC_F32) return (double)((const float*)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16; /* bf16 = top half of fp32 */
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

static int64_t elem_size(int dtype) { return dtype == ORC_F32 ? 4 : 2; }

/* Eq. 7.  e^{o_i} / (n + sum_j e^{o_j}) evaluated with every exponent shifted by the
 * row maximum m (numerator and denominator both multiplied by e^{-m}). */
void orc_nsoftmax(const double* o, int64_t len, double n, double* a) {
    if (len <= 0) return;
    double m = o[0];
    for (int64_t i = 1; i < len; ++i)
        if (o[i] > m) m = o[i];
    double z = 0.0;
    for (int64_t i = 0; i < len; ++i) z += exp(o[i] - m);
    double denom = n * exp(-m) + z;
    for (int64_t i = 0; i < len; ++i) a[i] = exp(o[i] - m) / denom;
}

static const uint8_t* mod_row(const orc_params* p, const uint8_t* modality, int mod_per_head,
                              int b, int h) {
    if (mod_per_head) return modality + ((int64_t)b * p->n_kv_heads + h) * p->max_len;
    return modality + (int64_t)b * p->max_len;
}

static int unit_is_short(const orc_params* p, int64_t L) {
    return L < p->window || L < p->recent;
}

/* Attention weights of one query head over the observation window (Eq. 5 then Eq. 7),
 * accumulated with weight `wgt` into abar[w][t] for the trimmed keys t < N.  */
static void window_rows(const orc_params* p, const void* q, const void* k, int b, int hq, int hkv,
                        int64_t L, const double* lse, double wgt, double* o, double* a,
                        double* abar, double* row_mass) {
    const int d = p->head_dim, W = p->window;
    const int64_t N = L - p->recent;
    const double scale = p->scale > 0.0 ? p->scale : 1.0 / sqrt((double)d);
    const int64_t qbase = (((int64_t)b * p->n_q_heads + hq) * W) * d;
    const int64_t kbase = (((int64_t)b * p->n_kv_heads + hkv) * p->max_len) * d;
    for (int w = 0; w < W; ++w) {
        const int64_t pos = L - W + w; /* position of this query; it sees keys 0..pos */
        for (int64_t t = 0; t <= pos; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += load_elem(q, qbase + (int64_t)w * d + c, p->dtype) *
                       load_elem(k, kbase + t * d + c, p->dtype);
            o[t] = acc * scale; /* Eq. 5 */
        }
        if (lse) {
            /* caller-supplied log of sum_t e^{o_t}: A = e^{o} / (n + e^{lse}) */
            const double l = lse[((int64_t)b * p->n_q_heads + hq) * W + w];
            const double denom = p->n * exp(-l) + 1.0;
            for (int64_t t = 0; t <= pos; ++t) a[t] = exp(o[t] - l) / denom;
        } else {
            orc_nsoftmax(o, pos + 1, p->n, a); /* Eq. 7 over every key in the cache */
        }
        double mass = 0.0;
        for (int64_t t = 0; t <= pos; ++t) mass += a[t];
        if (row_mass) row_mass[((int64_t)b * p->n_q_heads + hq) * W + w] = mass;
        for (int64_t t = 0; t < N && t <= pos; ++t) abar[(int64_t)w * p->max_len + t] += wgt * a[t];
    }
}

/* Eq. 1: per key, add up the window rows whose query has the same label (intra) and the
 * rows whose query has a different label (inter). */
static void split_sums(const orc_params* p, const uint8_t* mod, int64_t L, const double* abar,
                       double* s, double* c) {
    const int W = p->window;
    const int64_t N = L - p->recent;
    for (int64_t t = 0; t < p->max_len; ++t) { s[t] = 0.0; c[t] = 0.0; }
    for (int64_t t = 0; t < N; ++t) {
        for (int w = 0; w < W; ++w) {
            const int64_t pos = L - W + w;
            if (t > pos) continue;
            const double x = abar[(int64_t)w * p->max_len + t];
            if (mod[pos] == mod[t]) s[t] += x; else c[t] += x;
        }
    }
}

int orc_score(const orc_params* p, const void* q, const void* k,
              const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
              const double* lse, double* score_self, double* score_cross, double* row_mass) {
    if (!p || !q || !k || !modality || !seq_lens || !score_self || !score_cross) return -1;
    if (p->n_kv_heads <= 0 || p->n_q_heads % p->n_kv_heads) return -1;
    if (p->head_reduce == ORC_HEADS_MEAN_ALL && mod_per_head) return -1;
    const int G = p->n_q_heads / p->n_kv_heads;
    const int units = p->batch * p->n_kv_heads;
    int bad = 0;

    if (p->head_reduce == ORC_HEADS_PER_KV) {
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
        for (int u = 0; u < units; ++u) {
            const int b = u / p->n_kv_heads, h = u % p->n_kv_heads;
            const int64_t L = seq_lens[b];
            double* s = score_self + (int64_t)u * p->max_len;
            double* c = score_cross + (int64_t)u * p->max_len;
            for (int64_t t = 0; t < p->max_len; ++t) { s[t] = 0.0; c[t] = 0.0; }
            if (L > p->max_len) { bad = 1; continue; }
            if (unit_is_short(p, L)) continue;
            double* o = (double*)malloc(sizeof(double) * (size_t)p->max_len);
            double* a = (double*)malloc(sizeof(double) * (size_t)p->max_len);
            double* abar = (double*)calloc((size_t)p->window * (size_t)p->max_len, sizeof(double));
            for (int g = 0; g < G; ++g) /* mean over the query heads of this KV group */
                window_rows(p, q, k, b, h * G + g, h, L, lse, 1.0 / G, o, a, abar, row_mass);
            split_sums(p, mod_row(p, modality, mod_per_head, b, h), L, abar, s, c);
            free(o); free(a); free(abar);
        }
    } else {
        /* the paper's sentence: one attention matrix averaged over every head */
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
        for (int b = 0; b < p->batch; ++b) {
            const int64_t L = seq_lens[b];
            for (int h = 0; h < p->n_kv_heads; ++h) {
                double* s = score_self + ((int64_t)b * p->n_kv_heads + h) * p->max_len;
                double* c = score_cross + ((int64_t)b * p->n_kv_heads + h) * p->max_len;
                for (int64_t t = 0; t < p->max_len; ++t) { s[t] = 0.0; c[t] = 0.0; }
            }
            if (L > p->max_len) { bad = 1; continue; }
            if (unit_is_short(p, L)) continue;
            double* o = (double*)malloc(sizeof(double) * (size_t)p->max_len);
            double* a = (double*)malloc(sizeof(double) * (size_t)p->max_len);
            double* abar = (double*)calloc((size_t)p->window * (size_t)p->max_len, sizeof(double));
            for (int hq = 0; hq < p->n_q_heads; ++hq)
                window_rows(p, q, k, b, hq, hq / G, L, lse, 1.0 / p->n_q_heads, o, a, abar, row_mass);
            double* s0 = score_self + ((int64_t)b * p->n_kv_heads) * p->max_len;
            double* c0 = score_cross + ((int64_t)b * p->n_kv_heads) * p->max_len;
            split_sums(p, mod_row(p, modality, 0, b, 0), L, abar, s0, c0);
            for (int h = 1; h < p->n_kv_heads; ++h) {
                memcpy(s0 + (int64_t)h * p->max_len, s0, sizeof(double) * (size_t)p->max_len);
                memcpy(c0 + (int64_t)h * p->max_len, c0, sizeof(double) * (size_t)p->max_len);
            }
            free(o); free(a); free(abar);
        }
    }
    return bad ? -1 : 0;
}

/* ---- Eq. 2: top-K by a full sort ---------------------------------------------------- */

typedef struct { float score; int64_t index; } ranked;

static int ranked_before(const void* pa, const void* pb) {
    const ranked* a = (const ranked*)pa;
    const ranked* b = (const ranked*)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    if (a->index < b->index) return -1;
    if (a->index > b->index) return 1;
    return 0;
}

int orc_topk(const float* score, const uint8_t* cand, int64_t n_keys, int64_t k,
             uint8_t* mask, float* kth, float* knext) {
    int64_t n_cand = 0;
    for (int64_t t = 0; t < n_keys; ++t) n_cand += cand[t] != 0;
    ranked* r = (ranked*)malloc(sizeof(ranked) * (size_t)(n_cand > 0 ? n_cand : 1));
    int64_t j = 0;
    for (int64_t t = 0; t < n_keys; ++t)
        if (cand[t]) { r[j].score = score[t]; r[j].index = t; ++j; }
    qsort(r, (size_t)n_cand, sizeof(ranked), ranked_before); /* total order: unique result */
    if (k < 0) k = 0;
    if (k > n_cand) k = n_cand;
    for (int64_t i = 0; i < k; ++i) mask[r[i].index] = 1;
    if (kth) *kth = k >= 1 ? r[k - 1].score : NAN;
    if (knext) *knext = k < n_cand ? r[k].score : NAN;
    free(r);
    return (int)k;
}

int orc_select(const orc_params* p, const float* score_self, const float* score_cross,
               const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
               const int32_t* budgets, const int32_t* total_budget,
               int32_t* keep_idx, int32_t* n_out, int32_t* flags, float* margins) {
    if (!p || !score_self || !score_cross || !modality || !seq_lens || !budgets || !keep_idx || !n_out)
        return -1;
    const int units = p->batch * p->n_kv_heads;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
    for (int u = 0; u < units; ++u) {
        const int b = u / p->n_kv_heads, h = u % p->n_kv_heads;
        const int64_t L = seq_lens[b];
        const float* s = score_self + (int64_t)u * p->max_len;
        const float* c = score_cross + (int64_t)u * p->max_len;
        const uint8_t* mod = mod_row(p, modality, mod_per_head, b, h);
        int32_t* idx = keep_idx + (int64_t)u * p->out_capacity;
        int32_t fl = 0;
        if (margins) for (int i = 0; i < 8; ++i) margins[(int64_t)u * 8 + i] = NAN;
        if (L > p->max_len || L < 0) { bad = 1; n_out[u] = -1; if (flags) flags[u] = 0; continue; }

        /* Algorithm 1: a cache shorter than the budget T is returned unchanged; so is one
         * too short to hold an observation window or a recent block. */
        if (unit_is_short(p, L) || (total_budget && L < total_budget[b])) {
            fl |= ORC_FLAG_IDENTITY;
            if (L > p->out_capacity) { fl |= ORC_FLAG_CAPACITY; n_out[u] = -1; }
            else { for (int64_t t = 0; t < L; ++t) idx[t] = (int32_t)t; n_out[u] = (int32_t)L; }
            if (flags) flags[u] = fl;
            continue;
        }

        const int64_t N = L - p->recent; /* candidates are the keys before the recent block */
        uint8_t* cand = (uint8_t*)calloc((size_t)(N > 0 ? N : 1), 1);
        uint8_t* ms = (uint8_t*)calloc((size_t)(N > 0 ? N : 1), 1);
        uint8_t* mc = (uint8_t*)calloc((size_t)(N > 0 ? N : 1), 1);
        float* mg = margins ? margins + (int64_t)u * 8 : NULL;

        if (p->select_mode == ORC_SELECT_SEGMENTED) {
            const int32_t* kb = budgets + (int64_t)b * 4;
            for (int prob = 0; prob < 4; ++prob) {
                const int visual = prob & 1;       /* 0: text keys (label 0), 1: visual keys */
                const int cross = prob >> 1;       /* 0: intra score, 1: inter score */
                int64_t n_cand = 0;
                for (int64_t t = 0; t < N; ++t) { cand[t] = ((mod[t] != 0) == visual); n_cand += cand[t]; }
                if (kb[prob] > n_cand || kb[prob] < 0) fl |= ORC_FLAG_K_CLAMPED;
                orc_topk(cross ? c : s, cand, N, kb[prob], cross ? mc : ms,
                         mg ? mg + prob * 2 : NULL, mg ? mg + prob * 2 + 1 : NULL);
            }
        } else if (p->select_mode == ORC_SELECT_OVERALL) {
            /* the ablation's comparison arm ("Influence of n-softmax"): one top-k straight on the overall
             * selection function, i.e. on the column sums of A over the whole window = s + c (Eq. 1 without
             * the split); budgets [B, 1].  The sum is taken in fp32, the precision the scores are carried in. */
            const int32_t kb = budgets[b];
            float* mix = (float*)malloc(sizeof(float) * (size_t)(N > 0 ? N : 1));
            for (int64_t t = 0; t < N; ++t) { cand[t] = 1; mix[t] = s[t] + c[t]; }
            if (kb > N || kb < 0) fl |= ORC_FLAG_K_CLAMPED;
            orc_topk(mix, cand, N, kb, ms, mg ? mg : NULL, mg ? mg + 1 : NULL);
            memcpy(mc, ms, (size_t)(N > 0 ? N : 1));
            free(mix);
        } else {
            const int32_t* kb = budgets + (int64_t)b * 2;
            for (int64_t t = 0; t < N; ++t) cand[t] = 1;
            for (int prob = 0; prob < 2; ++prob) {
                if (kb[prob] > N || kb[prob] < 0) fl |= ORC_FLAG_K_CLAMPED;
                orc_topk(prob ? c : s, cand, N, kb[prob], prob ? mc : ms,
                         mg ? mg + prob * 2 : NULL, mg ? mg + prob * 2 + 1 : NULL);
            }
        }

        /* Eq. 3 (printed: AND; the prose describes OR) then the index list of Eq. 4 */
        int64_t n_keep = 0;
        for (int64_t t = 0; t < N; ++t) {
            const int m = p->combine == ORC_COMBINE_AND ? (ms[t] && mc[t]) : (ms[t] || mc[t]);
            n_keep += m;
        }
        if (n_keep + p->recent > p->out_capacity) {
            fl |= ORC_FLAG_CAPACITY;
            n_out[u] = -1;
        } else {
            int64_t j = 0;
            for (int64_t t = 0; t < N; ++t) {
                const int m = p->combine == ORC_COMBINE_AND ? (ms[t] && mc[t]) : (ms[t] || mc[t]);
                if (m) idx[j++] = (int32_t)t;
            }
            for (int64_t t = N; t < L; ++t) idx[j++] = (int32_t)t; /* (+) K[-R:] */
            n_out[u] = (int32_t)j;
        }
        if (flags) flags[u] = fl;
        free(cand); free(ms); free(mc);
    }
    return bad ? -1 : 0;
}

int orc_compact(const orc_params* p, const void* k, const void* v,
                const uint8_t* modality, int mod_per_head,
                const int32_t* keep_idx, const int32_t* n_out,
                void* k_out, void* v_out, uint8_t* mod_out) {
    if (!p || !k || !v || !keep_idx || !n_out || !k_out || !v_out) return -1;
    const int units = p->batch * p->n_kv_heads;
    const int64_t row = (int64_t)p->head_dim * elem_size(p->dtype);
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
    for (int u = 0; u < units; ++u) {
        const int b = u / p->n_kv_heads, h = u % p->n_kv_heads;
        const char* ku = (const char*)k + (int64_t)u * p->max_len * row;
        const char* vu = (const char*)v + (int64_t)u * p->max_len * row;
        char* ko = (char*)k_out + (int64_t)u * p->out_capacity * row;
        char* vo = (char*)v_out + (int64_t)u * p->out_capacity * row;
        const int32_t* idx = keep_idx + (int64_t)u * p->out_capacity;
        for (int64_t j = 0; j < n_out[u]; ++j) {
            const int64_t t = idx[j];
            if (t < 0 || t >= p->max_len) { bad = 1; continue; }
            memcpy(ko + j * row, ku + t * row, (size_t)row);
            memcpy(vo + j * row, vu + t * row, (size_t)row);
            if (mod_out && modality)
                mod_out[(int64_t)u * p->out_capacity + j] = mod_row(p, modality, mod_per_head, b, h)[t];
        }
    }
    return bad ? -1 : 0;
}

int orc_prune_layer(const orc_params* p, const void* q, const void* k, const void* v,
                    const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
                    const int32_t* budgets, const int32_t* total_budget, const double* lse,
                    float* score_self, float* score_cross,
                    int32_t* keep_idx, int32_t* n_out, int32_t* flags, float* margins,
                    void* k_out, void* v_out, uint8_t* mod_out) {
    const int64_t n = (int64_t)p->batch * p->n_kv_heads * p->max_len;
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    double* c = (double*)malloc(sizeof(double) * (size_t)n);
    int rc = orc_score(p, q, k, modality, mod_per_head, seq_lens, lse, s, c, NULL);
    /* the selection is decided on fp32 scores, the precision the library's interface carries */
    for (int64_t i = 0; i < n; ++i) { score_self[i] = (float)s[i]; score_cross[i] = (float)c[i]; }
    free(s); free(c);
    if (rc) return rc;
    rc = orc_select(p, score_self, score_cross, modality, mod_per_head, seq_lens, budgets,
                    total_budget, keep_idx, n_out, flags, margins);
    if (rc) return rc;
    return orc_compact(p, k, v, modality, mod_per_head, keep_idx, n_out, k_out, v_out, mod_out);
}

/* Section 3.3 / Eq. 7 applied to one decode query per head: logits over the rows of the pruned cache,
 * n-softmax weights (orc_nsoftmax), weighted sum of the value rows. */
int orc_decode_attn(const orc_params* p, const void* q, const void* k, const void* v,
                    const int32_t* n_rows, double* out) {
    const int64_t d = p->head_dim, cap = p->out_capacity;
    const int G = p->n_q_heads / p->n_kv_heads;
    const double scale = p->scale > 0.0 ? p->scale : 1.0 / sqrt((double)d);
    int bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic) reduction(|:bad)
    for (int b = 0; b < p->batch; ++b) {
        for (int hq = 0; hq < p->n_q_heads; ++hq) {
            const int hkv = hq / G;
            const int64_t rows = n_rows[(int64_t)b * p->n_kv_heads + hkv];
            double* o_vec = out + ((int64_t)b * p->n_q_heads + hq) * d;
            for (int64_t c = 0; c < d; ++c) o_vec[c] = 0.0;
            if (rows < 0 || rows > cap) { bad = 1; continue; }
            if (rows == 0) continue;
            const int64_t qbase = ((int64_t)b * p->n_q_heads + hq) * d;
            const int64_t kbase = ((int64_t)b * p->n_kv_heads + hkv) * cap * d;
            double* o = (double*)malloc(sizeof(double) * (size_t)rows);
            double* a = (double*)malloc(sizeof(double) * (size_t)rows);
            for (int64_t t = 0; t < rows; ++t) {
                double acc = 0.0;
                for (int64_t c = 0; c < d; ++c)
                    acc += load_elem(q, qbase + c, p->dtype) * load_elem(k, kbase + t * d + c, p->dtype);
                o[t] = acc * scale;
            }
            orc_nsoftmax(o, rows, p->n, a);
            for (int64_t t = 0; t < rows; ++t)
                for (int64_t c = 0; c < d; ++c) o_vec[c] += a[t] * load_elem(v, kbase + t * d + c, p->dtype);
            free(o); free(a);
        }
    }
    return bad ? -1 : 0;
}

/* Algorithm 1's iteration loop, one appended token: the decode attention of orc_decode_attn, and the row of
 * n-softmax weights it is built from added to the running sums of Eq. 1. */
int orc_decode_step(const orc_params* p, const void* q, const void* k, const void* v, const int32_t* n_rows,
                    const uint8_t* modality, const uint8_t* query_label, int first,
                    double* out, double* acc_self, double* acc_cross) {
    if (!p || !q || !k || !v || !n_rows || !modality || !query_label || !out || !acc_self || !acc_cross) return -1;
    const int64_t d = p->head_dim, cap = p->out_capacity;
    const int G = p->n_q_heads / p->n_kv_heads;
    const double scale = p->scale > 0.0 ? p->scale : 1.0 / sqrt((double)d);
    const int units = p->batch * p->n_kv_heads;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
    for (int u = 0; u < units; ++u) {
        const int b = u / p->n_kv_heads, h = u % p->n_kv_heads;
        const int64_t rows = n_rows[u];
        for (int g = 0; g < G; ++g)
            for (int64_t c = 0; c < d; ++c) out[((int64_t)b * p->n_q_heads + h * G + g) * d + c] = 0.0;
        if (rows < 0 || rows > cap) { bad = 1; continue; }
        double* as = acc_self + (int64_t)u * cap;
        double* ac = acc_cross + (int64_t)u * cap;
        /* a new window: every slot of the unit starts at zero, also those of rows still to be appended */
        if (first) for (int64_t t = 0; t < cap; ++t) { as[t] = 0.0; ac[t] = 0.0; }
        if (rows == 0) continue;
        const uint8_t* mod = modality + (int64_t)u * cap;
        const int64_t kbase = (int64_t)u * cap * d;
        double* o = (double*)malloc(sizeof(double) * (size_t)rows);
        double* a = (double*)malloc(sizeof(double) * (size_t)rows);
        for (int g = 0; g < G; ++g) {
            const int hq = h * G + g;
            const int64_t qbase = ((int64_t)b * p->n_q_heads + hq) * d;
            for (int64_t t = 0; t < rows; ++t) {
                double acc = 0.0;
                for (int64_t c = 0; c < d; ++c)
                    acc += load_elem(q, qbase + c, p->dtype) * load_elem(k, kbase + t * d + c, p->dtype);
                o[t] = acc * scale;                                   /* Eq. 5 for the one new query */
            }
            orc_nsoftmax(o, rows, p->n, a);                            /* Eq. 7 over the rows in the cache */
            double* o_vec = out + qbase;
            for (int64_t t = 0; t < rows; ++t) {
                for (int64_t c = 0; c < d; ++c) o_vec[c] += a[t] * load_elem(v, kbase + t * d + c, p->dtype);
                if (mod[t] == query_label[b]) as[t] += a[t] / G;       /* Eq. 1, one query row */
                else ac[t] += a[t] / G;
            }
        }
        free(o); free(a);
    }
    return bad ? -1 : 0;
}

/* ---- the distribution-gap diagnostic (Section 1) -------------------------------------------------- */

double orc_js_divergence(const int64_t* hp, const int64_t* hq, int bins) {
    double sp = 0.0, sq = 0.0;
    for (int j = 0; j < bins; ++j) { sp += (double)hp[j]; sq += (double)hq[j]; }
    if (sp <= 0.0 || sq <= 0.0) return NAN;
    double js = 0.0;
    for (int j = 0; j < bins; ++j) {
        const double pj = (double)hp[j] / sp, qj = (double)hq[j] / sq, mj = 0.5 * (pj + qj);
        if (pj > 0.0) js += 0.5 * pj * log(pj / mj);
        if (qj > 0.0) js += 0.5 * qj * log(qj / mj);
    }
    return js;
}

static int hist_bin(double log2w) {
    double j = floor((log2w - ORC_HIST_LO) / ORC_HIST_WIDTH);
    if (!(j >= 0.0)) j = 0.0;                      /* also catches -inf (weight 0) */
    if (j > ORC_HIST_BINS - 1) j = ORC_HIST_BINS - 1;
    return (int)j;
}

int orc_weight_histogram(const orc_params* p, const void* q, const void* k,
                         const uint8_t* modality, int mod_per_head, const int32_t* seq_lens,
                         int64_t* hist, int64_t* near, double near_eps, double* js, double* js_all) {
    if (!p || !q || !k || !modality || !seq_lens || !hist) return -1;
    if (p->n_kv_heads <= 0 || p->n_q_heads % p->n_kv_heads) return -1;
    const int G = p->n_q_heads / p->n_kv_heads, W = p->window, d = p->head_dim;
    const int units = p->batch * p->n_kv_heads;
    const double scale = p->scale > 0.0 ? p->scale : 1.0 / sqrt((double)d);
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(|:bad)
    for (int u = 0; u < units; ++u) {
        const int b = u / p->n_kv_heads, h = u % p->n_kv_heads;
        const int64_t L = seq_lens[b];
        int64_t* hu = hist + (int64_t)u * 2 * ORC_HIST_BINS;
        int64_t* nu = near ? near + (int64_t)u * 2 * ORC_HIST_BINS : NULL;
        for (int j = 0; j < 2 * ORC_HIST_BINS; ++j) { hu[j] = 0; if (nu) nu[j] = 0; }
        if (js) js[u] = NAN;
        if (L > p->max_len || L < 0) { bad = 1; continue; }
        if (unit_is_short(p, L)) continue;
        const int64_t N = L - p->recent;
        const uint8_t* mod = mod_row(p, modality, mod_per_head, b, h);
        double* o = (double*)malloc(sizeof(double) * (size_t)L);
        double* a = (double*)malloc(sizeof(double) * (size_t)L);
        const int64_t kbase = (int64_t)u * p->max_len * d;
        for (int g = 0; g < G; ++g) {
            const int64_t qbase = (((int64_t)b * p->n_q_heads + h * G + g) * W) * d;
            for (int w = 0; w < W; ++w) {
                const int64_t pos = L - W + w;
                for (int64_t t = 0; t <= pos; ++t) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c)
                        acc += load_elem(q, qbase + (int64_t)w * d + c, p->dtype) * load_elem(k, kbase + t * d + c, p->dtype);
                    o[t] = acc * scale;                           /* Eq. 5 */
                }
                orc_nsoftmax(o, pos + 1, p->n, a);                /* Eq. 7 */
                for (int64_t t = 0; t < N && t <= pos; ++t) {
                    const int cls = mod[pos] == mod[t] ? 0 : 1;   /* intra / inter, as in Eq. 1 */
                    const double l2 = a[t] > 0.0 ? log2(a[t]) : -INFINITY;
                    hu[cls * ORC_HIST_BINS + hist_bin(l2)] += 1;
                    if (nu && a[t] > 0.0) {
                        /* the nearest bin edge above the first and at or below the last bin's lower edge */
                        const double e = (l2 - ORC_HIST_LO) / ORC_HIST_WIDTH;
                        const double je = floor(e + 0.5);
                        if (je >= 1.0 && je <= ORC_HIST_BINS - 1 && fabs(e - je) * ORC_HIST_WIDTH <= near_eps)
                            nu[cls * ORC_HIST_BINS + (int)je] += 1;
                    }
                }
            }
        }
        free(o); free(a);
        if (js) js[u] = orc_js_divergence(hu, hu + ORC_HIST_BINS, ORC_HIST_BINS);
    }
    if (js_all) {
        int64_t tot[2 * ORC_HIST_BINS];
        for (int j = 0; j < 2 * ORC_HIST_BINS; ++j) tot[j] = 0;
        for (int u = 0; u < units; ++u)
            for (int j = 0; j < 2 * ORC_HIST_BINS; ++j) tot[j] += hist[(int64_t)u * 2 * ORC_HIST_BINS + j];
        *js_all = orc_js_divergence(tot, tot + ORC_HIST_BINS, ORC_HIST_BINS);
    }
    return bad ? -1 : 0;
}

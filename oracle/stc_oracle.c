/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow CPU statement of decode attention over a Quest-selected,
 * value-group-routed KV cache ("Sub-Token Routing for KV Cache Compression").
 * It exists so the CUDA library can be checked against something written
 * straight from the paper.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code with the CUDA
 * path and includes no CUDA header.
 *
 * Conventions
 *   - bf16 tensors are passed as uint16_t bit patterns.
 *   - One "problem" is one (batch, kv head) pair; every function with the
 *     suffix _batch loops over independent problems (OpenMP static split,
 *     no other parallelism, no blocking or fusion).
 *   - head_dim is 128, a page holds 16 tokens.
 *   - Integer-deciding arithmetic (the page bound) is fp32 in one declared
 *     summation order; attention arithmetic is fp64.
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py
 * (closed forms, brute force, textbook attention, invariants).  What is NOT
 * pinned, because it needs trained weights and evaluation suites: the paper's
 * accuracy tables -- "parity unpinned" for end-to-end model accuracy.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define D 128
#define PAGE 16

enum { CLS_DROP = 0, CLS_ROUTED = 1, CLS_FULL = 2 };
enum { MODE_GLOBAL = 0, MODE_PER_TOKEN = 1 };

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* Total order on bf16 bit patterns: numeric order, with -0 below +0. */
static int32_t bf16_order(uint16_t b) {
    return (b & 0x8000u) ? -(int32_t)(b & 0x7FFFu) - 1 : (int32_t)b;
}

/* ------------------------------------------------------------------------
 * Page metadata: per page and channel, the minimum and maximum key over the
 * page's valid tokens.  (Quest chunk size 16: Appendix C.1, Table "LLM
 * training configuration"; the page statistic is Quest's per-channel bound.)
 * k [len..][128], kmin/kmax [ceil(len/16)][128].
 * ---------------------------------------------------------------------- */
void stc_o_page_meta(const uint16_t* k, int32_t len, uint16_t* kmin, uint16_t* kmax) {
    int32_t n_pages = (len + PAGE - 1) / PAGE;
    for (int32_t p = 0; p < n_pages; ++p) {
        for (int c = 0; c < D; ++c) {
            uint16_t lo = 0, hi = 0;
            int first = 1;
            for (int32_t t = p * PAGE; t < (p + 1) * PAGE && t < len; ++t) {
                uint16_t x = k[(size_t)t * D + c];
                if (first) { lo = hi = x; first = 0; continue; }
                if (bf16_order(x) < bf16_order(lo)) lo = x;
                if (bf16_order(x) > bf16_order(hi)) hi = x;
            }
            kmin[(size_t)p * D + c] = lo;
            kmax[(size_t)p * D + c] = hi;
        }
    }
}

/* ------------------------------------------------------------------------
 * Page bound for one query head: U = sum_c max(q_c*kmin_c, q_c*kmax_c), an
 * upper bound of q.k_t for every token t of the page.
 *
 * Declared fp32 summation order (both sides of the parity check must use it,
 * because the bound decides integers): 16 partial sums; partial l covers
 * channels 8l..8l+7 and is formed as even + odd, where even adds the terms of
 * channels 8l, 8l+2, 8l+4, 8l+6 in ascending order starting from +0 and odd
 * does the same for 8l+1, 8l+3, 8l+5, 8l+7; the 16 partials are then combined
 * pairwise at distances 8, 4, 2, 1 (s[l] <- s[l] + s[l ^ dist]); the result
 * is s[0].
 * ---------------------------------------------------------------------- */
float stc_o_bound_f32(const uint16_t* q, const uint16_t* kmin, const uint16_t* kmax) {
    float s[16], n[16];
    for (int l = 0; l < 16; ++l) {
        float part[2] = {0.0f, 0.0f};           /* [0] even channels, [1] odd channels */
        for (int c = 8 * l; c < 8 * l + 8; ++c) {
            float qc = bf16_to_f32(q[c]);
            float a = qc * bf16_to_f32(kmin[c]);
            float b = qc * bf16_to_f32(kmax[c]);
            float t = a > b ? a : b;
            part[c & 1] = part[c & 1] + t;
        }
        s[l] = part[0] + part[1];
    }
    for (int dist = 8; dist >= 1; dist >>= 1) {
        for (int l = 0; l < 16; ++l) n[l] = s[l] + s[l ^ dist];
        memcpy(s, n, sizeof s);
    }
    return s[0];
}

double stc_o_bound_f64(const uint16_t* q, const uint16_t* kmin, const uint16_t* kmax) {
    double acc = 0.0;
    for (int c = 0; c < D; ++c) {
        double qc = bf16_to_f32(q[c]);
        double a = qc * bf16_to_f32(kmin[c]);
        double b = qc * bf16_to_f32(kmax[c]);
        acc += a > b ? a : b;
    }
    return acc;
}

/* Page scores for one problem: max over the query heads that share the KV
 * head.  q_group [gq][128]. */
void stc_o_page_scores(const uint16_t* q_group, int32_t gq, const uint16_t* kmin,
                       const uint16_t* kmax, int32_t n_pages, float* u) {
    for (int32_t p = 0; p < n_pages; ++p) {
        float best = 0.0f;
        for (int32_t h = 0; h < gq; ++h) {
            float x = stc_o_bound_f32(q_group + (size_t)h * D, kmin + (size_t)p * D,
                                      kmax + (size_t)p * D);
            if (h == 0 || x > best) best = x;
        }
        u[p] = best;
    }
}

typedef struct { float s; int64_t i; } cand_t;

static int cand_cmp(const void* a, const void* b) {
    const cand_t* x = (const cand_t*)a;
    const cand_t* y = (const cand_t*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);   /* ties: lower index first */
}

static int i32_cmp(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/* ------------------------------------------------------------------------
 * Page selection: keep the k_pg = min(n_pages, budget / 16) pages with the
 * largest score, ties to the lower page id; ids are emitted ascending.
 * Returns k_pg.
 * ---------------------------------------------------------------------- */
int32_t stc_o_select(const float* u, int32_t n_pages, int32_t token_budget, int32_t* page_ids) {
    int32_t k_pg = token_budget / PAGE;
    if (k_pg > n_pages) k_pg = n_pages;
    if (k_pg < 0) k_pg = 0;
    cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(n_pages > 0 ? n_pages : 1));
    for (int32_t p = 0; p < n_pages; ++p) { c[p].s = u[p]; c[p].i = p; }
    qsort(c, (size_t)n_pages, sizeof(cand_t), cand_cmp);
    for (int32_t j = 0; j < k_pg; ++j) page_ids[j] = (int32_t)c[j].i;
    qsort(page_ids, (size_t)k_pg, sizeof(int32_t), i32_cmp);
    free(c);
    return k_pg;
}

/* ------------------------------------------------------------------------
 * Page selection with a local window (Appendix C.1, LLM training configuration:
 * the table lists a Quest window of 64 beside the chunk of 16 -- read as Quest's
 * always-attended window of the most recent tokens, here n_recent_pages whole pages, counted against the
 * budget): with k_pg = min(n_pages, budget / 16) and w = min(n_recent_pages,
 * k_pg), the last w pages are kept and the other k_pg - w are the best-scoring
 * of the pages before them.  Ids ascending.  Returns k_pg.
 * ---------------------------------------------------------------------- */
int32_t stc_o_select_recent(const float* u, int32_t n_pages, int32_t token_budget,
                            int32_t n_recent_pages, int32_t* page_ids) {
    int32_t k_pg = token_budget / PAGE;
    if (k_pg > n_pages) k_pg = n_pages;
    if (k_pg < 0) k_pg = 0;
    int32_t w = n_recent_pages < 0 ? 0 : n_recent_pages;
    if (w > k_pg) w = k_pg;
    int32_t kept = stc_o_select(u, n_pages - w, (k_pg - w) * PAGE, page_ids);
    for (int32_t i = 0; i < w; ++i) page_ids[kept + i] = n_pages - w + i;
    return kept + w;
}

/* ------------------------------------------------------------------------
 * Routing mask (Section 3.3 "Routing mask", Section 3.4 global budget,
 * Appendix B.1 M = N*K).
 *   scores [len][S]; cls [len] or NULL (all routed); mask [len] out.
 *   GLOBAL:    N = number of routed tokens, M = N*k_nominal kept pairs.
 *              min_per_token = 1: each routed token first keeps its best group
 *              (first maximum), then the best M-N of the remaining pairs are
 *              kept; min_per_token = 0: the best M of all N*S pairs.
 *              Ties go to the lower flat index t*S+j.
 *   PER_TOKEN: every routed token keeps its best k_nominal groups
 *              (ties to the lower group).
 *   FULL tokens keep all S groups, DROP tokens none; neither uses budget.
 * Returns 0, or -1 when M < N with min_per_token = 1, or -2 on bad arguments.
 * ---------------------------------------------------------------------- */
int32_t stc_o_route(const float* scores, const uint8_t* cls, int32_t len, int32_t S,
                    int32_t k_nominal, int32_t min_per_token, int32_t mode, uint16_t* mask) {
    if (S < 1 || S > 16 || k_nominal < 0 || k_nominal > S) return -2;
    int64_t n_routed = 0;
    for (int32_t t = 0; t < len; ++t) {
        int c = cls ? cls[t] : CLS_ROUTED;
        mask[t] = (c == CLS_FULL) ? (uint16_t)((1u << S) - 1u) : 0;
        if (c == CLS_ROUTED) ++n_routed;
    }
    if (mode == MODE_PER_TOKEN) {
        cand_t g[16];
        for (int32_t t = 0; t < len; ++t) {
            if ((cls ? cls[t] : CLS_ROUTED) != CLS_ROUTED) continue;
            for (int j = 0; j < S; ++j) { g[j].s = scores[(size_t)t * S + j]; g[j].i = j; }
            qsort(g, (size_t)S, sizeof(cand_t), cand_cmp);
            for (int j = 0; j < k_nominal; ++j) mask[t] |= (uint16_t)(1u << g[j].i);
        }
        return 0;
    }
    int64_t m_total = n_routed * (int64_t)k_nominal;
    int64_t take = m_total;
    if (min_per_token) {
        if (m_total < n_routed) return -1;
        take = m_total - n_routed;
    }
    cand_t* c = (cand_t*)malloc(sizeof(cand_t) * (size_t)(n_routed * S + 1));
    int64_t n = 0;
    for (int32_t t = 0; t < len; ++t) {
        if ((cls ? cls[t] : CLS_ROUTED) != CLS_ROUTED) continue;
        int best = -1;
        if (min_per_token) {
            best = 0;
            for (int j = 1; j < S; ++j)
                if (scores[(size_t)t * S + j] > scores[(size_t)t * S + best]) best = j;
            mask[t] |= (uint16_t)(1u << best);
        }
        for (int j = 0; j < S; ++j) {
            if (j == best) continue;
            c[n].s = scores[(size_t)t * S + j];
            c[n].i = (int64_t)t * S + j;
            ++n;
        }
    }
    qsort(c, (size_t)n, sizeof(cand_t), cand_cmp);
    for (int64_t r = 0; r < take && r < n; ++r)
        mask[c[r].i / S] |= (uint16_t)(1u << (c[r].i % S));
    free(c);
    return 0;
}

/* ------------------------------------------------------------------------
 * Routing of pages completed during decoding (Section 3.4: global budget over the retained
 * tokens, M = N*K in Appendix B.1, query-region tokens uncompressed; the paper does not say
 * when a generated token leaves the query region -- reading taken: while its 16-token page is
 * still open; when the page completes, its 16 tokens join the routed set and the budget grows
 * by 16*K groups, which are allotted among the page's own (token, group) pairs by the rule of
 * stc_o_route, because the dropped groups of older tokens no longer exist in a packed store).
 *
 * One problem, in place.  Tokens first_page*16 .. len-1 are stored at full width (mask all
 * ones) behind the earlier tokens' groups.  Every complete page p, first_page <= p < len/16,
 * is routed on its own with scores [len][S] (rows of those pages are read); the tokens of the
 * still open page stay at full width and move down behind the compacted pages.  mask [len],
 * offs [len+1], packed [cap][128/S] are updated.  Returns the new total, -1 when the budget is
 * below one group per token with min_per_token = 1 (nothing changed), -2 on bad arguments or
 * when the range is not stored at full width (nothing changed).
 * ---------------------------------------------------------------------- */
int64_t stc_o_route_new_pages(const float* scores, int32_t len, int32_t S, int32_t first_page,
                              int32_t k_nominal, int32_t min_per_token, int32_t mode,
                              uint16_t* mask, uint32_t* offs, uint16_t* packed) {
    int g = D / S;
    int32_t t0 = first_page * PAGE;
    int32_t n_pages = len / PAGE - first_page;
    if (first_page < 0 || S < 1 || S > 16 || k_nominal < 0 || k_nominal > S) return -2;
    if (n_pages <= 0 || t0 >= len) return (int64_t)offs[len];
    for (int32_t t = t0; t < len; ++t)
        if (mask[t] != (uint16_t)((1u << S) - 1u) || offs[t + 1] - offs[t] != (uint32_t)S) return -2;
    if (mode == MODE_GLOBAL && min_per_token && k_nominal < 1) return -1;
    /* the full-width values of the range, read out before anything is overwritten */
    int32_t n_tok = len - t0;
    uint16_t* full = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n_tok * D);
    memcpy(full, packed + (size_t)offs[t0] * g, sizeof(uint16_t) * (size_t)n_tok * D);
    for (int32_t p = 0; p < n_pages; ++p)
        stc_o_route(scores + (size_t)(t0 + p * PAGE) * S, NULL, PAGE, S, k_nominal, min_per_token, mode,
                    mask + t0 + p * PAGE);
    int64_t n = offs[t0];
    for (int32_t t = t0; t < len; ++t) {
        offs[t] = (uint32_t)n;
        for (int j = 0; j < S; ++j) {
            if (!((mask[t] >> j) & 1u)) continue;
            memcpy(packed + (size_t)n * g, full + (size_t)(t - t0) * D + (size_t)j * g, sizeof(uint16_t) * (size_t)g);
            ++n;
        }
    }
    offs[len] = (uint32_t)n;
    free(full);
    return n;
}

/* ------------------------------------------------------------------------
 * Packing: walk the tokens in order; offs[t] is the number of groups kept
 * before token t (offs[len] = total); the kept groups of a token are stored
 * in ascending group order, each group_dim = 128/S bf16 values.
 * v [len][128], packed [cap_groups][128/S].  Returns the total, or -1 if it
 * exceeds cap_groups (nothing past the capacity is written).
 * ---------------------------------------------------------------------- */
int64_t stc_o_pack(const uint16_t* v, const uint16_t* mask, int32_t len, int32_t S,
                   int64_t cap_groups, uint32_t* offs, uint16_t* packed) {
    int g = D / S;
    int64_t n = 0;
    int over = 0;
    for (int32_t t = 0; t < len; ++t) {
        offs[t] = (uint32_t)n;
        for (int j = 0; j < S; ++j) {
            if (!((mask[t] >> j) & 1u)) continue;
            if (n < cap_groups)
                memcpy(packed + (size_t)n * g, v + (size_t)t * D + (size_t)j * g, (size_t)g * 2);
            else
                over = 1;
            ++n;
        }
    }
    offs[len] = (uint32_t)n;
    return over ? -1 : n;
}

/* ------------------------------------------------------------------------
 * Routed attention for one query head (Section 3.3, the attention equation):
 *   s_t = scale * q.k_t over the tokens of the listed pages (valid tokens
 *   only), p = softmax(s), out = sum_t p_t * v~_t, where v~_t has the kept
 *   groups of v_t and zero elsewhere.  The normaliser runs over every listed
 *   token, whether or not it kept any group.
 * page_ids NULL = all pages in order.  Values are read from the packed store
 * through mask/offs.  out [128] fp64; *lse = log sum_t exp(s_t) (natural log).
 * ---------------------------------------------------------------------- */
void stc_o_attend_packed(const uint16_t* q, const uint16_t* k, const uint16_t* packed,
                         const uint16_t* mask, const uint32_t* offs, int32_t len, int32_t S,
                         const int32_t* page_ids, int32_t n_pages_listed, double scale,
                         double* out, double* lse) {
    int g = D / S;
    int32_t total_pages = (len + PAGE - 1) / PAGE;
    int32_t n_list = page_ids ? n_pages_listed : total_pages;
    size_t n_tok = 0;
    double* s = (double*)malloc(sizeof(double) * ((size_t)n_list * PAGE + 1));
    int32_t* tok = (int32_t*)malloc(sizeof(int32_t) * ((size_t)n_list * PAGE + 1));
    for (int32_t i = 0; i < n_list; ++i) {
        int32_t p = page_ids ? page_ids[i] : i;
        for (int32_t t = p * PAGE; t < (p + 1) * PAGE && t < len; ++t) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c)
                dot += (double)bf16_to_f32(q[c]) * (double)bf16_to_f32(k[(size_t)t * D + c]);
            s[n_tok] = dot * scale;
            tok[n_tok] = t;
            ++n_tok;
        }
    }
    for (int c = 0; c < D; ++c) out[c] = 0.0;
    if (n_tok == 0) { if (lse) *lse = -INFINITY; free(s); free(tok); return; }
    double mx = s[0];
    for (size_t i = 1; i < n_tok; ++i) if (s[i] > mx) mx = s[i];
    double den = 0.0;
    for (size_t i = 0; i < n_tok; ++i) { s[i] = exp(s[i] - mx); den += s[i]; }
    for (size_t i = 0; i < n_tok; ++i) {
        int32_t t = tok[i];
        double p = s[i] / den;
        int64_t slot = offs[t];
        for (int j = 0; j < S; ++j) {
            if (!((mask[t] >> j) & 1u)) continue;
            for (int e = 0; e < g; ++e)
                out[j * g + e] += p * (double)bf16_to_f32(packed[(size_t)slot * g + e]);
            ++slot;
        }
    }
    if (lse) *lse = mx + log(den);
    free(s);
    free(tok);
}

/* Same definition, reading values from the dense V through the mask: the
 * attention equation applied to v~ = m * v literally. */
void stc_o_attend_masked_dense(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                               const uint16_t* mask, int32_t len, int32_t S,
                               const int32_t* page_ids, int32_t n_pages_listed, double scale,
                               double* out, double* lse) {
    int g = D / S;
    int32_t total_pages = (len + PAGE - 1) / PAGE;
    int32_t n_list = page_ids ? n_pages_listed : total_pages;
    size_t n_tok = 0;
    double* s = (double*)malloc(sizeof(double) * ((size_t)n_list * PAGE + 1));
    int32_t* tok = (int32_t*)malloc(sizeof(int32_t) * ((size_t)n_list * PAGE + 1));
    for (int32_t i = 0; i < n_list; ++i) {
        int32_t p = page_ids ? page_ids[i] : i;
        for (int32_t t = p * PAGE; t < (p + 1) * PAGE && t < len; ++t) {
            double dot = 0.0;
            for (int c = 0; c < D; ++c)
                dot += (double)bf16_to_f32(q[c]) * (double)bf16_to_f32(k[(size_t)t * D + c]);
            s[n_tok] = dot * scale;
            tok[n_tok] = t;
            ++n_tok;
        }
    }
    for (int c = 0; c < D; ++c) out[c] = 0.0;
    if (n_tok == 0) { if (lse) *lse = -INFINITY; free(s); free(tok); return; }
    double mx = s[0];
    for (size_t i = 1; i < n_tok; ++i) if (s[i] > mx) mx = s[i];
    double den = 0.0;
    for (size_t i = 0; i < n_tok; ++i) { s[i] = exp(s[i] - mx); den += s[i]; }
    for (size_t i = 0; i < n_tok; ++i) {
        int32_t t = tok[i];
        double p = s[i] / den;
        for (int c = 0; c < D; ++c) {
            double m = (double)((mask[t] >> (c / g)) & 1u);
            out[c] += p * m * (double)bf16_to_f32(v[(size_t)t * D + c]);
        }
    }
    if (lse) *lse = mx + log(den);
    free(s);
    free(tok);
}

/* Retained-KV fraction by counting stored bytes (Section 3.3 "Compression
 * ratio", Appendix C.2: rho_total = r * (1 + K/S) / 2): full-width keys of the
 * retained tokens plus the packed value groups, over dense keys + values of
 * all original tokens. */
double stc_o_kv_fraction(int64_t n_tokens_original, int64_t n_tokens_retained,
                         int64_t n_groups_kept, int32_t S) {
    double key_bytes = (double)n_tokens_retained * D * 2.0;
    double val_bytes = (double)n_groups_kept * (D / S) * 2.0;
    double dense = (double)n_tokens_original * D * 2.0 * 2.0;
    return (key_bytes + val_bytes) / dense;
}

/* ========================================================================
 * Batched drivers over the library's tensor layouts.  Problems (b, kv head)
 * are independent; the only parallelism is a static split of that loop.
 *   k, v        [B][Hkv][t_cap][128]
 *   kmin, kmax  [B][Hkv][p_cap][128],  p_cap = ceil(t_cap/16)
 *   q           [B][Hq][128]
 *   scores      [B][Hkv][t_cap][S]
 *   cls         [B][Hkv or 1][t_cap]   (cls_head_stride = t_cap or 0)
 *   mask        [B][Hkv][t_cap]; offs [B][Hkv][t_cap+1]
 *   packed      [B][Hkv][cap_groups][128/S]
 *   page_ids    [B][Hkv][max_pages]; n_pages [B][Hkv]
 * seq_len [B] gives the valid tokens per sequence (NULL = t_cap).
 * ====================================================================== */
static int32_t len_of(const int32_t* seq_len, int32_t b, int32_t t_cap) {
    int32_t n = seq_len ? seq_len[b] : t_cap;
    if (n < 0) n = 0;
    if (n > t_cap) n = t_cap;
    return n;
}

void stc_o_page_meta_batch(int32_t B, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                           const uint16_t* k, uint16_t* kmin, uint16_t* kmax) {
    int32_t p_cap = (t_cap + PAGE - 1) / PAGE;
#pragma omp parallel for schedule(static)
    for (int32_t pr = 0; pr < B * Hkv; ++pr) {
        int32_t b = pr / Hkv;
        stc_o_page_meta(k + (size_t)pr * t_cap * D, len_of(seq_len, b, t_cap),
                        kmin + (size_t)pr * p_cap * D, kmax + (size_t)pr * p_cap * D);
    }
}

void stc_o_select_batch_recent(int32_t B, int32_t Hq, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                               const uint16_t* q, const uint16_t* kmin, const uint16_t* kmax,
                               int32_t token_budget, int32_t n_recent_pages, int32_t max_pages,
                               int32_t* page_ids, int32_t* n_pages,
                               float* scores_out /* [B][Hkv][p_cap] or NULL */) {
    int32_t p_cap = (t_cap + PAGE - 1) / PAGE;
    int32_t gq = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int32_t pr = 0; pr < B * Hkv; ++pr) {
        int32_t b = pr / Hkv, hk = pr % Hkv;
        int32_t len = len_of(seq_len, b, t_cap);
        int32_t np = (len + PAGE - 1) / PAGE;
        float* u = (float*)malloc(sizeof(float) * (size_t)(p_cap + 1));
        int32_t* ids = (int32_t*)malloc(sizeof(int32_t) * (size_t)(p_cap + 1));
        stc_o_page_scores(q + ((size_t)b * Hq + (size_t)hk * gq) * D, gq,
                          kmin + (size_t)pr * p_cap * D, kmax + (size_t)pr * p_cap * D, np, u);
        int32_t kp = stc_o_select_recent(u, np, token_budget, n_recent_pages, ids);
        if (kp > max_pages) kp = max_pages;   /* caller sized the list too small: truncated */
        memcpy(page_ids + (size_t)pr * max_pages, ids, sizeof(int32_t) * (size_t)kp);
        n_pages[pr] = kp;
        if (scores_out) memcpy(scores_out + (size_t)pr * p_cap, u, sizeof(float) * (size_t)np);
        free(u);
        free(ids);
    }
}

void stc_o_select_batch(int32_t B, int32_t Hq, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                        const uint16_t* q, const uint16_t* kmin, const uint16_t* kmax,
                        int32_t token_budget, int32_t max_pages, int32_t* page_ids,
                        int32_t* n_pages, float* scores_out) {
    stc_o_select_batch_recent(B, Hq, Hkv, t_cap, seq_len, q, kmin, kmax, token_budget, 0, max_pages, page_ids,
                              n_pages, scores_out);
}

/* Near-tie count of the page selection, per problem: with U64[p] = max over the problem's query
 * heads of the bound accumulated in fp64 (stc_o_bound_f64) and U_k its k-th largest value
 * (k = min(n_pages, budget / 16)), the number of OTHER pages with |U64[p] - U_k| <=
 * rel * max(1, |U_k|).  0 when every page or no page is selected.  A reporting aid: these are the
 * pages whose membership in the selection hangs on the last bits of the fp32 sum. */
static int f64_desc(const void* a, const void* b) {
    double x = *(const double*)a, y = *(const double*)b;
    return x > y ? -1 : (x < y ? 1 : 0);
}

void stc_o_near_ties_batch(int32_t B, int32_t Hq, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                           const uint16_t* q, const uint16_t* kmin, const uint16_t* kmax,
                           int32_t token_budget, double rel, int32_t* counts /* [B][Hkv] */) {
    int32_t p_cap = (t_cap + PAGE - 1) / PAGE;
    int32_t gq = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int32_t pr = 0; pr < B * Hkv; ++pr) {
        int32_t b = pr / Hkv, hk = pr % Hkv;
        int32_t np = (len_of(seq_len, b, t_cap) + PAGE - 1) / PAGE;
        int32_t k = token_budget / PAGE < np ? token_budget / PAGE : np;
        counts[pr] = 0;
        if (k <= 0 || k >= np) continue;
        double* u = (double*)malloc(sizeof(double) * (size_t)np * 2);
        double* sorted = u + np;
        for (int32_t p = 0; p < np; ++p) {
            double best = 0.0;
            for (int32_t h = 0; h < gq; ++h) {
                double x = stc_o_bound_f64(q + ((size_t)b * Hq + (size_t)hk * gq + h) * D,
                                           kmin + ((size_t)pr * p_cap + p) * D, kmax + ((size_t)pr * p_cap + p) * D);
                if (h == 0 || x > best) best = x;
            }
            u[p] = best;
        }
        memcpy(sorted, u, sizeof(double) * (size_t)np);
        qsort(sorted, (size_t)np, sizeof(double), f64_desc);
        double uk = sorted[k - 1];
        double tol = rel * (fabs(uk) > 1.0 ? fabs(uk) : 1.0);
        int32_t c = 0;
        for (int32_t p = 0; p < np; ++p) c += fabs(u[p] - uk) <= tol;
        counts[pr] = c - 1;
        free(u);
    }
}

/* status [B*Hkv]: 0 ok, -1 budget below one group per token, -2 bad args,
 * -3 capacity overflow.  total [B*Hkv] = groups kept. */
void stc_o_route_pack_batch(int32_t B, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                            int32_t S, const uint16_t* v, const float* scores,
                            const uint8_t* cls, int64_t cls_head_stride, int32_t k_nominal,
                            int32_t min_per_token, int32_t mode, int64_t cap_groups,
                            uint16_t* mask, uint32_t* offs, uint16_t* packed, int64_t* total,
                            int32_t* status) {
    int g = D / S;
#pragma omp parallel for schedule(static)
    for (int32_t pr = 0; pr < B * Hkv; ++pr) {
        int32_t b = pr / Hkv, hk = pr % Hkv;
        int32_t len = len_of(seq_len, b, t_cap);
        const uint8_t* c = 0;
        if (cls) {
            int64_t per_b = cls_head_stride ? (int64_t)Hkv * cls_head_stride : (int64_t)t_cap;
            c = cls + (size_t)b * per_b + (size_t)hk * cls_head_stride;
        }
        uint16_t* m = mask + (size_t)pr * t_cap;
        uint32_t* o = offs + (size_t)pr * (t_cap + 1);
        int32_t rc = stc_o_route(scores + (size_t)pr * t_cap * S, c, len, S, k_nominal,
                                 min_per_token, mode, m);
        status[pr] = rc;
        total[pr] = 0;
        if (rc != 0) continue;
        int64_t n = stc_o_pack(v + (size_t)pr * t_cap * D, m, len, S, cap_groups, o,
                               packed + (size_t)pr * cap_groups * g);
        if (n < 0) { status[pr] = -3; total[pr] = o[len]; } else total[pr] = n;
    }
}

/* use_dense = 0: read values from the packed store; 1: from dense v through
 * the mask.  out [B][Hq][128] fp64, lse [B][Hq] fp64 (may be NULL). */
void stc_o_attend_batch(int32_t B, int32_t Hq, int32_t Hkv, int32_t t_cap, const int32_t* seq_len,
                        int32_t S, const uint16_t* q, const uint16_t* k, const uint16_t* v_dense,
                        const uint16_t* packed, int64_t cap_groups, const uint16_t* mask,
                        const uint32_t* offs, const int32_t* page_ids, const int32_t* n_pages,
                        int32_t max_pages, double scale, int32_t use_dense, double* out,
                        double* lse) {
    int g = D / S;
    int32_t gq = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int32_t bh = 0; bh < B * Hq; ++bh) {
        int32_t b = bh / Hq, h = bh % Hq;
        int32_t pr = b * Hkv + h / gq;
        int32_t len = len_of(seq_len, b, t_cap);
        const int32_t* ids = page_ids ? page_ids + (size_t)pr * max_pages : 0;
        int32_t nl = page_ids ? n_pages[pr] : 0;
        double* l = lse ? lse + bh : 0;
        if (use_dense)
            stc_o_attend_masked_dense(q + (size_t)bh * D, k + (size_t)pr * t_cap * D,
                                      v_dense + (size_t)pr * t_cap * D, mask + (size_t)pr * t_cap,
                                      len, S, ids, nl, scale, out + (size_t)bh * D, l);
        else
            stc_o_attend_packed(q + (size_t)bh * D, k + (size_t)pr * t_cap * D,
                                packed + (size_t)pr * cap_groups * g, mask + (size_t)pr * t_cap,
                                offs + (size_t)pr * (t_cap + 1), len, S, ids, nl, scale,
                                out + (size_t)bh * D, l);
    }
}

/* ------------------------------------------------------------------------
 * Value-group router (Appendix B.1 "Value-Group Router": a single linear
 * projection from the layer input hidden state to S group logits; Section 3.4
 * gives the LLM form a = g(h, s_Q), read here as the same linear map applied to
 * [h ; s_Q], whose s_Q part is one additive vector per sequence).
 *   h     [B][T][d_model]  bf16 hidden states
 *   w     [Hkv*S][d_model] bf16 router weights, row hk*S + j = group j of KV head hk
 *   bias  [B][Hkv*S] fp32 or NULL (the query-summary term)
 *   out   [B][Hkv][T][S]   fp64 logits, the layout of the routing scores
 * ---------------------------------------------------------------------- */
void stc_o_router_logits(int32_t B, int32_t Hkv, int32_t T, int32_t S, int32_t d_model,
                         const uint16_t* h, const uint16_t* w, const float* bias, double* out) {
    int32_t N = Hkv * S;
#pragma omp parallel for schedule(static)
    for (int64_t bt = 0; bt < (int64_t)B * T; ++bt) {
        int32_t b = (int32_t)(bt / T), t = (int32_t)(bt % T);
        const uint16_t* hr = h + (size_t)bt * d_model;
        for (int32_t n = 0; n < N; ++n) {
            const uint16_t* wr = w + (size_t)n * d_model;
            double acc = 0.0;
            for (int32_t c = 0; c < d_model; ++c)
                acc += (double)bf16_to_f32(hr[c]) * (double)bf16_to_f32(wr[c]);
            if (bias) acc += (double)bias[(size_t)b * N + n];
            out[(((size_t)b * Hkv + n / S) * T + t) * S + n % S] = acc;
        }
    }
}

/* ----------------------------------------------------------------------
 * Query summary and its router term (Section 3.4: the router sees the token's
 * hidden state and a summary s_Q of the query region; the summary operator and
 * g are not specified, the reading taken here is s_Q = mean of the query-region
 * hidden states and g linear in [h ; s_Q], so the query enters as one additive
 * term per sequence):
 *     s_q[b][c]  = (1 / q_len[b]) * sum_{t < q_len[b]} h_q[b][t][c]     (0 when q_len[b] = 0)
 *     bias[b][n] = sum_c s_q[b][c] * w_q[n][c]
 *   h_q   [B][Lq][d_model] bf16 bits, q_len [B] or NULL (= Lq), w_q [N][d_model] bf16 bits
 *   s_q   [B][d_model] fp64, bias [B][N] fp64
 * ---------------------------------------------------------------------- */
void stc_o_query_bias(int32_t B, int32_t Lq, int32_t d_model, int32_t N, const uint16_t* h_q,
                      const int32_t* q_len, const uint16_t* w_q, double* s_q, double* bias) {
    for (int32_t b = 0; b < B; ++b) {
        int32_t n_tok = q_len ? q_len[b] : Lq;
        if (n_tok < 0) n_tok = 0;
        if (n_tok > Lq) n_tok = Lq;
        for (int32_t c = 0; c < d_model; ++c) {
            double acc = 0.0;
            for (int32_t t = 0; t < n_tok; ++t)
                acc += (double)bf16_to_f32(h_q[((size_t)b * Lq + t) * d_model + c]);
            s_q[(size_t)b * d_model + c] = n_tok > 0 ? acc / (double)n_tok : 0.0;
        }
        for (int32_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int32_t c = 0; c < d_model; ++c)
                acc += s_q[(size_t)b * d_model + c] * (double)bf16_to_f32(w_q[(size_t)n * d_model + c]);
            bias[(size_t)b * N + n] = acc;
        }
    }
}

int32_t stc_o_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

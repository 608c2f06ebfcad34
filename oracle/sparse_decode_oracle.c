/*
 * CPU oracle for query-aware sparse decode attention over a paged KV cache.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It exists so that the CUDA path can
 * be checked against the paper's equations.  Only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it.  It shares no code, header, table or
 * helper with the CUDA library and is never a fallback for it.
 *
 * Everything is computed in fp64 on the bf16-rounded inputs (a bf16 value converts to
 * double exactly), with plain loops in the order the paper's definitions give them:
 *
 *   se_oracle_meta     Quest page summaries            (Appendix A, Quest, summary eq.)
 *   se_oracle_scores   Quest page score, group max     (Appendix A, Quest, score eq.)
 *   se_oracle_topk     TopK_b(s; A)                    (Appendix A, notation table)
 *   se_oracle_attend   attention over selected tokens  (Appendix A, selected-attention eq.)
 *                      + H2O accumulated score         (Appendix A, H2O score eq.)
 *   se_oracle_h2o_retain   H2O retained set R = W u TopK(u; A \ W)   (Appendix A, H2O retention eq.)
 *   se_oracle_h2o_compact  eviction: retained tokens moved to the front of the request's cache
 *   se_oracle_token_scores observation-layer selector s(j) = max_a z_j^(a)   (Appendix A, OmniKV selection eq.)
 *   se_oracle_token_topk   J = TopK_b(s; [i]) plus the always-kept recent tokens
 *   se_oracle_token_attend attention of every head over one token set per request (OmniKV reuse eq.)
 *
 * Conventions (0-based everywhere; the paper's positions are 1-based):
 *   logical page b of request r holds tokens [b*p, min(len_r, (b+1)*p)); its physical
 *   page is page_table[r][b]; an entry of -1 means the page has no physical KV and is
 *   never summarised, scored, selected or attended.  Query head a reads kv-head
 *   g(a) = a / G with G = H_q / H_kv.
 *
 * Parity pins (tests, CPU only): brute-force min/max, the bound property of the page
 * score, equality with a token logit on single-token pages, unit-vector closed forms,
 * argsort brute force for top-k, equality with dense attention when every page is
 * selected, log-sum-exp against a library routine, the unit sum of attention mass.
 * For the H2O retention: the paper's budget-4 / two-recent-tokens example, argsort brute force,
 * the "a token that leaves the window competes on its score" scenario, and equality of attention
 * over the retained tokens before and after compaction.
 * Parity with the authors' own code is unpinned: the paper prints no numbers for
 * this path, and the reduction of a GQA group to one per-kv-head score (max) is a
 * convention of this build.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t bits) {
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static int tokens_in_page(int len, int b, int p) {
    int nv = len - b * p;
    if (nv > p) nv = p;
    return nv < 0 ? 0 : nv;
}

/* strictly "x sorts below y" with -0 below +0, so that ties between the two zeros are
 * resolved the same way on every platform (min keeps -0, max keeps +0). */
static int lt_signed_zero(uint16_t xb, uint16_t yb) {
    double x = bf16_to_f64(xb), y = bf16_to_f64(yb);
    if (x < y) return 1;
    if (x > y) return 0;
    return (xb >> 15) > (yb >> 15);
}

/*
 * Quest page summaries: for every request r, every logical page b >= first_tok[r]/p that
 * has a physical page pid, every kv-head h and channel c,
 *     m[pid,h,c] = min_t K[pid,h,t,c],  M[pid,h,c] = max_t K[pid,h,t,c]
 * over the tokens t of the page that lie below len_r.  first_tok == NULL recomputes only
 * the page that holds each request's newest token.  A min or max of bf16 values is one
 * of them, so the summary is stored as bf16 bits and is exact.
 *   k_cache [P, H_kv, p, D] bf16 bits      meta [P, H_kv, 2, D] bf16 bits (row 0 min, row 1 max)
 */
void se_oracle_meta(int B, int H_kv, int D, int p, int max_pages,
                    const uint16_t *k_cache, const int32_t *page_table,
                    const int32_t *seq_lens, const int32_t *first_tok,
                    uint16_t *meta) {
    for (int r = 0; r < B; ++r) {
        int len = seq_lens[r];
        if (len <= 0) continue;
        int n_r = (len + p - 1) / p;
        int b0 = first_tok ? first_tok[r] / p : n_r - 1;
        if (b0 < 0) b0 = 0;
        for (int b = b0; b < n_r; ++b) {
            int pid = page_table[(size_t)r * max_pages + b];
            if (pid < 0) continue;
            int nv = tokens_in_page(len, b, p);
            for (int h = 0; h < H_kv; ++h) {
                const uint16_t *kp = k_cache + (((size_t)pid * H_kv + h) * p) * D;
                uint16_t *mn = meta + (((size_t)pid * H_kv + h) * 2 + 0) * D;
                uint16_t *mx = meta + (((size_t)pid * H_kv + h) * 2 + 1) * D;
                for (int c = 0; c < D; ++c) {
                    uint16_t lo = kp[c], hi = kp[c];
                    for (int t = 1; t < nv; ++t) {
                        uint16_t v = kp[(size_t)t * D + c];
                        if (lt_signed_zero(v, lo)) lo = v;
                        if (lt_signed_zero(hi, v)) hi = v;
                    }
                    mn[c] = lo;
                    mx[c] = hi;
                }
            }
        }
    }
}

/*
 * Quest page score.  For query head a of request r and logical page b with physical page
 * pid >= 0:
 *     S[r,a,b] = sm_scale * sum_c max( q[r,a,c]*m[pid,g(a),c], q[r,a,c]*M[pid,g(a),c] )
 * (channels summed left to right), and the per-kv-head score that is ranked
 *     P[r,h,b] = max over the query heads a of group h of S[r,a,b]
 * (group_sum != 0 replaces that max by a sum; the CUDA path implements the max only).
 * Pages that are absent or lie past the request's length get present = 0 and score 0.
 *   q [B,H_q,D] bf16 bits   S [B,H_q,max_pages]   P [B,H_kv,max_pages]   present [B,max_pages]
 */
void se_oracle_scores(int B, int H_q, int H_kv, int D, int p, int max_pages,
                      double sm_scale, int group_sum,
                      const uint16_t *q, const uint16_t *meta,
                      const int32_t *page_table, const int32_t *seq_lens,
                      double *S, double *P, uint8_t *present) {
    int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic)
    for (int rh = 0; rh < B * H_kv; ++rh) {
        int r = rh / H_kv, h = rh % H_kv;
        int len = seq_lens[r];
        int n_r = len > 0 ? (len + p - 1) / p : 0;
        for (int b = 0; b < max_pages; ++b) {
            int pid = b < n_r ? page_table[(size_t)r * max_pages + b] : -1;
            if (h == 0) present[(size_t)r * max_pages + b] = (uint8_t)(pid >= 0);
            double best = 0.0, total = 0.0;
            for (int g = 0; g < G; ++g) {
                int a = h * G + g;
                double s = 0.0;
                if (pid >= 0) {
                    const uint16_t *mn = meta + (((size_t)pid * H_kv + h) * 2 + 0) * D;
                    const uint16_t *mx = meta + (((size_t)pid * H_kv + h) * 2 + 1) * D;
                    const uint16_t *qa = q + ((size_t)r * H_q + a) * D;
                    for (int c = 0; c < D; ++c) {
                        double qc = bf16_to_f64(qa[c]);
                        double lo = qc * bf16_to_f64(mn[c]);
                        double hi = qc * bf16_to_f64(mx[c]);
                        s += lo > hi ? lo : hi;
                    }
                    s *= sm_scale;
                }
                S[((size_t)r * H_q + a) * max_pages + b] = s;
                if (g == 0 || s > best) best = s;
                total += s;
            }
            P[((size_t)r * H_kv + h) * max_pages + b] = group_sum ? total : best;
        }
    }
}

typedef struct { double s; int b; } cand_t;

static int cand_cmp(const void *x, const void *y) {
    const cand_t *a = (const cand_t *)x, *c = (const cand_t *)y;
    if (a->s > c->s) return -1;
    if (a->s < c->s) return 1;
    return a->b - c->b;                       /* equal scores: lower page first */
}

static int int_cmp(const void *x, const void *y) {
    return *(const int *)x - *(const int *)y;
}

/*
 * TopK: among the present pages of request r, the k_eff = min(floor(budget/p), #candidates)
 * pages with the largest P[r,h,.]; equal scores are ordered by lower logical page.  The
 * chosen logical page numbers are written in ascending order, the rest of the row is -1.
 * Forced pages (the paper's Quest settings keep "sink" and "recent" tokens outside the selected
 * budget): the first sink_pages logical pages and the last recent_pages logical pages of the
 * request (n_pages[r] = pages the request's length spans) are always in the result when present;
 * they are not candidates and do not count against the budget.
 * theta[r,h,0] is the k_eff-th largest candidate score, theta[r,h,1] the (k_eff+1)-th (NaN if
 * none): the caller uses them to see how close a decision was.
 *   sel_idx [B,H_kv,k_max]   sel_cnt [B,H_kv]   theta [B,H_kv,2]
 */
void se_oracle_topk(int B, int H_kv, int p, int max_pages, int k_max, int budget,
                    int sink_pages, int recent_pages, const int32_t *n_pages,
                    const double *P, const uint8_t *present,
                    int32_t *sel_idx, int32_t *sel_cnt, double *theta) {
    int k = budget / p;
#pragma omp parallel for schedule(dynamic)
    for (int rh = 0; rh < B * H_kv; ++rh) {
        int r = rh / H_kv;
        int n_r = n_pages ? n_pages[r] : max_pages;
        cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(max_pages > 0 ? max_pages : 1));
        int *chosen = (int *)malloc(sizeof(int) * (size_t)(max_pages > 0 ? max_pages : 1));
        int n = 0, n_chosen = 0;
        for (int b = 0; b < max_pages; ++b) {
            if (!present[(size_t)r * max_pages + b]) continue;
            int forced = (b < sink_pages) || (b >= n_r - recent_pages && b < n_r);
            if (forced) {
                chosen[n_chosen++] = b;
            } else {
                cand[n].s = P[(size_t)rh * max_pages + b];
                cand[n].b = b;
                ++n;
            }
        }
        qsort(cand, (size_t)n, sizeof(cand_t), cand_cmp);
        int k_eff = k < n ? k : n;
        if (k_eff > k_max - n_chosen) k_eff = k_max - n_chosen > 0 ? k_max - n_chosen : 0;
        if (n_chosen > k_max) n_chosen = k_max;
        for (int i = 0; i < k_eff; ++i) chosen[n_chosen++] = cand[i].b;
        qsort(chosen, (size_t)n_chosen, sizeof(int), int_cmp);
        for (int i = 0; i < k_max; ++i)
            sel_idx[(size_t)rh * k_max + i] = i < n_chosen ? chosen[i] : -1;
        sel_cnt[rh] = n_chosen;
        theta[(size_t)rh * 2 + 0] = k_eff > 0 ? cand[k_eff - 1].s : NAN;
        theta[(size_t)rh * 2 + 1] = k_eff < n ? cand[k_eff].s : NAN;
        free(chosen);
        free(cand);
    }
}

/*
 * Attention over the tokens of the selected pages.  For query head a of request r the
 * attended set T holds every token (b,t) with b in sel_idx[r,g(a),0..sel_cnt) and
 * t below the number of valid tokens of page b.  Then
 *     z_j = sm_scale * sum_c q_c k_{j,c},   alpha_j = exp(z_j) / sum_{u in T} exp(z_u),
 *     out_c = sum_j alpha_j v_{j,c},        lse = ln sum_{u in T} exp(z_u)
 * (evaluated with the maximum logit subtracted).  An empty T gives out = 0, lse = -inf.
 * If u_accum is not NULL, the H2O statistic of every attended token slot grows by the
 * attention mass it received, summed over the query heads of its kv-head:
 *     u[pid,h,t] += sum_{a in group h} alpha_{a,(b,t)} .
 *   out [B,H_q,D]   lse [B,H_q]   u_accum [P,H_kv,p] (in/out)
 */
void se_oracle_attend(int B, int H_q, int H_kv, int D, int p, int max_pages, int k_max,
                      double sm_scale,
                      const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                      const int32_t *page_table, const int32_t *seq_lens,
                      const int32_t *sel_idx, const int32_t *sel_cnt,
                      double *out, double *lse, double *u_accum) {
    int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic)
    for (int rh = 0; rh < B * H_kv; ++rh) {
        int r = rh / H_kv, h = rh % H_kv;
        int len = seq_lens[r];
        int cnt = sel_cnt[rh];
        double *z = (double *)malloc(sizeof(double) * (size_t)(cnt > 0 ? cnt : 1) * p);
        for (int g = 0; g < G; ++g) {
            int a = h * G + g;
            const uint16_t *qa = q + ((size_t)r * H_q + a) * D;
            double *o = out + ((size_t)r * H_q + a) * D;
            for (int c = 0; c < D; ++c) o[c] = 0.0;
            /* logits */
            double zmax = -INFINITY;
            int any = 0;
            for (int i = 0; i < cnt; ++i) {
                int b = sel_idx[(size_t)rh * k_max + i];
                int pid = b >= 0 ? page_table[(size_t)r * max_pages + b] : -1;
                int nv = (b >= 0 && pid >= 0) ? tokens_in_page(len, b, p) : 0;
                for (int t = 0; t < p; ++t) {
                    double zz = -INFINITY;
                    if (t < nv) {
                        const uint16_t *kt = k_cache + ((((size_t)pid * H_kv + h) * p) + t) * D;
                        double s = 0.0;
                        for (int c = 0; c < D; ++c) s += bf16_to_f64(qa[c]) * bf16_to_f64(kt[c]);
                        zz = s * sm_scale;
                        any = 1;
                        if (zz > zmax) zmax = zz;
                    }
                    z[(size_t)i * p + t] = zz;
                }
            }
            if (!any) {
                lse[(size_t)r * H_q + a] = -INFINITY;
                continue;
            }
            /* normaliser */
            double denom = 0.0;
            for (int i = 0; i < cnt * p; ++i)
                if (z[i] > -INFINITY) denom += exp(z[i] - zmax);
            lse[(size_t)r * H_q + a] = zmax + log(denom);
            /* weighted values and the H2O statistic */
            for (int i = 0; i < cnt; ++i) {
                int b = sel_idx[(size_t)rh * k_max + i];
                int pid = b >= 0 ? page_table[(size_t)r * max_pages + b] : -1;
                for (int t = 0; t < p; ++t) {
                    double zz = z[(size_t)i * p + t];
                    if (!(zz > -INFINITY)) continue;
                    double alpha = exp(zz - zmax) / denom;
                    const uint16_t *vt = v_cache + ((((size_t)pid * H_kv + h) * p) + t) * D;
                    for (int c = 0; c < D; ++c) o[c] += alpha * bf16_to_f64(vt[c]);
                    if (u_accum) u_accum[((size_t)pid * H_kv + h) * p + t] += alpha;
                }
            }
        }
        free(z);
    }
}

/*
 * H2O retained set (Appendix A, "H2O: Accumulated Scores and Online Eviction", retention equation).
 * For request r (len_r tokens, token j in logical page j/p, slot j%p) and kv-head h:
 *     A = the tokens of the request whose page has a physical page,
 *     W = the tokens of A among the last w = min(recent, budget) positions of the request,
 *     R = W  u  TopK_{budget-|W|}(u; A \ W)      (all of A \ W if it has fewer members),
 * where u[pid,h,t] is the accumulated score of the token stored in slot t of physical page pid.
 * Equal scores are ordered by lower position.  keep_idx[r,h,:] lists R in ascending token
 * position, padded with -1 up to `budget` entries; keep_cnt[r,h] = |R| (the same for every head
 * of a request, since it only depends on |A|).
 *   u [P, H_kv, p] (double)   keep_idx [B, H_kv, budget]   keep_cnt [B, H_kv]
 */
typedef struct { double u; int pos; } tok_t;

static int tok_cmp(const void *x, const void *y) {
    const tok_t *a = (const tok_t *)x, *b = (const tok_t *)y;
    if (a->u > b->u) return -1;
    if (a->u < b->u) return 1;
    return (a->pos > b->pos) - (a->pos < b->pos);
}

void se_oracle_h2o_retain(int B, int H_kv, int p, int max_pages, int budget, int recent,
                          const double *u, const int32_t *page_table, const int32_t *seq_lens,
                          int32_t *keep_idx, int32_t *keep_cnt) {
    const int w = recent < budget ? recent : budget;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int r = 0; r < B; ++r)
        for (int h = 0; h < H_kv; ++h) {
            int len = seq_lens[r];
            if (len > max_pages * p) len = max_pages * p;
            if (len < 0) len = 0;
            int32_t *row = keep_idx + ((size_t)r * H_kv + h) * budget;
            for (int i = 0; i < budget; ++i) row[i] = -1;
            tok_t *cand = (tok_t *)malloc(sizeof(tok_t) * (size_t)(len > 0 ? len : 1));
            int *kept = (int *)malloc(sizeof(int) * (size_t)(budget > 0 ? budget : 1));
            int n_cand = 0, n_kept = 0;
            for (int j = 0; j < len; ++j) {
                const int pid = page_table[(size_t)r * max_pages + j / p];
                if (pid < 0) continue;                       /* not in A */
                if (j >= len - w) {                          /* protected recent window */
                    kept[n_kept++] = j;
                } else {
                    cand[n_cand].u = u[((size_t)pid * H_kv + h) * p + j % p];
                    cand[n_cand].pos = j;
                    ++n_cand;
                }
            }
            int k = budget - n_kept;
            if (k > n_cand) k = n_cand;
            qsort(cand, (size_t)n_cand, sizeof(tok_t), tok_cmp);
            for (int i = 0; i < k; ++i) kept[n_kept++] = cand[i].pos;
            qsort(kept, (size_t)n_kept, sizeof(int), int_cmp);
            for (int i = 0; i < n_kept; ++i) row[i] = kept[i];
            keep_cnt[(size_t)r * H_kv + h] = n_kept;
            free(cand);
            free(kept);
        }
}

/*
 * Eviction as slot compaction: for every request r and kv-head h the retained tokens
 * keep_idx[r,h,0..cnt) move, in order, to token positions 0..cnt-1 of the request: K, V and the
 * accumulated score of position i become those of position keep_idx[r,h,i] ("the scores of
 * retained entries persist").  Everything is gathered from a snapshot of the caches, so the
 * result does not depend on the order of the moves.  new_lens[r] = cnt (the heads of a request
 * must agree on it; the first ceil(cnt/p) logical pages of the request must be present).
 * Slots past the new length keep whatever they held.
 *   k_cache, v_cache [P, H_kv, p, D] bf16 bits (in/out)   u [P, H_kv, p] (in/out)
 */
void se_oracle_h2o_compact(int B, int H_kv, int D, int p, int max_pages, int P, int budget,
                           uint16_t *k_cache, uint16_t *v_cache, double *u,
                           const int32_t *page_table, const int32_t *keep_idx,
                           const int32_t *keep_cnt, int32_t *new_lens) {
    const size_t n_kv = (size_t)P * H_kv * p * D, n_u = (size_t)P * H_kv * p;
    uint16_t *k0 = (uint16_t *)malloc(n_kv * sizeof(uint16_t));
    uint16_t *v0 = (uint16_t *)malloc(n_kv * sizeof(uint16_t));
    double *u0 = (double *)malloc(n_u * sizeof(double));
    memcpy(k0, k_cache, n_kv * sizeof(uint16_t));
    memcpy(v0, v_cache, n_kv * sizeof(uint16_t));
    memcpy(u0, u, n_u * sizeof(double));
    for (int r = 0; r < B; ++r) {
        for (int h = 0; h < H_kv; ++h) {
            const int cnt = keep_cnt[(size_t)r * H_kv + h];
            const int32_t *row = keep_idx + ((size_t)r * H_kv + h) * budget;
            for (int i = 0; i < cnt; ++i) {
                const int j = row[i];
                const int pid_d = page_table[(size_t)r * max_pages + i / p];
                const int pid_s = page_table[(size_t)r * max_pages + j / p];
                if (pid_d < 0 || pid_s < 0) continue;        /* precondition violated: leave alone */
                const size_t d = ((size_t)pid_d * H_kv + h) * p + i % p;
                const size_t sidx = ((size_t)pid_s * H_kv + h) * p + j % p;
                memcpy(k_cache + d * D, k0 + sidx * D, (size_t)D * sizeof(uint16_t));
                memcpy(v_cache + d * D, v0 + sidx * D, (size_t)D * sizeof(uint16_t));
                u[d] = u0[sidx];
            }
        }
        new_lens[r] = keep_cnt[(size_t)r * H_kv];
    }
    free(k0);
    free(v0);
    free(u0);
}

/*
 * Observation-layer selector (Appendix A, "OmniKV: Selection Reuse across Layers", selection
 * equation): for request r and token j < len_r whose page is present,
 *     s[r,j] = max over all query heads a of  z_j^(a) = sm_scale * sum_c q[r,a,c] k[j,g(a),c];
 * tokens that are absent (or lie past the length) get present = 0 and s = 0.
 *   s [B, max_pages*p]   present [B, max_pages*p]
 */
void se_oracle_token_scores(int B, int H_q, int H_kv, int D, int p, int max_pages, double sm_scale,
                            const uint16_t *q, const uint16_t *k_cache, const int32_t *page_table,
                            const int32_t *seq_lens, double *s, uint8_t *present) {
    const int G = H_q / H_kv, n_max = max_pages * p;
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < B; ++r) {
        int len = seq_lens[r];
        if (len > n_max) len = n_max;
        for (int j = 0; j < n_max; ++j) {
            s[(size_t)r * n_max + j] = 0.0;
            present[(size_t)r * n_max + j] = 0;
            if (j >= len) continue;
            const int pid = page_table[(size_t)r * max_pages + j / p];
            if (pid < 0) continue;
            double best = -INFINITY;
            for (int a = 0; a < H_q; ++a) {
                const uint16_t *qa = q + ((size_t)r * H_q + a) * D;
                const uint16_t *kt = k_cache + ((((size_t)pid * H_kv + a / G) * p) + j % p) * D;
                double z = 0.0;
                for (int c = 0; c < D; ++c) z += bf16_to_f64(qa[c]) * bf16_to_f64(kt[c]);
                z *= sm_scale;
                if (z > best) best = z;
            }
            s[(size_t)r * n_max + j] = best;
            present[(size_t)r * n_max + j] = 1;
        }
    }
}

/*
 * Token selection of an observation layer: J = TopK_b(s; present tokens), equal scores to the
 * lower position; the last `recent` positions of the request (when present) are always in the
 * result and do not count against b (the paper's OmniKV settings list "selected" and "recent"
 * tokens separately).  tok_idx[r,:] = the set in ascending position, -1 padded to n_out entries;
 * theta[r] = the score of the last token taken by rank (NaN if none competes).
 */
void se_oracle_token_topk(int B, int n_max, int n_out, int budget, int recent, const double *s,
                          const uint8_t *present, const int32_t *seq_lens, int32_t *tok_idx,
                          int32_t *tok_cnt, double *theta) {
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < B; ++r) {
        int len = seq_lens[r];
        if (len > n_max) len = n_max;
        if (len < 0) len = 0;
        int32_t *row = tok_idx + (size_t)r * n_out;
        for (int i = 0; i < n_out; ++i) row[i] = -1;
        tok_t *cand = (tok_t *)malloc(sizeof(tok_t) * (size_t)(len > 0 ? len : 1));
        int *kept = (int *)malloc(sizeof(int) * (size_t)(n_out > 0 ? n_out : 1));
        int n_cand = 0, n_kept = 0;
        for (int j = 0; j < len; ++j) {
            if (!present[(size_t)r * n_max + j]) continue;
            if (j >= len - recent) {
                if (n_kept < n_out) kept[n_kept++] = j;
            } else {
                cand[n_cand].u = s[(size_t)r * n_max + j];
                cand[n_cand].pos = j;
                ++n_cand;
            }
        }
        int k = budget < n_cand ? budget : n_cand;
        if (k > n_out - n_kept) k = n_out - n_kept;
        qsort(cand, (size_t)n_cand, sizeof(tok_t), tok_cmp);
        theta[r] = k > 0 ? cand[k - 1].u : NAN;
        for (int i = 0; i < k; ++i) kept[n_kept++] = cand[i].pos;
        qsort(kept, (size_t)n_kept, sizeof(int), int_cmp);
        for (int i = 0; i < n_kept; ++i) row[i] = kept[i];
        tok_cnt[r] = n_kept;
        free(cand);
        free(kept);
    }
}

/*
 * Attention of a sparse layer that reuses an observation layer's token set (Appendix A, OmniKV
 * reuse equation): every query head a of request r attends the tokens tok_idx[r,0..tok_cnt[r])
 * of this layer's own cache,
 *     out = sum_{j in I} alpha_j v_j^(g(a)),  alpha = softmax over I of sm_scale * q_a . k_j^(g(a)),
 * lse = ln sum_{j in I} exp(z_j).  Tokens whose page is absent or that lie past the length are
 * skipped; an empty set gives out = 0, lse = -inf.
 */
void se_oracle_token_attend(int B, int H_q, int H_kv, int D, int p, int max_pages, int n_out,
                            double sm_scale, const uint16_t *q, const uint16_t *k_cache,
                            const uint16_t *v_cache, const int32_t *page_table, const int32_t *seq_lens,
                            const int32_t *tok_idx, const int32_t *tok_cnt, double *out, double *lse) {
    const int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic)
    for (int ra = 0; ra < B * H_q; ++ra) {
        const int r = ra / H_q, a = ra % H_q, h = a / G;
        const int cnt = tok_cnt[r], len = seq_lens[r];
        const uint16_t *qa = q + (size_t)ra * D;
        double *o = out + (size_t)ra * D;
        double *z = (double *)malloc(sizeof(double) * (size_t)(cnt > 0 ? cnt : 1));
        double zmax = -INFINITY;
        for (int c = 0; c < D; ++c) o[c] = 0.0;
        for (int i = 0; i < cnt; ++i) {
            const int j = tok_idx[(size_t)r * n_out + i];
            z[i] = -INFINITY;
            if (j < 0 || j >= len || j >= max_pages * p) continue;
            const int pid = page_table[(size_t)r * max_pages + j / p];
            if (pid < 0) continue;
            const uint16_t *kt = k_cache + ((((size_t)pid * H_kv + h) * p) + j % p) * D;
            double acc = 0.0;
            for (int c = 0; c < D; ++c) acc += bf16_to_f64(qa[c]) * bf16_to_f64(kt[c]);
            z[i] = acc * sm_scale;
            if (z[i] > zmax) zmax = z[i];
        }
        if (!(zmax > -INFINITY)) {
            lse[ra] = -INFINITY;
            free(z);
            continue;
        }
        double denom = 0.0;
        for (int i = 0; i < cnt; ++i)
            if (z[i] > -INFINITY) denom += exp(z[i] - zmax);
        lse[ra] = zmax + log(denom);
        for (int i = 0; i < cnt; ++i) {
            if (!(z[i] > -INFINITY)) continue;
            const int j = tok_idx[(size_t)r * n_out + i];
            const int pid = page_table[(size_t)r * max_pages + j / p];
            const uint16_t *vt = v_cache + ((((size_t)pid * H_kv + h) * p) + j % p) * D;
            const double alpha = exp(z[i] - zmax) / denom;
            for (int c = 0; c < D; ++c) o[c] += alpha * bf16_to_f64(vt[c]);
        }
        free(z);
    }
}

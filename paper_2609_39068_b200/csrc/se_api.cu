// C ABI entry points: argument validation, workspace layout, launch geometry.
#include <math.h>

#include "se_internal.h"

namespace se {

namespace {

constexpr int kAssumedSMs = 148;      // B200; launch geometry and workspace size are derived from
                                      // this constant so that se_workspace_bytes is a pure function

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int validate(const se_params *p) {
    if (!p) return SE_ERR_NULL_POINTER;
    if (p->page_size != kPage) return SE_ERR_UNSUPPORTED_SHAPE;
    if (p->D != 64 && p->D != 128) return SE_ERR_UNSUPPORTED_SHAPE;
    if (p->B < 1 || p->H_q < 1 || p->H_kv < 1) return SE_ERR_INVALID_ARG;
    if (p->B > 8192) return SE_ERR_UNSUPPORTED_SHAPE;      // the scoring kernel keeps three ints per request in shared memory
    if (p->H_q % p->H_kv != 0) return SE_ERR_INVALID_ARG;
    const int G = p->H_q / p->H_kv;
    if (G < 1 || G > 8) return SE_ERR_UNSUPPORTED_SHAPE;
    if (p->max_pages < 1 || p->max_pages > 8192 || p->num_phys_pages < 1) return SE_ERR_INVALID_ARG;
    if (p->k_max < 1 || p->k_max > 4096) return SE_ERR_INVALID_ARG;
    if (p->flags != 0) return SE_ERR_INVALID_ARG;
    if (p->sink_pages < 0 || p->recent_pages < 0 || p->sink_pages > 4096 || p->recent_pages > 4096)
        return SE_ERR_INVALID_ARG;
    if (!(p->sm_scale >= 0.f) || isinf(p->sm_scale)) return SE_ERR_INVALID_ARG;
    // index arithmetic inside the kernels uses 32-bit page counts and 64-bit byte offsets
    if ((long long)p->B * p->H_kv > (1ll << 24)) return SE_ERR_INVALID_ARG;
    if ((long long)p->B * p->max_pages > (1ll << 31) - 1) return SE_ERR_INVALID_ARG;
    if ((long long)p->num_phys_pages * p->H_kv * kPage > (1ll << 31) - 1) return SE_ERR_INVALID_ARG;
    if ((long long)p->B * p->H_kv * p->k_max > (1ll << 30)) return SE_ERR_INVALID_ARG;
    if (p->H_kv > 127) return SE_ERR_INVALID_ARG;
    return SE_OK;
}

bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

}  // namespace

int device_sm_count() { return kAssumedSMs; }

// cudaOccupancyMaxActiveClusters on a B200 for a 256-thread CTA with 217 KB of shared memory (one CTA per SM)
int max_resident_clusters(int size) {
    static const int kTable[9] = {0, 148, 74, 45, 33, 26, 22, 15, 15};
    return (size >= 1 && size <= 8) ? kTable[size] : 0;
}

int validate_params(const se_params *p) { return validate(p); }

float effective_scale(const se_params &p) {
    return p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.D);
}

int decode_warps_per_cta();

// Launch geometry of the attention step, from the shape alone.
//  - at most one pair per SM: CTA units.  A pair gets cpp = min(SMs / pairs, ceil(k_max / 8)) CTAs (a
//    warp should hold at least one page); up to 8 of them form a thread-block cluster and merge
//    their partials themselves, more are merged by the merge kernel.
//  - fewer than two pairs per SM: warp units, every pair cut into as many splits as the persistent
//    warps of the grid can take in one round; the merge kernel combines them.
//  - two to four pairs per SM: two adjacent warps per pair, merged through shared memory (decode_duo_kernel).
//  - more: warp units, one warp per pair (splitting would only add the merge).
DecodePlan make_decode_plan(const se_params &p, bool warp_units_only) {
    DecodePlan plan;
    const int warps_per_cta = decode_warps_per_cta();
    const long long pairs = (long long)p.B * p.H_kv;
    plan.cta_units = !warp_units_only && pairs <= kAssumedSMs;
    plan.merge_in_kernel = false;
    plan.duo = false;
    if (plan.cta_units) {
        long long cpp = kAssumedSMs / pairs;
        const long long useful = (p.k_max + warps_per_cta - 1) / warps_per_cta;
        if (cpp > useful) cpp = useful;
        if (cpp < 1) cpp = 1;
        // as a cluster (up to 8 CTAs) all pairs' clusters must be resident at once: a second wave doubles the time
        if (cpp <= 8)
            while (cpp > 1 && max_resident_clusters((int)cpp) < pairs) --cpp;
        plan.max_splits = (int)cpp;
        plan.pages_per_split = (int)((p.k_max + cpp - 1) / cpp);
        plan.merge_in_kernel = cpp <= 8;
        plan.grid = (int)(pairs * cpp);
        return plan;
    }
    const long long warps = (long long)kAssumedSMs * warps_per_cta;
    long long splits = warps / pairs;
    if (splits < 1 || pairs >= 2LL * kAssumedSMs) splits = 1;
    if (splits > p.k_max) splits = p.k_max;
    const int pps = (int)((p.k_max + splits - 1) / splits);
    plan.pages_per_split = pps;
    plan.max_splits = (p.k_max + pps - 1) / pps;
    const long long units = pairs * plan.max_splits;
    long long grid = units < kAssumedSMs ? units : kAssumedSMs;
    plan.grid = (int)grid;
    // two to four unsplit pairs per SM: two warps per pair (more busy warps per SM, even load)
    plan.duo = !warp_units_only && plan.max_splits == 1 && pairs <= 4LL * kAssumedSMs;
    return plan;
}

// The attention kernel selects the pages itself where a whole CTA works on one pair (cta_topk in the
// prologue: 2-5 us).  With warp units a warp would have to run the top-k alone: measured 10 us (256
// pages) to 45 us (4096 pages) per pair against 7.5 us for the top-k kernel over all 512 pairs of
// config 3, so those shapes keep the top-k kernel.
bool select_in_decode_ok(const se_params &p) { return make_decode_plan(p).cta_units; }

// The fused step needs the CTAs of a pair in one thread-block cluster (portable size: up to 8).
bool score_in_decode_ok(const se_params &p) {
    const DecodePlan plan = make_decode_plan(p);
    return plan.cta_units && plan.max_splits <= 8;
}

WorkspaceLayout make_layout(const se_params &p) {
    WorkspaceLayout L;
    const DecodePlan plan = make_decode_plan(p);
    const DecodePlan plan_w = make_decode_plan(p, true);       // observation / token layers use warp units
    const int max_splits = plan.max_splits > plan_w.max_splits ? plan.max_splits : plan_w.max_splits;
    const size_t pairs = (size_t)p.B * p.H_kv;
    const int G = p.H_q / p.H_kv;
    const int GP = next_pow2(G);
    size_t off = 0;
    L.status = off;      off += 256;
    L.pairctl = off;     off += align256(pairs * 2 * sizeof(uint32_t));
    L.has_pairctl = true;
    L.scores = off;      off += align256(pairs * (size_t)score_pitch(p) * 4);
    L.partials = off;    off += align256((size_t)p.B * p.H_q * max_splits * (p.D + 4) * 4);
    L.zbuf = off;        off += align256(pairs * (size_t)p.k_max * kPage * GP * 4);
    L.total = off;
    L.max_splits = max_splits;
    return L;
}

}  // namespace se

using namespace se;

extern "C" {

int se_version(void) { return 100; }

const char *se_strerror(int code) {
    switch (code) {
        case SE_OK: return "ok";
        case SE_ERR_INVALID_ARG: return "invalid argument";
        case SE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (need page_size 16, D in {64,128}, 1 <= H_q/H_kv <= 8, B <= 8192)";
        case SE_ERR_NULL_POINTER: return "required pointer is NULL";
        case SE_ERR_MISALIGNED: return "pointer is not 16-byte aligned";
        case SE_ERR_CUDA: return "CUDA runtime error";
        case SE_ERR_SCRATCH_TOO_SMALL: return "problem exceeds the built-in scratch array";
    }
    return "unknown error code";
}

size_t se_workspace_bytes(const se_params *p) {
    if (validate(p) != SE_OK) return 0;
    return make_layout(*p).total;
}

int se_decode_num_splits(const se_params *p) {
    if (validate(p) != SE_OK) return 0;
    return make_decode_plan(*p).max_splits;
}

int se_workspace_init(const se_params *p, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!workspace) return SE_ERR_NULL_POINTER;
    if (!aligned16(workspace)) return SE_ERR_MISALIGNED;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = cudaMemsetAsync(workspace, 0, L.scores, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_meta_update(const se_params *p, const void *k_cache, const int32_t *page_table,
                   const int32_t *seq_lens, const int32_t *first_tok, void *meta, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!k_cache || !page_table || !seq_lens || !meta) return SE_ERR_NULL_POINTER;
    if (!aligned16(k_cache) || !aligned16(meta) || !aligned16(page_table) || !aligned16(seq_lens) ||
        !aligned16(first_tok))
        return SE_ERR_MISALIGNED;
    cudaError_t e = launch_meta_update(*p, k_cache, page_table, seq_lens, first_tok, meta,
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

static int page_select_stages(const se_params *p, const void *q, const void *meta, const int32_t *page_table,
                   const int32_t *seq_lens, int32_t budget_tokens, int32_t *sel_idx,
                   int32_t *sel_cnt, void *workspace, void *stream, int stages) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!q || !meta || !page_table || !seq_lens || !sel_idx || !sel_cnt || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(meta) || !aligned16(page_table) || !aligned16(seq_lens) ||
        !aligned16(sel_idx) || !aligned16(sel_cnt) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < kPage) return SE_ERR_INVALID_ARG;
    const int k_pages = budget_tokens / kPage;
    if (k_pages + p->sink_pages + p->recent_pages > p->k_max) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_page_select(*p, q, meta, nullptr, page_table, seq_lens, k_pages, sel_idx, sel_cnt,
                                       workspace, L, static_cast<cudaStream_t>(stream), stages);
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_page_select(const se_params *p, const void *q, const void *meta, const int32_t *page_table,
                   const int32_t *seq_lens, int32_t budget_tokens, int32_t *sel_idx,
                   int32_t *sel_cnt, void *workspace, void *stream) {
    return page_select_stages(p, q, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt, workspace, stream, 3);
}

int se_page_select_scores(const se_params *p, const void *q, const void *meta, const int32_t *page_table,
                          const int32_t *seq_lens, int32_t budget_tokens, int32_t *sel_idx,
                          int32_t *sel_cnt, void *workspace, void *stream) {
    return page_select_stages(p, q, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt, workspace, stream, 1);
}

int se_page_select_topk(const se_params *p, const void *q, const void *meta, const int32_t *page_table,
                        const int32_t *seq_lens, int32_t budget_tokens, int32_t *sel_idx,
                        int32_t *sel_cnt, void *workspace, void *stream) {
    return page_select_stages(p, q, meta, page_table, seq_lens, budget_tokens, sel_idx, sel_cnt, workspace, stream, 2);
}

int se_page_select_fused(const se_params *p, const void *q, const void *k_cache, void *meta,
                         const int32_t *page_table, const int32_t *seq_lens, int32_t budget_tokens,
                         int32_t *sel_idx, int32_t *sel_cnt, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!q || !k_cache || !meta || !page_table || !seq_lens || !sel_idx || !sel_cnt || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(meta) || !aligned16(page_table) ||
        !aligned16(seq_lens) || !aligned16(sel_idx) || !aligned16(sel_cnt) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < kPage) return SE_ERR_INVALID_ARG;
    const int k_pages = budget_tokens / kPage;
    if (k_pages + p->sink_pages + p->recent_pages > p->k_max) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_page_select(*p, q, meta, k_cache, page_table, seq_lens, k_pages, sel_idx, sel_cnt,
                                       workspace, L, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

static int sparse_decode_stages(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                                const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                                const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                                uint32_t *tok_keys, void *workspace, int stages, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!q || !k_cache || !v_cache || !page_table || !seq_lens || !sel_idx || !sel_cnt || !out ||
        !lse || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(page_table) ||
        !aligned16(seq_lens) || !aligned16(sel_idx) || !aligned16(sel_cnt) || !aligned16(out) ||
        !aligned16(lse) || !aligned16(score_accum) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    const WorkspaceLayout L = make_layout(*p);
    if (tok_keys) {
        if (!aligned16(tok_keys)) return SE_ERR_MISALIGNED;
        if (cudaMemsetAsync(tok_keys, 0, (size_t)p->B * p->max_pages * kPage * sizeof(uint32_t),
                            static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return SE_ERR_CUDA;
    }
    // the kernels only read the caller's selection here (from_scores == nullptr)
    cudaError_t e = launch_sparse_decode(*p, q, k_cache, v_cache, page_table, seq_lens,
                                         const_cast<int32_t *>(sel_idx), const_cast<int32_t *>(sel_cnt), nullptr, out,
                                         lse, score_accum, tok_keys, workspace, L, stages,
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

// What se_decode_step launches for `p`: 0 = dense layer (summary update, list of all pages, attention),
// 1 = scoring kernel + attention kernel that selects in its prologue, 2 = scoring, top-k kernel, attention,
// 3 = one kernel that scores, selects and attends.
static int step_plan(const se_params &p, int k_pages) {
    if (k_pages >= p.max_pages && p.k_max >= p.max_pages) return 0;
    if (score_in_decode_ok(p)) return 3;
    return select_in_decode_ok(p) ? 1 : 2;
}

int se_decode_step(const se_params *p, const void *q, const void *k_cache, const void *v_cache, void *meta,
                   const int32_t *page_table, const int32_t *seq_lens, int32_t budget_tokens, int32_t *sel_idx,
                   int32_t *sel_cnt, float *out, float *lse, float *score_accum, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!q || !k_cache || !v_cache || !meta || !page_table || !seq_lens || !sel_idx || !sel_cnt || !out || !lse ||
        !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(meta) || !aligned16(page_table) ||
        !aligned16(seq_lens) || !aligned16(sel_idx) || !aligned16(sel_cnt) || !aligned16(out) || !aligned16(lse) ||
        !aligned16(score_accum) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < kPage) return SE_ERR_INVALID_ARG;
    const int k_pages = budget_tokens / kPage;
    if (k_pages + p->sink_pages + p->recent_pages > p->k_max) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int plan = step_plan(*p, k_pages);
    // plan 1: only the scoring kernel of the selection runs (stages = 1); the scores stay in the workspace
    cudaError_t e = cudaSuccess;
    if (plan != 3) {
        e = launch_page_select(*p, q, meta, k_cache, page_table, seq_lens, k_pages, sel_idx, sel_cnt, workspace, L, s,
                               plan == 1 ? 1 : 3);
        if (e != cudaSuccess) return SE_ERR_CUDA;
    }
    const SelectFromScores from_scores = {k_pages, plan == 3 ? meta : nullptr};
    e = launch_sparse_decode(*p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                             (plan == 1 || plan == 3) ? &from_scores : nullptr, out, lse, score_accum, nullptr,
                             workspace, L, 3, s);
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_decode_step_launches(const se_params *p, int32_t budget_tokens, int with_score_accum) {
    if (validate(p) != SE_OK || budget_tokens < kPage) return 0;
    const int plan = step_plan(*p, budget_tokens / kPage);
    const DecodePlan dp = make_decode_plan(*p);
    const bool merged = dp.max_splits == 1 || (dp.cta_units && dp.merge_in_kernel);
    // CTA units with the in-kernel merge also run the H2O epilogue in the kernel
    const bool second = (dp.cta_units && dp.merge_in_kernel) ? false : (!merged || with_score_accum);
    const int attention = 1 + (second ? 1 : 0);
    return (plan == 3 ? 0 : plan == 1 ? 1 : 2) + attention;
}

int se_sparse_decode(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                     const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                     const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                     void *workspace, void *stream) {
    return sparse_decode_stages(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
                                score_accum, nullptr, workspace, 3, stream);
}

int se_observe_decode(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                      const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                      const int32_t *sel_cnt, float *out, float *lse, uint32_t *tok_keys, void *workspace,
                      void *stream) {
    if (!tok_keys) return SE_ERR_NULL_POINTER;
    return sparse_decode_stages(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
                                nullptr, tok_keys, workspace, 3, stream);
}

int se_sparse_decode_splits(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                            const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                            const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                            void *workspace, void *stream) {
    return sparse_decode_stages(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
                                score_accum, nullptr, workspace, 1, stream);
}

int se_combine(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
               const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
               const int32_t *sel_cnt, float *out, float *lse, float *score_accum, void *workspace,
               void *stream) {
    return sparse_decode_stages(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
                                score_accum, nullptr, workspace, 2, stream);
}

int se_token_select(const se_params *p, const uint32_t *tok_keys, const int32_t *seq_lens, int32_t budget_tokens,
                    int32_t recent_tokens, int32_t *tok_idx, int32_t *tok_cnt, int32_t n_out, void *workspace,
                    void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!tok_keys || !seq_lens || !tok_idx || !tok_cnt || !workspace) return SE_ERR_NULL_POINTER;
    if (!aligned16(tok_keys) || !aligned16(seq_lens) || !aligned16(tok_idx) || !aligned16(tok_cnt) ||
        !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < 0 || recent_tokens < 0 || n_out < 1 || n_out > (1 << 20) ||
        (long long)budget_tokens + recent_tokens > n_out)
        return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_token_select(*p, tok_keys, seq_lens, budget_tokens, recent_tokens, n_out, tok_idx, tok_cnt,
                                        reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + L.status),
                                        static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_token_decode(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                    const int32_t *page_table, const int32_t *seq_lens, const int32_t *tok_idx,
                    const int32_t *tok_cnt, int32_t n_out, float *out, float *lse, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!q || !k_cache || !v_cache || !page_table || !seq_lens || !tok_idx || !tok_cnt || !out || !lse || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(page_table) ||
        !aligned16(seq_lens) || !aligned16(tok_idx) || !aligned16(tok_cnt) || !aligned16(out) || !aligned16(lse) ||
        !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    // the workspace is sized for k_max units per pair; a unit here is a 16-token tile
    if (n_out < 1 || (n_out + kPage - 1) / kPage > p->k_max) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_token_decode(*p, q, k_cache, v_cache, page_table, seq_lens, tok_idx, tok_cnt, n_out, out,
                                        lse, workspace, L, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_h2o_retain(const se_params *p, const float *score_accum, const int32_t *page_table,
                  const int32_t *seq_lens, int32_t budget_tokens, int32_t recent_tokens, int32_t *keep_idx,
                  int32_t *keep_cnt, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!score_accum || !page_table || !seq_lens || !keep_idx || !keep_cnt || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(score_accum) || !aligned16(page_table) || !aligned16(seq_lens) || !aligned16(keep_idx) ||
        !aligned16(keep_cnt) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < 1 || budget_tokens > (1 << 20) || recent_tokens < 0) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_h2o_retain(*p, score_accum, page_table, seq_lens, budget_tokens, recent_tokens, keep_idx,
                                      keep_cnt, reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + L.status),
                                      static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_h2o_compact(const se_params *p, void *k_cache, void *v_cache, float *score_accum,
                   const int32_t *page_table, const int32_t *keep_idx, const int32_t *keep_cnt,
                   int32_t budget_tokens, int32_t *new_seq_lens, void *workspace, void *stream) {
    int rc = validate(p);
    if (rc != SE_OK) return rc;
    if (!k_cache || !v_cache || !score_accum || !page_table || !keep_idx || !keep_cnt || !new_seq_lens || !workspace)
        return SE_ERR_NULL_POINTER;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(score_accum) || !aligned16(page_table) ||
        !aligned16(keep_idx) || !aligned16(keep_cnt) || !aligned16(new_seq_lens) || !aligned16(workspace))
        return SE_ERR_MISALIGNED;
    if (budget_tokens < 1 || budget_tokens > (1 << 20)) return SE_ERR_INVALID_ARG;
    const WorkspaceLayout L = make_layout(*p);
    cudaError_t e = launch_h2o_compact(*p, k_cache, v_cache, score_accum, page_table, keep_idx, keep_cnt, budget_tokens,
                                       new_seq_lens,
                                       reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + L.status),
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

int se_last_device_status(void *workspace, void *stream, int32_t *host_out) {
    if (!workspace || !host_out) return SE_ERR_NULL_POINTER;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(workspace, 0, sizeof word, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return SE_ERR_CUDA;
    *host_out = (int32_t)word;
    return SE_OK;
}

}  // extern "C"

// Host-side declarations shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "se_device.cuh"

namespace se {

// Decode-kernel geometry that both the workspace sizing and the launcher derive from
// the problem shape alone (never from device data).
struct DecodePlan {
    int grid;               // CTAs
    bool cta_units;         // true: decode_cta_kernel, one CTA per (pair, CTA-split); false: decode_kernel,
                            // one warp per (pair, split)
    int pages_per_split;    // warp units: selected pages of one split
    int max_splits;         // splits per pair (warp units: ceil(k_max / pages_per_split); CTA units: CTAs per pair)
    bool merge_in_kernel;   // CTA units: the CTAs of a pair are a cluster and merge their partials themselves
    bool duo;               // warp units, unsplit pairs: decode_duo_kernel - two adjacent warps share a pair
};

// the selection comes from the page scores in the workspace: the attention kernel runs the top-k
struct SelectFromScores {
    int k_pages;
    void *meta;              // != nullptr: fused step - the attention kernel also scores the pages (CTA units whose
                             // CTAs per pair fit a thread-block cluster), refreshing the newest page's summary
};

int  device_sm_count();
// Thread-block clusters of `size` CTAs that can be resident at once when a CTA fills an SM (B200: the CTAs
// of a cluster sit in one GPC, so not every size packs all 148 SMs).
int  max_resident_clusters(int size);
int  validate_params(const se_params *p);        // SE_OK or the SE_ERR_* code every entry point returns for a bad `p`
DecodePlan make_decode_plan(const se_params &p, bool warp_units_only = false);
// whether the attention kernel's own top-k covers the shape (otherwise the top-k kernel runs)
bool select_in_decode_ok(const se_params &p);
// whether the attention kernel can also score the pages (one launch for the whole step)
bool score_in_decode_ok(const se_params &p);
WorkspaceLayout make_layout(const se_params &p);
float effective_scale(const se_params &p);
// floats per (request, kv-head) row of the score scratch: rows start 16-byte aligned
inline int score_pitch(const se_params &p) { return (p.max_pages + 3) & ~3; }

// kernels' launchers; each returns a cudaError_t from the launch
cudaError_t launch_meta_update(const se_params &p, const void *k_cache, const int32_t *page_table,
                               const int32_t *seq_lens, const int32_t *first_tok, void *meta,
                               cudaStream_t stream);

// k_cache != nullptr: the summary of the page holding each request's newest token is recomputed
// from K inside the scoring kernel (and written back to `meta`) instead of being read
cudaError_t launch_page_select(const se_params &p, const void *q, const void *meta, const void *k_cache,
                               const int32_t *page_table, const int32_t *seq_lens, int k_pages,
                               int32_t *sel_idx, int32_t *sel_cnt, void *workspace,
                               const WorkspaceLayout &L, cudaStream_t stream, int stages = 3);
// stages: 1 = scoring kernel only (scores stay in the workspace), 2 = top-k kernel only, 3 = both

// from_scores != nullptr: sel_idx / sel_cnt are OUTPUTS - the attention kernel selects the pages
// itself from the scores a scoring kernel left in the workspace
cudaError_t launch_sparse_decode(const se_params &p, const void *q, const void *k_cache,
                                 const void *v_cache, const int32_t *page_table,
                                 const int32_t *seq_lens, int32_t *sel_idx, int32_t *sel_cnt,
                                 const SelectFromScores *from_scores, float *out, float *lse, float *score_accum,
                                 uint32_t *tok_keys, void *workspace, const WorkspaceLayout &L, int stages,
                                 cudaStream_t stream);
// tok_keys != nullptr: observation layer - [B, 16*max_pages] order-preserving integer images of
// max-over-heads logits, merged with atomic max (the caller zeroes the array first)
// H2O retention (retained positions per (request, kv-head)) and eviction (in-place compaction)
cudaError_t launch_h2o_retain(const se_params &p, const float *score_accum, const int32_t *page_table,
                              const int32_t *seq_lens, int budget, int recent, int32_t *keep_idx,
                              int32_t *keep_cnt, uint32_t *status, cudaStream_t stream);
cudaError_t launch_h2o_compact(const se_params &p, void *k_cache, void *v_cache, float *score_accum,
                               const int32_t *page_table, const int32_t *keep_idx, const int32_t *keep_cnt,
                               int budget, int32_t *new_lens, uint32_t *status, cudaStream_t stream);
cudaError_t launch_token_select(const se_params &p, const uint32_t *tok_keys, const int32_t *seq_lens, int budget,
                                int recent, int n_out, int32_t *tok_idx, int32_t *tok_cnt, uint32_t *status,
                                cudaStream_t stream);
cudaError_t launch_token_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                                const int32_t *page_table, const int32_t *seq_lens, const int32_t *tok_idx,
                                const int32_t *tok_cnt, int n_out, float *out, float *lse, void *workspace,
                                const WorkspaceLayout &L, cudaStream_t stream);
// stages: 1 = split attention kernel, 2 = combine kernel (merge + H2O epilogue), 3 = both

}  // namespace se

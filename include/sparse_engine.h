/*
 * sparse_engine.h — C ABI of the B200 (sm_100a) sparse decode-attention library.
 *
 * The library implements the data-parallel hot path of one decode step of a sparse-first
 * inference engine: Quest-style page summaries, query-dependent page scoring, per
 * (request, kv-head) top-k page selection under a token budget, and split-K paged
 * attention over the selected pages with a log-sum-exp merge and an optional H2O
 * accumulated-attention epilogue.  (Paper: Appendix A "Detailed Background and
 * Notations"; Appendix B "Lifecycle Implementation Details" for the attention-view
 * payload and the CUDA-graph buffer rules the interface follows.)
 *
 * General rules, valid for every entry point
 * ------------------------------------------
 *  - All data pointers are DEVICE pointers to contiguous buffers owned by the caller;
 *    `const se_params*` and `int32_t* host_out` are HOST pointers.  The library never
 *    allocates, frees or keeps a pointer after the call returns.
 *  - `stream` is a `cudaStream_t` passed as `void*` (NULL = the default stream).  Calls
 *    enqueue work on it and return; only `se_last_device_status` synchronises.
 *  - Return value: SE_OK (0) or a negative SE_ERR_* code.  Arguments are validated on
 *    the host before anything is launched: a call that fails validation enqueues nothing.
 *    SE_ERR_CUDA (a launch or a runtime call failed after validation) may leave part of
 *    the call's work - a memset, an earlier kernel of a multi-kernel call - enqueued.
 *  - Shapes: B requests, H_q query heads, H_kv kv-heads, G = H_q / H_kv in 1..8,
 *    D in {64, 128}, page size 16 tokens.  Query head a reads kv-head a / G
 *    (Appendix A, "MHA, MQA, and GQA").
 *  - Layouts (row-major, innermost last):
 *      q           [B, H_q, D]               bf16
 *      k_cache     [P_phys, H_kv, 16, D]     bf16   (one page of one kv-head is contiguous)
 *      v_cache     [P_phys, H_kv, 16, D]     bf16
 *      meta        [P_phys, H_kv, 2, D]      bf16   row 0 = channel-wise min, row 1 = max;
 *                                                   indexed by PHYSICAL page, so aliased
 *                                                   prefix pages share their summaries
 *      page_table  [B, max_pages]            int32  physical page of logical page b, or -1
 *                                                   if that page has no physical KV
 *                                                   (Appendix A, "Logical Positions and
 *                                                   Physical Blocks"; 0-based here)
 *      seq_lens    [B]                       int32  logical tokens of the request, the
 *                                                   current one included; 0 = padding slot
 *      sel_idx     [B, H_kv, k_max]          int32  selected LOGICAL pages, ascending,
 *                                                   padded with -1
 *      sel_cnt     [B, H_kv]                 int32  number of valid entries per row
 *      out         [B, H_q, D]               fp32
 *      lse         [B, H_q]                  fp32   natural-log log-sum-exp of the logits
 *      score_accum [P_phys, H_kv, 16]        fp32   H2O statistic per token slot
 *  - All pointers must be 16-byte aligned.
 *  - Inputs must be finite; behaviour with NaN/Inf in q, K, V is unspecified.
 *  - Physical page ids outside [0, num_phys_pages) and selected pages outside the
 *    request are never dereferenced: the access is skipped and a bit is set in the
 *    device status word (see se_last_device_status).  se_meta_update is the one exception:
 *    it takes no workspace, hence has no status word, and skips such a page id silently.
 */
#ifndef SPARSE_ENGINE_H_
#define SPARSE_ENGINE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SE_OK                       0
#define SE_ERR_INVALID_ARG         -1   /* a size or value is out of range                 */
#define SE_ERR_UNSUPPORTED_SHAPE   -2   /* D, G, page_size or B not supported              */
#define SE_ERR_NULL_POINTER        -3   /* a required pointer is NULL                      */
#define SE_ERR_MISALIGNED          -4   /* a pointer is not 16-byte aligned                */
#define SE_ERR_CUDA                -5   /* a CUDA runtime call failed (launch, attribute)  */
#define SE_ERR_SCRATCH_TOO_SMALL   -6   /* problem exceeds the built-in scratch (se_page_select_static) */

/* bits of the device status word */
#define SE_DEV_BAD_PAGE_ID          1u  /* page_table entry >= num_phys_pages              */
#define SE_DEV_BAD_SELECTION        2u  /* sel_idx entry outside the request / sel_cnt > k_max */
#define SE_DEV_WAIT_TIMEOUT         4u  /* a bounded wait (200 ms) on an asynchronous copy gave up */

typedef struct se_params {
    int32_t B;               /* requests in the batch, 1..8192                              */
    int32_t H_q;             /* query heads                                                 */
    int32_t H_kv;            /* kv heads; H_q % H_kv == 0, H_q / H_kv in 1..8               */
    int32_t D;               /* head dimension, 64 or 128                                   */
    int32_t page_size;       /* must be 16                                                  */
    int32_t max_pages;       /* row stride of page_table, >= ceil(max seq_len / 16), <= 8192
                                (contexts up to 131072 tokens)                              */
    int32_t num_phys_pages;  /* P_phys, pages in k_cache / v_cache / meta / score_accum     */
    int32_t k_max;           /* row stride of sel_idx, >= floor(budget / 16), 1..4096       */
    float   sm_scale;        /* logit scale; 0 selects 1/sqrt(D)                            */
    uint32_t flags;          /* reserved, must be 0                                         */
    int32_t sink_pages;      /* se_page_select: the first this many logical pages of every  */
    int32_t recent_pages;    /* request and the last this many are always selected, outside
                                the budget (0 = pure top-k); see se_page_select             */
} se_params;

/* Library version (major*10000 + minor*100 + patch). */
int se_version(void);

/* Text for an SE_ERR_* code (static storage, never NULL). */
const char *se_strerror(int code);

/*
 * Bytes of device scratch the calls below need for `p` (host, pure; 0 if `p` is invalid).
 * The caller allocates that many bytes (256-byte aligned), runs se_workspace_init once,
 * and may then reuse the buffer for any number of calls with the same `p`.  Calls that
 * share a workspace must be ordered on the device (same stream or explicit dependencies).
 * Calls whose `p` differ only in k_max, sm_scale, flags, sink_pages or recent_pages (the layers
 * of one model step, some dense and some sparse) may share one workspace sized and
 * initialised for the `p` with the largest se_workspace_bytes: the control block at its head
 * depends on B and H_kv only.
 */
size_t se_workspace_bytes(const se_params *p);

/*
 * Split-K geometry se_sparse_decode uses for `p` (host, pure): the number of splits every
 * (request, kv-head) pair is cut into (warps, or whole CTAs when there is at most one pair per
 * SM), or 0 if `p` is invalid.  1 means every pair is attended by one worker, which writes out/lse
 * itself.  Informational: lets a caller size its own tooling.
 */
int se_decode_num_splits(const se_params *p);

/*
 * Zeroes the control block (status word, work-queue and per-pair arrival counters) at the
 * head of the workspace.  Required once after allocation; the kernels leave the counters at
 * zero when they finish, so it need not be repeated - except after a call that reported
 * SE_DEV_WAIT_TIMEOUT, which may have left counters behind: run it again then.
 */
int se_workspace_init(const se_params *p, void *workspace, void *stream);

/*
 * Quest page summaries (Appendix A, "Quest: Query-Dependent Page Selection", summary
 * equation): for every kv-head h and channel c of a page,
 *     meta[pid,h,0,c] = min_t K[pid,h,t,c],   meta[pid,h,1,c] = max_t K[pid,h,t,c]
 * over the tokens t of the page that lie below the request's length.
 *   first_tok == NULL : incremental mode - recompute only the summary of the page that
 *                       holds each request's newest token (same passage, the sentence after
 *                       the score equation); run after the token's K is in k_cache.
 *   first_tok != NULL : [B] int32; recompute every page of request r from the page
 *                       holding token first_tok[r] on (0 = rebuild all, e.g. after prefill).
 * Pages with page_table == -1, pages whose id is outside [0, num_phys_pages) (skipped without a
 * report: this call has no status word) and pages no request refers to are left untouched.  The
 * result is exact (a min/max of bf16 values); -0 orders below +0.  Requests that alias
 * the same physical page write identical values.  A request's partially filled last
 * page must not be aliased by another request of a different length.
 */
int se_meta_update(const se_params *p, const void *k_cache, const int32_t *page_table,
                   const int32_t *seq_lens, const int32_t *first_tok, void *meta,
                   void *stream);

/*
 * Page scoring and top-k selection (Appendix A, Quest score equation and the TopK entry
 * of the notation table).  For request r, kv-head h and every logical page b < ceil(len_r/16)
 * that has a physical page:
 *     S[a,b] = sm_scale * sum_c max(q[r,a,c]*min[b,c], q[r,a,c]*max[b,c])   (fp32)
 *     P[h,b] = max over the query heads a of group h of S[a,b]
 * and sel_idx[r,h,:] receives the k_eff = min(floor(budget_tokens/16), #present pages)
 * pages with the largest P (equal scores: lower page first), in ascending page order,
 * padded with -1; sel_cnt[r,h] = k_eff.  A request with seq_len 0 or no present page
 * gets sel_cnt 0.  Never writes q, meta or the page table.  Uses the workspace for the fp32
 * scores.
 * Forced pages (the paper's Quest settings read "sink" and "recent" tokens in addition to the
 * selected budget, Appendix C "Experimental Settings"): with p->sink_pages = s and
 * p->recent_pages = t, the logical pages 0..s-1 and ceil(len_r/16)-t..ceil(len_r/16)-1 of every
 * request are always part of the result when they are present; they are not candidates of the
 * top-k and do not count against the budget, so sel_cnt can reach floor(budget/16) + s + t.
 * Requires 16 <= budget_tokens and floor(budget_tokens/16) + s + t <= k_max.
 * Dense-layer mode: when budget_tokens / 16 >= max_pages and k_max >= max_pages the budget covers
 * any context of this shape, nothing is scored (meta is not read) and every present page is
 * selected.
 */
int se_page_select(const se_params *p, const void *q, const void *meta,
                   const int32_t *page_table, const int32_t *seq_lens,
                   int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                   void *workspace, void *stream);

/*
 * se_meta_update(first_tok = NULL) and se_page_select in one call (the decode step's usual order:
 * the newest token's K is in the cache, its page's summary is stale).  The scoring kernel recomputes
 * the summary of the page that holds each request's newest token from k_cache - for every
 * kv-head, over the tokens below the length, exactly as se_meta_update does - uses it for the
 * score and writes it to `meta`; every other page's summary is read from `meta` as usual.  Saves
 * the separate kernel of se_meta_update.  Results (meta, sel_idx, sel_cnt) are identical to the
 * two calls made one after the other.  (Appendix A, Quest summary and score equations and the
 * incremental-update sentence after them; TopK entry of the notation table.)
 */
int se_page_select_fused(const se_params *p, const void *q, const void *k_cache, void *meta,
                         const int32_t *page_table, const int32_t *seq_lens,
                         int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                         void *workspace, void *stream);

/*
 * Attention over the tokens of the selected pages (Appendix A, "Attention over Selected
 * Positions"): for every query head a of request r, with T the tokens (below len_r) of
 * the pages sel_idx[r, a/G, 0..sel_cnt),
 *     z_j = sm_scale * q.k_j,  alpha_j = exp(z_j)/sum_{u in T} exp(z_u),
 *     out = sum_j alpha_j v_j,  lse = ln sum_{u in T} exp(z_u).
 * The selected pages are split over several workers (split-K) whose partial results are
 * merged through their running maxima by a second kernel; out/lse do not depend on the split
 * beyond fp32 rounding.  An empty T gives out = 0 and lse = -inf.
 * score_accum != NULL additionally applies the H2O update (Appendix A, H2O accumulated
 * score equation) to every attended token slot:
 *     score_accum[pid,h,t] += sum over the query heads a of group h of alpha_{a,(pid,t)} .
 * With score_accum the physical pages selected by different requests must be distinct
 * (no aliased prefix), otherwise the read-modify-write races.  Never writes q, K, V,
 * the page table or the selection.
 */
int se_sparse_decode(const se_params *p, const void *q, const void *k_cache,
                     const void *v_cache, const int32_t *page_table,
                     const int32_t *seq_lens, const int32_t *sel_idx,
                     const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                     void *workspace, void *stream);

/*
 * One decode step of a layer in one call: se_meta_update(first_tok = NULL), se_page_select and
 * se_sparse_decode, with the same results (meta, sel_idx, sel_cnt, out, lse, score_accum; Appendix A,
 * Quest summary and score equations, TopK, selected-attention and H2O equations; the fused per-pair
 * form follows Appendix B's requirement that a step replays as a fixed sequence of launches over
 * stable buffers).  The call picks the launch plan from the shape alone:
 *   - a sparse layer (budget_tokens/16 < max_pages) with at most one (request, kv-head) pair per SM
 *     and at most 8 CTAs per pair: ONE kernel.  The CTAs of a pair form a thread-block cluster; each
 *     scores its share of the pair's pages (refreshing the summary of the request's newest page),
 *     after a cluster barrier every CTA selects the pair's pages from the score row (top-k in shared
 *     memory), attends its share of them with eight warps, merges the warps' partials through shared
 *     memory, and the CTA that arrives last merges the CTAs' partials and applies the H2O update.
 *   - a sparse layer with more pairs: the scoring kernel, the top-k kernel, the attention kernel
 *     (one warp per pair or per split of a pair), and the merge kernel where pairs are split or
 *     score_accum is given.
 *   - a dense layer (budget_tokens/16 >= max_pages and k_max >= max_pages, e.g. the first layers of
 *     a model whose remaining layers are sparse): summary update, list of all present pages,
 *     attention.
 * sel_idx / sel_cnt are outputs here; the fp32 page scores are left in the workspace as
 * se_page_select_scores leaves them.  se_decode_step_launches tells how many kernels a step
 * launches for `p` (host, pure; 0 if the arguments are invalid).
 */
int se_decode_step(const se_params *p, const void *q, const void *k_cache, const void *v_cache, void *meta,
                   const int32_t *page_table, const int32_t *seq_lens, int32_t budget_tokens,
                   int32_t *sel_idx, int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                   void *workspace, void *stream);
int se_decode_step_launches(const se_params *p, int32_t budget_tokens, int with_score_accum);

/*
 * se_page_select without any caller-provided scratch.  (The paper has no counterpart: this entry
 * point exists for the way some hosts have to call the library.)
 *
 * Who needs it: code that may not allocate device memory at the point where it runs the
 * selection - a serving loop whose memory pool is fully handed out before the first request, a
 * plug-in that receives tensors but no allocator, a real-time thread in which cudaMalloc's
 * implicit synchronisation is not acceptable.  Those callers cannot size and allocate the
 * workspace that se_page_select wants, so here the only scratch the selection needs - the fp32
 * page scores - lives in a fixed array inside the library: SE_STATIC_SCRATCH_BYTES of device
 * memory that every GPU which loads the library holds until the process exits.
 *
 * Same arguments, same results (bit for bit) as se_page_select, except:
 *   - no workspace argument; nothing is allocated or freed, by this call or on its behalf;
 *   - dev_status (nullable, 4-byte aligned DEVICE pointer, caller-owned) receives the status
 *     word of this call (SE_DEV_* bits) once the stream reaches that point;
 *   - the shape is limited by the array: 256 + 4*B*H_kv*P bytes, P = max_pages rounded up to a
 *     multiple of 4 (score rows start 16-byte aligned), must not exceed SE_STATIC_SCRATCH_BYTES, otherwise SE_ERR_SCRATCH_TOO_SMALL is returned and nothing is
 *     enqueued.
 * The first call on a device looks up the array's device address (a set-up step, done once per
 * device with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps the contents of the last call: the call
 * clears the status word itself, and the scores are rewritten before they are read.  Two calls
 * whose kernels may overlap on the GPU (different streams without an ordering between them)
 * race on the array; order them.
 */
#define SE_STATIC_SCRATCH_BYTES (4u * 1024u * 1024u)
int se_page_select_static(const se_params *p, const void *q, const void *meta,
                          const int32_t *page_table, const int32_t *seq_lens,
                          int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                          int32_t *dev_status, void *stream);

/*
 * The two halves of se_page_select as separate calls (same arguments, same workspace): first
 * se_page_select_scores - the scoring kernel; the fp32 page scores stay in the workspace - then
 * se_page_select_topk - the top-k kernel, which reads them.  One after the other on the same stream
 * they are exactly se_page_select (except in dense-layer mode, which only the single call takes);
 * they exist so that a profiler or a benchmark can time the two kernels apart, and so that a test can
 * read the scores: after se_page_select_scores the workspace holds, from byte offset
 * 256 + (8*B*H_kv rounded up to a multiple of 256) on, B*H_kv rows of P floats, P = max_pages rounded up to a multiple of 4; element b of row r*H_kv + h is
 * the fp32 score of logical page b of request r for kv-head h, -inf where the page is absent;
 * elements from ceil(len_r/16) on are not written.
 */
int se_page_select_scores(const se_params *p, const void *q, const void *meta,
                          const int32_t *page_table, const int32_t *seq_lens,
                          int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                          void *workspace, void *stream);
int se_page_select_topk(const se_params *p, const void *q, const void *meta,
                        const int32_t *page_table, const int32_t *seq_lens,
                        int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                        void *workspace, void *stream);

/*
 * The two halves of se_sparse_decode as separate calls (same arguments, same workspace): first
 * se_sparse_decode_splits - the split-K attention kernel; pairs held by a single worker get their
 * final out/lse, the others leave partial results in the workspace - then se_combine - the
 * log-sum-exp merge of the partials and, with score_accum, the H2O epilogue.  Calling one after
 * the other on the same stream is exactly se_sparse_decode; they exist so that a profiler or a
 * benchmark can time the two kernels apart.
 */
int se_sparse_decode_splits(const se_params *p, const void *q, const void *k_cache,
                            const void *v_cache, const int32_t *page_table,
                            const int32_t *seq_lens, const int32_t *sel_idx,
                            const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                            void *workspace, void *stream);
int se_combine(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
               const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
               const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
               void *workspace, void *stream);

/*
 * Selection reuse across layers (Appendix A, "OmniKV: Selection Reuse across Layers").
 *
 * se_observe_decode - an observation (filter) layer: se_sparse_decode (normally with every page
 * selected, i.e. full attention) that also leaves, for every attended token j of request r,
 *     s[r,j] = max over all query heads a of the logit z_j^(a) = sm_scale * q_a . k_j      (selection eq.)
 * in tok_keys ([B, 16*max_pages] uint32, device) as the order-preserving integer image of the fp32
 * score: key = bits ^ 0xffffffff for negative values, bits | 0x80000000 otherwise; 0 = token not
 * attended.  The call zeroes tok_keys itself (a memset on `stream`) before the kernel runs.
 *
 * se_token_select - J = TopK_b(s; attended tokens) per request, equal scores to the lower
 * position, plus the attended tokens among the request's last recent_tokens positions, which are
 * always kept and do not count against b (the paper's OmniKV settings list "selected" and
 * "recent" tokens separately).  tok_idx[r,:] ([B, n_out] int32) receives the set in ascending
 * position, -1 padded; tok_cnt[r] its size.  budget_tokens + recent_tokens <= n_out <= 2^20.
 *
 * se_token_decode - a sparse layer that reuses the set (reuse equation): every query head of
 * request r attends the tokens tok_idx[r, 0..tok_cnt[r]) of THIS layer's k_cache / v_cache,
 *     out = sum_j alpha_j v_j,   alpha = softmax over the set,   lse = ln sum_j exp(z_j).
 * Tokens whose page is absent are skipped; tokens outside [0, seq_lens[r]) are skipped and
 * reported through the status word; an empty set gives out = 0, lse = -inf.  Needs
 * ceil(n_out / 16) <= k_max (the workspace holds one partial per 16-token tile group).
 * All three are asynchronous on `stream` and allocate nothing.
 */
int se_observe_decode(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                      const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                      const int32_t *sel_cnt, float *out, float *lse, uint32_t *tok_keys,
                      void *workspace, void *stream);
int se_token_select(const se_params *p, const uint32_t *tok_keys, const int32_t *seq_lens,
                    int32_t budget_tokens, int32_t recent_tokens, int32_t *tok_idx, int32_t *tok_cnt,
                    int32_t n_out, void *workspace, void *stream);
int se_token_decode(const se_params *p, const void *q, const void *k_cache, const void *v_cache,
                    const int32_t *page_table, const int32_t *seq_lens, const int32_t *tok_idx,
                    const int32_t *tok_cnt, int32_t n_out, float *out, float *lse, void *workspace,
                    void *stream);

/*
 * H2O retained set (Appendix A, "H2O: Accumulated Scores and Online Eviction", retention
 * equation).  For request r (seq_lens[r] tokens; token j lives in slot j % 16 of logical page
 * j / 16) and kv-head h, with u = score_accum as maintained by se_sparse_decode:
 *     A = the request's tokens whose logical page is present (page_table >= 0),
 *     W = the tokens of A among the last min(recent_tokens, budget_tokens) positions,
 *     R = W  u  TopK_{budget - |W|}(u; A \ W)       (all of A \ W if it has fewer members);
 * equal scores go to the lower position.  keep_idx[r,h,:] ([B, H_kv, budget_tokens] int32, device)
 * receives R in ascending token position, padded with -1; keep_cnt[r,h] = |R| (the same for every
 * head of a request).  Reads score_accum, page_table, seq_lens; writes only keep_idx / keep_cnt.
 * 1 <= budget_tokens <= 2^20.  Scores must be finite.  Asynchronous on `stream`,
 * allocates nothing; bad page ids are reported through the workspace's status word.
 */
int se_h2o_retain(const se_params *p, const float *score_accum, const int32_t *page_table,
                  const int32_t *seq_lens, int32_t budget_tokens, int32_t recent_tokens,
                  int32_t *keep_idx, int32_t *keep_cnt, void *workspace, void *stream);

/*
 * H2O eviction as slot compaction of the retained set (Appendix A, H2O retention equation and the
 * sentence after it: what is not retained leaves the cache, retained tokens keep their accumulated
 * scores): for every (request, kv-head) the retained tokens keep_idx[r,h,0..keep_cnt) move, in
 * order, to token positions 0..keep_cnt-1 of the request - K row, V row and accumulated score of
 * position i become those of position keep_idx[r,h,i] - and new_seq_lens[r] = keep_cnt[r,0].
 * In place: k_cache, v_cache and score_accum are read and written; slots past the new length keep
 * what they held.  Requirements: keep_idx rows ascending (as se_h2o_retain writes them), the heads
 * of a request agree on keep_cnt, the request's first ceil(cnt/16) logical pages are present, and
 * no physical page is shared between requests.  Page summaries (meta) of the touched pages are
 * stale afterwards: rebuild them with se_meta_update(first_tok = 0) before the next page
 * selection.  budget_tokens is the row length of keep_idx.  Invalid rows (a source before its
 * destination, absent or out-of-range pages) are skipped and reported through the status word.
 */
int se_h2o_compact(const se_params *p, void *k_cache, void *v_cache, float *score_accum,
                   const int32_t *page_table, const int32_t *keep_idx, const int32_t *keep_cnt,
                   int32_t budget_tokens, int32_t *new_seq_lens, void *workspace, void *stream);

/*
 * Measurement aid (no counterpart in the paper): a read-only gather with the access pattern and
 * pipeline shape of the library's kernels and no arithmetic, to find what the memory system of a
 * given GPU allows for that pattern.  Piece i of the list lives at base + piece_idx[i]*piece_bytes
 * (with base1 != NULL the odd lanes of a batch read from base1 instead: K and V pages of the same
 * list).  Every warp of a persistent grid (148 * ctas_per_sm CTAs of warps_per_cta warps) keeps
 * stages_per_warp batches of pieces_per_stage (<= 32) pieces in flight in shared memory, fetched by
 * bulk asynchronous copies.  piece_bytes is a multiple of 16; the shared memory needed
 * (warps * stages * pieces * piece_bytes) must fit 227 KB.  All pointers are DEVICE pointers, 16-byte
 * aligned; the call is asynchronous on `stream`.  Shapes used by the benchmark: summaries 512 B x 16 x 2
 * stages x 4 warps x 3 CTAs/SM; pages 4096 B x 2 x 5 x 4 x 1; token rows 256 B x 32 x 5 x 4 x 1.
 */
int se_probe_gather(const void *base0, const void *base1, const int32_t *piece_idx, int64_t n_pieces,
                    int32_t piece_bytes, int32_t pieces_per_stage, int32_t stages_per_warp,
                    int32_t warps_per_cta, int32_t ctas_per_sm, void *stream);

/*
 * Copies the device status word (an OR of SE_DEV_* bits, 0 = clean) to *host_out and
 * clears it.  Synchronises `stream`; the only entry point that does.
 */
int se_last_device_status(void *workspace, void *stream, int32_t *host_out);

#ifdef __cplusplus
}
#endif
#endif /* SPARSE_ENGINE_H_ */

// H2O retention and eviction (Appendix A, "H2O: Accumulated Scores and Online Eviction",
// retention equation): the consumer of the accumulated scores that se_sparse_decode maintains.
//
// retain_kernel       (H2O form) one CTA per (request, kv-head).  The request's token scores are read page
//                     row by page row (one thread = one 64-byte row of 16 scores, a chunk = one
//                     row per thread) as order-preserving integer keys; tokens of the protected
//                     recent window are kept unconditionally and do not compete.  Pass 1 finds
//                     the span [kmin, kmax] and the number of competitors, pass 2 fills a
//                     2048-bin histogram over the span and locates the bin holding the k-th
//                     largest key (a crowded bin gets another level over its own span), a few
//                     keys are ranked by brute force, equal keys go to the lower position.  The
//                     last pass writes the retained positions in ascending order with a running
//                     CTA prefix sum.  The scores are re-read in every pass (they are at most a
//                     few hundred KB per pair and stay in L2).
// h2o_compact_kernel  one CTA per (request, kv-head): the retained tokens' K rows, V rows and
//                     scores move to positions 0..cnt-1.  A destination never lies behind its
//                     source (keep_idx is ascending), so the move is done in place, 128 tokens
//                     per iteration: every warp reads the 16 source rows of one destination page
//                     into registers, the CTA synchronises, then the rows are written.  Pages
//                     whose 16 tokens stay where they are are skipped.
#include "se_internal.h"

namespace se {

namespace {

constexpr int kRetBins = 2048;
constexpr int kRetBinBits = 11;
constexpr int kRetList = 32;

// kTok == false: H2O retention.  One CTA per (request, kv-head); scores are score_accum rows found
//   through the page table; the window counts against the budget; rows of `budget` entries.
// kTok == true: token selection of an observation layer (Appendix A, OmniKV selection equation).
//   One CTA per request; scores are the integer keys an observation layer left in tok_keys
//   [B, 16*max_pages] (0 = token not attended); the recent window is kept on top of the budget;
//   rows of n_out entries.
template <int kRetThreads, bool kTok>
__global__ void __launch_bounds__(kRetThreads)
retain_kernel(const float *__restrict__ score_accum, const uint32_t *__restrict__ tok_keys,
              const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens, int H_kv,
              int max_pages, int P_phys, int budget, int recent, int n_out, int32_t *__restrict__ keep_idx,
              int32_t *__restrict__ keep_cnt, uint32_t *status) {
    constexpr int NW = kRetThreads / 32;
    constexpr int BPT = kRetBins / kRetThreads;
    __shared__ __align__(16) int s_hist[kRetBins];     // bin = (kmax' - key) >> shift: prefix = better keys
    __shared__ int s_tot[2][32];
    __shared__ int s_red[4][NW];
    __shared__ int s_res[6];
    __shared__ uint32_t s_lkey[kRetList];
    __shared__ int s_lpos[kRetList];
    __shared__ int s_ln;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair = blockIdx.x;
    const int r = kTok ? pair : pair / H_kv, h = kTok ? 0 : pair - r * H_kv;
    int n = seq_lens[r];
    if (n > max_pages * kPage) n = max_pages * kPage;
    if (n < 0) n = 0;
    const int w = kTok ? min(recent, n_out) : min(recent, budget);
    const int wstart = n - w;                           // positions >= wstart form the protected window
    const int npages = (n + kPage - 1) / kPage;
    const int chunks = (npages + kRetThreads - 1) / kRetThreads;
    int32_t *out = keep_idx + (size_t)pair * n_out;
    int scan_par = 0;

    // keys of this thread's page row in chunk c; bit t of winmask = token t is in the window
    auto load_row = [&](int c, uint32_t (&keys)[kPage], uint32_t &winmask) {
        const int b = c * kRetThreads + tid;
        winmask = 0;
        if (kTok) {
            if (b >= npages) {
#pragma unroll
                for (int t = 0; t < kPage; ++t) keys[t] = kKeyAbsent;
                return;
            }
            const uint4 *src = reinterpret_cast<const uint4 *>(tok_keys + (size_t)r * max_pages * kPage + b * kPage);
#pragma unroll
            for (int t4 = 0; t4 < kPage / 4; ++t4) {
                const uint4 v = __ldg(src + t4);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t = 4 * t4 + e;
                    const int pos = b * kPage + t;
                    const uint32_t x = e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w;
                    uint32_t key = kKeyAbsent;
                    if (pos < n && x != 0u) {                // 0 = the observation layer did not attend it
                        if (pos >= wstart) winmask |= 1u << t;
                        else key = max(x, kKeyAbsent + 1u);
                    }
                    keys[t] = key;
                }
            }
            return;
        }
        int pid = -1;
        if (b < npages) pid = __ldg(page_table + (size_t)r * max_pages + b);
        if (pid >= P_phys) {
            atomicOr(status, SE_DEV_BAD_PAGE_ID);
            pid = -1;
        }
        if (pid < 0) {
#pragma unroll
            for (int t = 0; t < kPage; ++t) keys[t] = kKeyAbsent;
            return;
        }
        const float4 *src = reinterpret_cast<const float4 *>(score_accum + ((size_t)pid * H_kv + h) * kPage);
#pragma unroll
        for (int t4 = 0; t4 < kPage / 4; ++t4) {
            const float4 v = __ldg(src + t4);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = 4 * t4 + e;
                const int pos = b * kPage + t;
                const float x = e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w;
                uint32_t key = kKeyAbsent;
                if (pos < n) {
                    if (pos >= wstart) winmask |= 1u << t;
                    else key = max(f32_key(x), kKeyAbsent + 1u);     // a stored -inf still competes
                }
                keys[t] = key;
            }
        }
    };

    // ---- pass 1: competitors, window tokens, span of the competitors' keys
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    int present = 0, nwin = 0;
    for (int c = 0; c < chunks; ++c) {
        uint32_t keys[kPage], winmask;
        load_row(c, keys, winmask);
        nwin += __popc(winmask);
#pragma unroll
        for (int t = 0; t < kPage; ++t) {
            const bool ok = keys[t] != kKeyAbsent;
            present += ok;
            kmin = ok ? min(kmin, keys[t]) : kmin;
            kmax = max(kmax, keys[t]);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        present += __shfl_xor_sync(kFull, present, o);
        nwin += __shfl_xor_sync(kFull, nwin, o);
        kmin = min(kmin, __shfl_xor_sync(kFull, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(kFull, kmax, o));
    }
    if (lane == 0) {
        s_red[0][warp] = present;
        s_red[1][warp] = (int)kmin;
        s_red[2][warp] = (int)kmax;
        s_red[3][warp] = nwin;
    }
#pragma unroll
    for (int e = 0; e < BPT; ++e) s_hist[tid * BPT + e] = 0;
    if (tid == 0) s_ln = 0;
    __syncthreads();
    present = 0;
    nwin = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) {
        present += s_red[0][i];
        nwin += s_red[3][i];
        kmin = min(kmin, (uint32_t)s_red[1][i]);
        kmax = max(kmax, (uint32_t)s_red[2][i]);
    }
    nwin = min(nwin, n_out);
    const int k_take = kTok ? min(min(budget, n_out - nwin), present)     // competitors that stay
                            : min(budget - nwin, present);
    const int total = k_take + nwin;
    if (total == 0) {
        for (int i = tid; i < n_out; i += kRetThreads) out[i] = -1;
        if (tid == 0) keep_cnt[pair] = 0;
        return;
    }

    // ---- threshold (T_key, T_pos): a competitor stays <=> key > T_key || (key == T_key && pos <= T_pos)
    uint32_t T_key = 0xffffffffu;
    int T_pos = -1;                          // k_take == 0: only the window stays
    int remaining = k_take;
    bool ties = false;
    if (k_take > 0 && k_take == present) {
        T_key = kmin;
        T_pos = 0x7fffffff;
    } else if (k_take > 0 && kmin == kmax) {
        T_key = kmin;
        ties = true;
    } else if (k_take > 0) {
        uint32_t hi = kmax;                              // the current span is (hi - span, hi]
        uint32_t span = kmax - kmin + 1u;
        int width = 32 - __clz(kmax - kmin);
        for (int level = 0;; ++level) {
            const int sh = width > kRetBinBits ? width - kRetBinBits : 0;
            if (level > 0) {
#pragma unroll
                for (int e = 0; e < BPT; ++e) s_hist[tid * BPT + e] = 0;
                __syncthreads();
            }
            for (int c = 0; c < chunks; ++c) {
                uint32_t keys[kPage], winmask;
                load_row(c, keys, winmask);
#pragma unroll
                for (int t = 0; t < kPage; ++t) {
                    const uint32_t d = hi - keys[t];
                    if (d < span) atomicAdd(&s_hist[d >> sh], 1);
                }
            }
            __syncthreads();
            int loc[BPT], sum = 0;
#pragma unroll
            for (int e = 0; e < BPT; ++e) {
                loc[e] = s_hist[tid * BPT + e];
                sum += loc[e];
            }
            const int excl = cta_excl_scan<NW>(sum, s_tot[scan_par], lane, warp);
            scan_par ^= 1;
            if (excl < remaining && remaining <= excl + sum) {
                int run = excl;
#pragma unroll
                for (int e = 0; e < BPT; ++e) {
                    if (run < remaining && remaining <= run + loc[e]) {
                        s_res[0] = tid * BPT + e;
                        s_res[1] = run;
                        s_res[2] = loc[e];
                    }
                    run += loc[e];
                }
            }
            __syncthreads();
            const int bin = s_res[0];
            const int inbin = s_res[2];
            remaining -= s_res[1];
            hi -= (uint32_t)bin << sh;                   // the bin is (hi - 2^sh, hi]
            span = 1u << sh;
            width = sh;
            T_key = hi - (span - 1u);                    // lowest key of the bin
            if (inbin == remaining) {                    // the whole bin stays
                T_pos = 0x7fffffff;
                break;
            }
            if (sh == 0) {                               // the bin is one key value
                ties = true;
                break;
            }
            if (inbin <= kRetList) {
                for (int c = 0; c < chunks; ++c) {
                    uint32_t keys[kPage], winmask;
                    load_row(c, keys, winmask);
#pragma unroll
                    for (int t = 0; t < kPage; ++t) {
                        if (hi - keys[t] < span) {
                            const int pos = atomicAdd(&s_ln, 1);
                            if (pos < kRetList) {
                                s_lkey[pos] = keys[t];
                                s_lpos[pos] = (c * kRetThreads + tid) * kPage + t;
                            }
                        }
                    }
                }
                __syncthreads();
                const bool has = lane < inbin;
                const uint32_t mk = has ? s_lkey[lane] : 0u;
                const int mp = has ? s_lpos[lane] : 0x7fffffff;
                int rank = 0;
                for (int i = 0; i < inbin; ++i) {
                    const uint32_t ok = __shfl_sync(kFull, mk, i);
                    const int op = __shfl_sync(kFull, mp, i);
                    rank += (ok > mk) || (ok == mk && op < mp);
                }
                const int owner = __ffs(__ballot_sync(kFull, has && rank == remaining - 1)) - 1;
                T_key = __shfl_sync(kFull, mk, owner);
                T_pos = __shfl_sync(kFull, mp, owner);
                break;
            }
        }
    }
    if (ties) {
        // T_pos = the remaining-th position, in order, among the competitors equal to T_key
        int seen = 0;                                    // equal keys in earlier chunks
        T_pos = 0x7fffffff;
        for (int c = 0; c < chunks; ++c) {
            uint32_t keys[kPage], winmask;
            load_row(c, keys, winmask);
            int cnt = 0;
#pragma unroll
            for (int t = 0; t < kPage; ++t) cnt += keys[t] == T_key;
            const int excl = seen + cta_excl_scan<NW>(cnt, s_tot[scan_par], lane, warp);
            scan_par ^= 1;
            if (excl < remaining && remaining <= excl + cnt) {
                int run = excl;
#pragma unroll
                for (int t = 0; t < kPage; ++t) {
                    if (keys[t] == T_key) {
                        ++run;
                        if (run == remaining) s_res[5] = (c * kRetThreads + tid) * kPage + t;
                    }
                }
            }
            // equal keys of the whole chunk: the last thread's inclusive count
            if (tid == kRetThreads - 1) s_res[4] = excl + cnt;
            __syncthreads();
            seen = s_res[4];
            if (seen >= remaining) {
                T_pos = s_res[5];
                break;
            }
            __syncthreads();                             // s_res[4] is rewritten by the next chunk
        }
    }

    // ---- ordered output
    int base_out = 0;
    for (int c = 0; c < chunks; ++c) {
        uint32_t keys[kPage], winmask;
        load_row(c, keys, winmask);
        const int pos0 = (c * kRetThreads + tid) * kPage;
        uint32_t takemask = winmask;
        const int tT = T_pos - pos0;
#pragma unroll
        for (int t = 0; t < kPage; ++t) {
            const bool take = keys[t] > T_key || (keys[t] == T_key && t <= tT);
            takemask |= (uint32_t)take << t;
        }
        const int cnt = __popc(takemask);
        int pos = base_out + cta_excl_scan<NW>(cnt, s_tot[scan_par], lane, warp);
        if (tid == kRetThreads - 1) s_res[3] = pos + cnt;            // retained so far
#pragma unroll
        for (int t = 0; t < kPage; ++t) {
            if ((takemask >> t) & 1u) {
                if (pos < n_out) out[pos] = pos0 + t;
                ++pos;
            }
        }
        __syncthreads();
        base_out = s_res[3];
        scan_par ^= 1;
    }
    for (int i = total + tid; i < n_out; i += kRetThreads) out[i] = -1;
    if (tid == 0) keep_cnt[pair] = total;
}

constexpr int kCmpWarps = 8;

template <int D>
__global__ void __launch_bounds__(kCmpWarps * 32)
h2o_compact_kernel(uint4 *k_cache, uint4 *v_cache, float *score_accum, const int32_t *__restrict__ page_table,
                   const int32_t *__restrict__ keep_idx, const int32_t *__restrict__ keep_cnt,
                   int32_t *__restrict__ new_lens, int H_kv, int max_pages, int P_phys, int budget,
                   uint32_t *status) {
    constexpr int LPR = D / 8;               // lanes per token row (16-byte pieces)
    constexpr int RPI = 32 / LPR;            // rows per warp instruction
    constexpr int NI = kPage / RPI;          // instructions per page
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pair = blockIdx.x;
    const int r = pair / H_kv, h = pair - r * H_kv;
    int cnt = keep_cnt[pair];
    if (cnt > budget) cnt = budget;
    if (cnt < 0) cnt = 0;
    const int32_t *row = keep_idx + (size_t)pair * budget;
    const int32_t *pt = page_table + (size_t)r * max_pages;
    const int rg = lane / LPR, lr = lane % LPR;
    if (h == 0 && threadIdx.x == 0) new_lens[r] = cnt;

    for (int i0 = 0; i0 < cnt; i0 += kCmpWarps * kPage) {
        const int d0 = i0 + warp * kPage;                  // first destination position of this warp
        // lane t < 16: source position and physical page of destination d0 + t
        int src = -1, spid = -1;
        if (lane < kPage && d0 + lane < cnt) {
            src = __ldg(row + d0 + lane);
            if (src < d0 + lane || src >= max_pages * kPage) {
                atomicOr(status, SE_DEV_BAD_SELECTION);
                src = -1;
            } else {
                spid = __ldg(pt + src / kPage);
                if (spid < 0 || spid >= P_phys) {
                    atomicOr(status, spid < 0 ? SE_DEV_BAD_SELECTION : SE_DEV_BAD_PAGE_ID);
                    src = -1;
                }
            }
        }
        int dpid = (d0 < cnt) ? __ldg(pt + d0 / kPage) : -1;
        if (dpid >= P_phys || (d0 < cnt && dpid < 0)) {
            if (lane == 0) atomicOr(status, dpid < 0 ? SE_DEV_BAD_SELECTION : SE_DEV_BAD_PAGE_ID);
            dpid = -1;
        }
        const bool moved = __any_sync(kFull, lane < kPage && src >= 0 && src != d0 + lane) && dpid >= 0;
        uint4 kr[NI], vr[NI];
        float ur = 0.f;
        if (moved) {
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int t = i * RPI + rg;
                const int s = __shfl_sync(kFull, src, t);
                const int sp = __shfl_sync(kFull, spid, t);
                if (s >= 0) {
                    const size_t off = (((size_t)sp * H_kv + h) * kPage + s % kPage) * LPR + lr;
                    kr[i] = k_cache[off];
                    vr[i] = v_cache[off];
                }
            }
            if (lane < kPage && src >= 0) ur = score_accum[((size_t)spid * H_kv + h) * kPage + src % kPage];
        }
        __syncthreads();            // every source of this iteration is in registers before any row is written
        if (moved) {
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int t = i * RPI + rg;
                const int s = __shfl_sync(kFull, src, t);
                if (s >= 0) {
                    const size_t off = (((size_t)dpid * H_kv + h) * kPage + t) * LPR + lr;
                    k_cache[off] = kr[i];
                    v_cache[off] = vr[i];
                }
            }
            if (lane < kPage && src >= 0) score_accum[((size_t)dpid * H_kv + h) * kPage + lane] = ur;
        }
    }
}

}  // namespace

cudaError_t launch_h2o_retain(const se_params &p, const float *score_accum, const int32_t *page_table,
                              const int32_t *seq_lens, int budget, int recent, int32_t *keep_idx,
                              int32_t *keep_cnt, uint32_t *status, cudaStream_t stream) {
    retain_kernel<256, false><<<p.B * p.H_kv, 256, 0, stream>>>(score_accum, nullptr, page_table, seq_lens, p.H_kv,
                                                                 p.max_pages, p.num_phys_pages, budget, recent,
                                                                 budget, keep_idx, keep_cnt, status);
    return cudaGetLastError();
}

cudaError_t launch_token_select(const se_params &p, const uint32_t *tok_keys, const int32_t *seq_lens, int budget,
                                int recent, int n_out, int32_t *tok_idx, int32_t *tok_cnt, uint32_t *status,
                                cudaStream_t stream) {
    retain_kernel<1024, true><<<p.B, 1024, 0, stream>>>(nullptr, tok_keys, nullptr, seq_lens, p.H_kv, p.max_pages,
                                                         p.num_phys_pages, budget, recent, n_out, tok_idx, tok_cnt,
                                                         status);
    return cudaGetLastError();
}

cudaError_t launch_h2o_compact(const se_params &p, void *k_cache, void *v_cache, float *score_accum,
                               const int32_t *page_table, const int32_t *keep_idx, const int32_t *keep_cnt,
                               int budget, int32_t *new_lens, uint32_t *status, cudaStream_t stream) {
    const int grid = p.B * p.H_kv;
    if (p.D == 128)
        h2o_compact_kernel<128><<<grid, kCmpWarps * 32, 0, stream>>>(
            (uint4 *)k_cache, (uint4 *)v_cache, score_accum, page_table, keep_idx, keep_cnt, new_lens, p.H_kv,
            p.max_pages, p.num_phys_pages, budget, status);
    else
        h2o_compact_kernel<64><<<grid, kCmpWarps * 32, 0, stream>>>(
            (uint4 *)k_cache, (uint4 *)v_cache, score_accum, page_table, keep_idx, keep_cnt, new_lens, p.H_kv,
            p.max_pages, p.num_phys_pages, budget, status);
    return cudaGetLastError();
}

}  // namespace se

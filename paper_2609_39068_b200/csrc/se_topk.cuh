// Top-k page selection (TopK entry of the paper's notation table) as a device function, shared by the
// stand-alone top-k kernel and by the attention kernel that selects in its prologue.
//
// cta_topk returns the k_eff = min(k_pages, #candidates) best candidates by (score descending, page
// ascending) plus the forced pages (first `sink` / last `recent` logical pages, when present; they
// do not compete), as an ascending list of logical pages.  Scores are compared as order-preserving
// integer keys, which live in SHARED memory: the passes below are short loops over 16-byte groups.
//
// The k_eff-th best key is located with a histogram over the span [kmin, kmax] of the candidates'
// keys (bins = (kmax' - key) >> shift, so a prefix sum counts the better keys); the bin that holds it
// usually has a handful of keys, which are ranked by brute force (a crowded bin gets another
// histogram level over its own span; a bin that is one key value goes to the tie rule).  The result
// is a threshold (key, page): taken <=> key above the threshold key, or equal to it and page <=
// threshold page.
//
// All NT threads of a CTA take part; thread t owns a run of consecutive pages (16-byte groups in slots
// of its own), so thread order is page order and one prefix sum places the taken pages.  Keys and
// histogram are accessed with explicit shared-space instructions.  Measured on a B200, 256 threads:
// 4.8 K cycles for 128 pages, 6.3 K for 2048, 8.8 K for 4060, 12.1 K for 8192 with the CTA alone on its
// SM.  (A one-warp form of the same algorithm took 7 K cycles for 264 pages and 46 K for 4060: too slow
// for the prologue of a warp-per-pair attention kernel, which therefore keeps the top-k kernel.)
#pragma once

#include "se_device.cuh"

namespace se {

constexpr int kTopkBins = 2048;
constexpr int kTopkBinBits = 11;
constexpr int kTopkList = 32;        // bins with up to this many keys are ranked by brute force

// Shared-memory scratch of one top-k besides the keys (CTA form: one per CTA; warp form: one per warp).
struct TopkScratch {
    int hist[kTopkBins];             // indexed by 2047 - digit: prefix = keys above
    int tot[4][32];
    int red[6][32];
    int res[8];
    uint32_t lkey[kTopkList];
    int lpage[kTopkList];
    int ln;
};

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// explicit shared-space accesses (32-bit shared addresses): the keys and the histogram are reached
// through pointers whose address space the compiler cannot see, and generic loads / atomics on
// shared memory cost several times more
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void red_shared_inc(uint32_t addr) {
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}

// words of shared memory cta_topk needs for the keys of up to n_max pages: every thread owns an odd
// number of 16-byte slots (no bank conflicts between the threads' 16-byte reads)
__host__ __device__ constexpr int cta_topk_key_words(int n_max, int nt) {
    return nt * 4 * (((n_max + 4 * nt - 1) / (4 * nt)) | 1);
}
constexpr int kCtaTopkMaxGroups = 8;     // 16-byte groups per thread: n <= 32 * NT pages

// ---------------------------------------------------------------------------------
// CTA form.  Returns the number of selected pages (k_eff + forced).  The ascending list goes to
// `list` (shared memory, k_max ints) when list != nullptr and to `out` (global row of k_max ints,
// padded with -1) when out != nullptr.  `keys` = cta_topk_key_words(n, NT) words of shared memory,
// 16-byte aligned.  Thread t owns the pages [t*4*r4, (t+1)*4*r4), r4 = ceil(n / (4*NT)) <= 8: it
// loads them itself, keeps them in its own slots and is the only one to read them.
// Every thread of the CTA must call it; it ends with a __syncthreads(), after which `list` is complete.
// ---------------------------------------------------------------------------------
template <int NT>
__device__ __forceinline__ int cta_topk(const float *row, int n, int k_pages, int k_max, int sink_pages,
                                        int recent_pages, uint32_t *keys, TopkScratch &S, int *list, int32_t *out) {
    constexpr int NW = NT / 32;
    constexpr int BPT = kTopkBins / NT;                // histogram bins per thread
    static_assert(NW <= 32 && BPT >= 1, "top-k shape");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (n > 4 * kCtaTopkMaxGroups * NT) n = 4 * kCtaTopkMaxGroups * NT;      // cannot happen: max_pages <= 8192
    const int n4 = (n + 3) >> 2;
    const int r4 = (n4 + NT - 1) / NT;                 // 16-byte groups per thread
    const int base = tid * 4 * r4;                     // first page of this thread
    const int my4 = max(0, min(r4, n4 - tid * r4));    // groups of this thread that hold pages
    const uint32_t kbase = smem_u32(keys) + (uint32_t)tid * (r4 | 1) * 16;
    const uint32_t hbase = smem_u32(S.hist);

    // ---- load, scores -> keys, candidates, span.  The loads are coalesced (group g = j*NT + tid, all of
    // a thread's loads in flight at once); each group is then stored into the slots of its owner.
    // Besides the span the threads reduce a lower bound of the threshold: `holders` threads loaded at
    // least one candidate, so at least `holders` keys are >= tau = the smallest of those threads'
    // maxima, and with k_eff <= holders the k_eff-th best key cannot lie below tau.
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    int present = 0, forced = 0;
    {
        const float4 *row4 = reinterpret_cast<const float4 *>(row);
        const uint32_t kb0 = smem_u32(keys);
        float4 v[kCtaTopkMaxGroups];
#pragma unroll
        for (int j = 0; j < kCtaTopkMaxGroups; ++j)
            if (j < r4 && j * NT + tid < n4) v[j] = __ldcg(row4 + j * NT + tid);
#pragma unroll
        for (int j = 0; j < kCtaTopkMaxGroups; ++j) {
            const int g = j * NT + tid;
            if (j < r4 && g < n4) {
                uint32_t k[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int page = 4 * g + c;
                    const float ev = c == 0 ? v[j].x : c == 1 ? v[j].y : c == 2 ? v[j].z : v[j].w;
                    uint32_t key = page < n ? f32_key(ev) : kKeyAbsent;      // absent pages score -inf = kKeyAbsent
                    if (key != kKeyAbsent) {
                        if (page < sink_pages || page >= n - recent_pages) {
                            key = kKeyForced;
                            ++forced;
                        } else {
                            ++present;
                            kmin = min(kmin, key);
                            kmax = max(kmax, key);
                        }
                    }
                    k[c] = key;
                }
                const int owner = g / r4;
                sts128(kb0 + (uint32_t)(owner * (r4 | 1) + (g - owner * r4)) * 16, make_uint4(k[0], k[1], k[2], k[3]));
            }
        }
    }
#pragma unroll
    for (int e = 0; e < BPT; ++e) S.hist[tid * BPT + e] = 0;
    if (tid == 0) S.ln = 0;
    uint32_t tau = present > 0 ? kmax : 0xffffffffu;           // this thread's best candidate
    int holders = present > 0 ? 1 : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        present += __shfl_xor_sync(kFull, present, o);
        forced += __shfl_xor_sync(kFull, forced, o);
        holders += __shfl_xor_sync(kFull, holders, o);
        kmin = min(kmin, __shfl_xor_sync(kFull, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(kFull, kmax, o));
        tau = min(tau, __shfl_xor_sync(kFull, tau, o));
    }
    if (lane == 0) {
        S.red[0][warp] = present;
        S.red[1][warp] = (int)kmin;
        S.red[2][warp] = (int)kmax;
        S.red[3][warp] = forced;
        S.red[4][warp] = holders;
        S.red[5][warp] = (int)tau;
    }
    __syncthreads();
    present = 0;
    forced = 0;
    holders = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        present += S.red[0][w];
        forced += S.red[3][w];
        holders += S.red[4][w];
        kmin = min(kmin, (uint32_t)S.red[1][w]);
        kmax = max(kmax, (uint32_t)S.red[2][w]);
        tau = min(tau, (uint32_t)S.red[5][w]);
    }
    forced = min(forced, k_max);
    const int k_eff = min(min(k_pages, k_max - forced), present);      // candidates to take
    const int total = k_eff + forced;
    if (total == 0) {
        if (out != nullptr)
            for (int i = tid; i < k_max; i += NT) out[i] = -1;
        __syncthreads();
        return 0;
    }

    // ---- threshold (T_key, T_page): taken <=> key > T_key || (key == T_key && page <= T_page)
    uint32_t T_key = 0xffffffffu;
    int T_page = -1;                         // k_eff == 0: nothing competes
    int remaining = k_eff;                   // still to take among the keys inside the current span
    bool ties = false;                       // the keys equal to T_key are taken in page order
    if (k_eff > 0 && k_eff == present) {     // every candidate is wanted
        T_key = kmin;
        T_page = 0x7fffffff;
    } else if (k_eff > 0 && kmin == kmax) {  // all equal
        T_key = kmin;
        ties = true;
    } else if (k_eff > 0) {
        // keys below tau cannot be taken (see above): they stay out of the histogram, and the bins get finer
        uint32_t lo = k_eff <= holders ? tau : kmin;     // the current span is [lo, lo + span)
        uint32_t span = kmax - lo + 1u;
        int width = 32 - __clz(kmax - lo);               // span <= 2^width
        for (int level = 0;; ++level) {
            const int sh = width > kTopkBinBits ? width - kTopkBinBits : 0;
            if (level > 0) {
#pragma unroll
                for (int e = 0; e < BPT; ++e) S.hist[tid * BPT + e] = 0;
                __syncthreads();
            }
            // keys spread over the bins nearly evenly, so shared-memory atomics rarely collide
            for (int j = 0; j < my4; ++j) {
                const uint4 v = lds128(kbase + j * 16);
                const uint32_t k[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t d = k[c] - lo;
                    if (d < span) red_shared_inc(hbase + 4 * ((kTopkBins - 1) - (int)(d >> sh)));
                }
            }
            __syncthreads();
            // the bin b with  #(keys in bins above b) < remaining <= #(keys in bins above or in b)
            int loc[BPT], sum = 0;
#pragma unroll
            for (int e = 0; e < BPT; ++e) {
                loc[e] = S.hist[tid * BPT + e];
                sum += loc[e];
            }
            const int excl = cta_excl_scan<NW>(sum, S.tot[level & 1], lane, warp);
            if (excl < remaining && remaining <= excl + sum) {
                int acc = excl;
#pragma unroll
                for (int e = 0; e < BPT; ++e) {
                    if (acc < remaining && remaining <= acc + loc[e]) {
                        S.res[0] = tid * BPT + e;
                        S.res[1] = acc;
                        S.res[2] = loc[e];
                    }
                    acc += loc[e];
                }
            }
            __syncthreads();
            const int digit = (kTopkBins - 1) - S.res[0];
            const int inbin = S.res[2];
            remaining -= S.res[1];
            lo += (uint32_t)digit << sh;
            span = 1u << sh;
            width = sh;
            T_key = lo;
            if (inbin == remaining) {            // the whole bin is taken
                T_page = 0x7fffffff;
                break;
            }
            if (sh == 0) {                       // the bin is one key value: ties
                ties = true;
                break;
            }
            if (inbin <= kTopkList) {
                // few keys left: collect them and rank each against the others
                for (int j = 0; j < my4; ++j) {
                    const uint4 v = lds128(kbase + j * 16);
                    const uint32_t k[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if (k[c] - lo < span) {
                            const int pos = atomicAdd(&S.ln, 1);
                            if (pos < kTopkList) {
                                S.lkey[pos] = k[c];
                                S.lpage[pos] = base + 4 * j + c;
                            }
                        }
                    }
                }
                __syncthreads();
                // every warp ranks the (at most 32) collected keys on its own: lane i holds entry i,
                // the entry that `remaining - 1` others precede is the threshold
                const bool has = lane < inbin;
                const uint32_t mk = has ? S.lkey[lane] : 0u;
                const int mp = has ? S.lpage[lane] : 0x7fffffff;
                int rank = 0;
                for (int i = 0; i < inbin; ++i) {
                    const uint32_t ok = __shfl_sync(kFull, mk, i);
                    const int op = __shfl_sync(kFull, mp, i);
                    rank += (ok > mk) || (ok == mk && op < mp);
                }
                const int owner = __ffs(__ballot_sync(kFull, has && rank == remaining - 1)) - 1;
                T_key = __shfl_sync(kFull, mk, owner);
                T_page = __shfl_sync(kFull, mp, owner);
                break;
            }
        }
    }
    if (ties) {
        // T_page = the remaining-th page, in page order, among the keys equal to T_key
        int cnt = 0;
        for (int j = 0; j < my4; ++j) {
            const uint4 v = lds128(kbase + j * 16);
            cnt += (v.x == T_key) + (v.y == T_key) + (v.z == T_key) + (v.w == T_key);
        }
        const int excl = cta_excl_scan<NW>(cnt, S.tot[2], lane, warp);
        if (excl < remaining && remaining <= excl + cnt) {
            int acc = excl;
            for (int j = 0; j < my4; ++j) {
                const uint4 v = lds128(kbase + j * 16);
                const uint32_t k[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (k[c] == T_key && ++acc == remaining) S.res[5] = base + 4 * j + c;
            }
        }
        __syncthreads();
        T_page = S.res[5];
    }

    // ---- ordered compaction: mark (bit 4j + c of `taken` = page base + 4j + c), prefix, write
    uint32_t taken = 0u;
    for (int j = 0; j < my4; ++j) {
        const uint4 v = lds128(kbase + j * 16);
        const uint32_t k[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (k[c] == kKeyForced || k[c] > T_key || (k[c] == T_key && base + 4 * j + c <= T_page))
                taken |= 1u << (4 * j + c);
    }
    int pos = cta_excl_scan<NW>(__popc(taken), S.tot[3], lane, warp);
    // the list is put together in shared memory (the caller's list, or the histogram, which is no longer
    // needed, when it is large enough) and written out with coalesced stores, padding included
    int *stage = list != nullptr ? list : (k_max <= kTopkBins ? S.hist : nullptr);
    while (taken != 0u) {
        const int page = base + __ffs(taken) - 1;
        taken &= taken - 1u;
        if (pos < k_max) {
            if (stage != nullptr) stage[pos] = page;
            else out[pos] = page;
        }
        ++pos;
    }
    __syncthreads();
    if (out != nullptr) {
        if (stage != nullptr) {
            for (int i = tid; i < k_max; i += NT) out[i] = i < total ? stage[i] : -1;
        } else {
            for (int i = total + tid; i < k_max; i += NT) out[i] = -1;
        }
    }
    return total;
}

}  // namespace se

// Page scoring and top-k page selection (Appendix A, Quest score equation; TopK entry of
// the notation table).
//
// score_kernel   streams the page summaries.  Every warp is an autonomous pipeline: it owns
//                two shared-memory buffers of 16 page summaries, fills them with 1-D bulk
//                asynchronous copies (one per page and head, completion on an mbarrier) and
//                computes on one buffer while the other is in flight.  The bound
//                    sum_c max(q_c*m_c, q_c*M_c)
//                equals  sum_c (q_c^- * m_c + q_c^+ * M_c)  with q^+ = max(q,0), q^- = min(q,0)
//                (M >= m, so one product is the maximum and the other factor is zero).  That
//                is a dense [16 pages x 2D] . [2D x G] contraction per batch: the summaries
//                are the row-major A operand straight out of shared memory (rows padded by
//                16 bytes so that ldmatrix is bank-conflict free), (q^-|q^+) of the G query
//                heads is the B operand held in registers, products of bf16 values are exact
//                and accumulate in fp32.  An earlier plain-FMA version of this kernel was
//                issue-bound at 64 % of the copy bandwidth (57 warp instructions per page
//                summary); this one needs 3.
// topk_kernel    one CTA per (request, kv-head) runs cta_topk (se_topk.cuh): order-preserving integer
//                keys in thread-private 16-byte groups of shared memory, threshold by a histogram
//                over the keys' span plus a brute-force ranking of the crossing bin, then a
//                page-ordered compaction, so equal scores go to the lower page and the list is
//                ascending.  The attention kernel of small shapes calls the same function itself.
#include <atomic>

#include "se_internal.h"
#include "se_topk.cuh"

namespace se {

namespace {

// Fault injection for the test of the bounded waits (a second build of the library, -DSE_TEST_SHORT_TX,
// never the product): every batch announces 16 bytes more than its copies deliver, so the wait for it
// runs out, the kernel reports SE_DEV_WAIT_TIMEOUT and returns.
#ifdef SE_TEST_SHORT_TX
constexpr uint32_t kTestExtraTx = 16;
#else
constexpr uint32_t kTestExtraTx = 0;
#endif

constexpr int kScoreWarps = 4;     // warps per CTA of the score kernel
constexpr int kPB = 16;            // pages per warp batch (one m16 tile)
constexpr int kNBU = 4;            // batches per work unit  -> 64 pages per (pair, unit)
constexpr int kUnitPages = kPB * kNBU;

template <int D>
struct ScoreCfg {
    static constexpr int PHB = 2 * D * 2;               // bytes of one page summary (min row, max row)
    static constexpr int PITCH = PHB + 16;              // shared-memory pitch of a summary
    static constexpr int KSTEPS = 2 * D / 16;           // k16 steps over (min row | max row)
    static constexpr int BUF = kPB * PITCH;             // one buffer
};

struct Batch {
    int r, h, b0, n_r;      // request, kv-head, first logical page, pages of the request
    int unit;               // ticket this batch was handed out under (-1 = end of stream)
    int left;               // batches of this hand-out after this one
};

// Ticket t -> (request, head, first page).  Units of 64 pages are numbered request-major, head
// fastest; prefix[r] = units before request r.  The first `big` tickets are whole units; the
// tickets after that are single 16-page batches of the remaining units, so that the warps run
// dry within one batch of each other instead of one unit.
__device__ __forceinline__ bool decode_unit(int t, int total_units, int big, const int *prefix, const int *npages,
                                            int B, int H_kv, Batch &d) {
    int u = t, k0 = 0, kend = kNBU;
    if (t >= big) {
        u = big + (t - big) / kNBU;
        k0 = (t - big) % kNBU;
        kend = k0 + 1;
    }
    if (u >= total_units) {
        d.unit = -1;
        return false;
    }
    int lo = 0, hi = B - 1;
    while (lo < hi) {                       // largest r with prefix[r] <= u
        int mid = (lo + hi + 1) >> 1;
        if (prefix[mid] <= u) lo = mid; else hi = mid - 1;
    }
    const int local = u - prefix[lo];
    d.r = lo;
    d.h = local % H_kv;
    d.b0 = (local / H_kv) * kUnitPages + k0 * kPB;
    d.n_r = npages[lo];
    d.unit = t;
    d.left = kend - k0 - 1;
    return true;
}

template <int D>
__global__ void __launch_bounds__(kScoreWarps * 32)
score_kernel(const uint16_t *__restrict__ q, const uint8_t *meta, const uint8_t *__restrict__ k_cache,
             uint8_t *meta_out, const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens,
             float *__restrict__ scores, int pitch, int B, int H_kv, int G, int max_pages, int P_phys, float scale,
             uint32_t *status) {
    using C = ScoreCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // layout: [buffers: warps*2*BUF] [mbarriers: warps*2*8] [prefix: B+1 ints] [npages: B ints] [lens: B ints]
    uint8_t *bufs = smem_raw;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)kScoreWarps * 2 * C::BUF);
    int *prefix = reinterpret_cast<int *>(bars + kScoreWarps * 2);
    int *npages = prefix + (B + 1);
    int *lens = npages + B;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H_q = H_kv * G;

    // ---- per-CTA: units before each request (exclusive prefix over ceil(n_r/64)*H_kv).  All threads
    // fetch the lengths (one round trip for up to 128 requests), one warp scans them.
    for (int r = threadIdx.x; r < B; r += kScoreWarps * 32) {
        const int len = __ldg(seq_lens + r);
        int n = len > 0 ? (len + kPage - 1) / kPage : 0;
        if (n > max_pages) n = max_pages;
        npages[r] = n;
        lens[r] = len;
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0;
        for (int base = 0; base < B; base += 32) {
            const int r = base + lane;
            const int n = r < B ? npages[r] : 0;
            int u = ((n + kUnitPages - 1) / kUnitPages) * H_kv;
            int inc = u;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(kFull, inc, o);
                if (lane >= o) inc += t;
            }
            if (r < B) prefix[r] = run + inc - u;
            run += __shfl_sync(kFull, inc, 31);
        }
        if (lane == 0) prefix[B] = run;
    }
    if (lane == 0) {
        mbar_init(smem_u32(&bars[warp * 2 + 0]), 1);
        mbar_init(smem_u32(&bars[warp * 2 + 1]), 1);
        mbar_fence_init();
    }
    __syncthreads();
    const int total_units = prefix[B];
    const int big_units = total_units - total_units / 8;      // the last eighth goes out batch by batch
    const int gw = blockIdx.x * kScoreWarps + warp;
    const int tw = gridDim.x * kScoreWarps;

    uint8_t *my_buf = bufs + (size_t)warp * 2 * C::BUF;
    const uint32_t buf0 = smem_u32(my_buf);
    const uint32_t bar0 = smem_u32(&bars[warp * 2]);
    const int gid = lane >> 2, tid4 = lane & 3;      // fragment coordinates of this lane

    // B operand: column n = query head n of the group (zero for n >= G); rows k < D carry q^-
    // (they meet the min row), rows k >= D carry q^+ (they meet the max row).
    uint32_t bfrag[C::KSTEPS][2];
    uint32_t qraw[D / 16][2];                // raw q pairs of the pair whose batch was issued last

    auto load_qraw = [&](const Batch &d) {
        const uint16_t *src = q + ((size_t)d.r * H_q + d.h * G + (gid < G ? gid : 0)) * D + 2 * tid4;
#pragma unroll
        for (int s = 0; s < D / 16; ++s) {
            const uint32_t w0 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16));
            const uint32_t w1 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16 + 8));
            qraw[s][0] = gid < G ? w0 : 0u;
            qraw[s][1] = gid < G ? w1 : 0u;
        }
    };
    auto convert_q = [&]() {
#pragma unroll
        for (int s = 0; s < D / 16; ++s)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t w = qraw[s][j];
                const uint32_t negmask = ((w >> 15) & 0x00010001u) * 0xffffu;   // all-ones per negative half
                bfrag[s][j] = w & negmask;                   // q^-  (min row part)
                bfrag[D / 16 + s][j] = w & ~negmask;         // q^+  (max row part)
            }
    };

    // Work units are handed out dynamically: a warp's first unit is its own index, every further
    // one comes from a global counter.  The counter is bumped when a unit is entered and the
    // answer is only needed when that unit ends (four batches later), so the round trip is hidden.
    // SMs that get less memory bandwidth simply fetch fewer units.
    uint32_t *queue = status + 16, *done = status + 17;
    int pending_unit = 0;                        // valid in lane 0
    auto request_unit = [&]() {
        if (lane == 0) pending_unit = tw + (int)atomicAdd(queue, 1u);
    };
    // advance a descriptor to the next batch of this warp's stream
    auto next_batch = [&](Batch &d) {
        if (d.unit < 0) return;
        if (d.left > 0 && d.b0 + kPB < d.n_r) {
            d.left -= 1;
            d.b0 += kPB;
            return;
        }
        const int u = __shfl_sync(kFull, pending_unit, 0);
        if (decode_unit(u, total_units, big_units, prefix, npages, B, H_kv, d)) request_unit();
    };
    // every warp checks out once; the last one leaves the counters at zero for the next launch
    auto check_out = [&]() {
        if (lane == 0) {
            const uint32_t old = atomicAdd(done, 1u);
            if (old == (uint32_t)tw - 1u) {
                *queue = 0u;
                *done = 0u;
            }
        }
    };

    // page-table entries of a batch: lane j < 16 loads the entry of page b0 + j.  The value is not
    // looked at here, so the load stays in flight while the warp carries on.
    auto load_pids = [&](const Batch &d) -> int {
        int pid = -1;
        if (d.unit >= 0 && lane < kPB && d.b0 + lane < d.n_r)
            pid = __ldg(page_table + (size_t)d.r * max_pages + d.b0 + lane);
        return pid;
    };
    // Summary of one K page computed on the spot (fused summary update): the page that holds the
    // request's newest token may have changed since its summary was stored, so, when the caller
    // hands in the K cache, that one page per (request, head) is summarised from K here - written
    // to the summary array and straight into the batch buffer - instead of being copied.
    // The K page is fetched into registers when its batch is issued and reduced when the batch is
    // consumed, one buffer later, so the warp does not sit out the load.
    constexpr int LPR = D / 8;               // lanes per token row (16-byte pieces)
    constexpr int TPP = 32 / LPR;            // token rows per warp pass
    constexpr int KROWS = kPage / TPP;       // 16-byte pieces of the page per lane
    const int tg = lane / LPR, lr = lane % LPR;
    auto fetch_page = [&](uint4 (&w)[KROWS], int pid, int h, int nv) {
        const uint4 *kp = reinterpret_cast<const uint4 *>(k_cache) + ((size_t)pid * H_kv + h) * (kPage * D / 8);
#pragma unroll
        for (int i = 0; i < KROWS; ++i) {
            const int t = i * TPP + tg;
            w[i] = __ldg(kp + (t < nv ? t : 0) * LPR + lr);      // rows past the length repeat row 0
        }
    };
    auto reduce_page = [&](const uint4 (&w)[KROWS], int pid, int h, uint32_t dst_smem) {
        uint4 mn = w[0], mx = w[0];
#pragma unroll
        for (int i = 1; i < KROWS; ++i) {
            mn.x = bmin2(mn.x, w[i].x); mn.y = bmin2(mn.y, w[i].y); mn.z = bmin2(mn.z, w[i].z); mn.w = bmin2(mn.w, w[i].w);
            mx.x = bmax2(mx.x, w[i].x); mx.y = bmax2(mx.y, w[i].y); mx.z = bmax2(mx.z, w[i].z); mx.w = bmax2(mx.w, w[i].w);
        }
#pragma unroll
        for (int m = LPR; m < 32; m <<= 1) {
            mn.x = bmin2(mn.x, __shfl_xor_sync(kFull, mn.x, m)); mn.y = bmin2(mn.y, __shfl_xor_sync(kFull, mn.y, m));
            mn.z = bmin2(mn.z, __shfl_xor_sync(kFull, mn.z, m)); mn.w = bmin2(mn.w, __shfl_xor_sync(kFull, mn.w, m));
            mx.x = bmax2(mx.x, __shfl_xor_sync(kFull, mx.x, m)); mx.y = bmax2(mx.y, __shfl_xor_sync(kFull, mx.y, m));
            mx.z = bmax2(mx.z, __shfl_xor_sync(kFull, mx.z, m)); mx.w = bmax2(mx.w, __shfl_xor_sync(kFull, mx.w, m));
        }
        uint4 *gp = reinterpret_cast<uint4 *>(meta_out) + ((size_t)pid * H_kv + h) * (2 * D / 8);
        if (tg < 2) {
            const uint4 val = tg == 0 ? mn : mx;
            gp[tg * LPR + lr] = val;
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst_smem + (tg * LPR + lr) * 16),
                         "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
        }
    };
    bool wrote_generic = false;              // a summary was stored into a buffer with ordinary stores
    uint4 kpend[KROWS];                      // K page on its way for the batch in buffer pend_slot
    int pend_slot = -1, pend_pid = 0, pend_h = 0, pend_lane = 0;
    // issue the copies of one batch into buffer `slot`; returns this lane's physical page (or -1)
    auto issue = [&](const Batch &d, int slot, int pid) -> int {
        if (wrote_generic) {
            // ordinary stores into a buffer come before the bulk copies that refill it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            wrote_generic = false;
        }
        if (pid >= P_phys) {
            atomicOr(status, SE_DEV_BAD_PAGE_ID);
            pid = -1;
        }
        int fresh = -1;                        // lane of the page to summarise from K, if any
        if (k_cache != nullptr) {
            const int last = d.n_r - 1 - d.b0;
            if (last >= 0 && last < kPB && __shfl_sync(kFull, pid, last) >= 0) fresh = last;
        }
        const unsigned valid = __ballot_sync(kFull, pid >= 0 && lane != fresh);
        const uint32_t bar = bar0 + slot * 8;
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(valid) * C::PHB + kTestExtraTx);
        __syncwarp();
        if (pid >= 0 && lane != fresh) {
            const uint8_t *src = meta + ((size_t)pid * H_kv + d.h) * C::PHB;
            bulk_g2s(buf0 + slot * C::BUF + lane * C::PITCH, src, C::PHB, bar);
        }
        if (fresh >= 0) {
            const int fpid = __shfl_sync(kFull, pid, fresh);
            const int nv = min(kPage, lens[d.r] - (d.n_r - 1) * kPage);
            if (pend_slot < 0) {
                fetch_page(kpend, fpid, d.h, nv);
                pend_slot = slot;
                pend_pid = fpid;
                pend_h = d.h;
                pend_lane = fresh;
            } else {                          // both buffers hold a newest page (very short requests)
                uint4 w[KROWS];
                fetch_page(w, fpid, d.h, nv);
                reduce_page(w, fpid, d.h, buf0 + slot * C::BUF + fresh * C::PITCH);
                wrote_generic = true;
            }
        }
        return pid;
    };

    // Three batches are live: `cur` is computed, `nxt` is in flight, `nn` has only its page-table
    // entries on the way, so that its copies can be issued the moment a buffer frees up.
    Batch cur, nxt, nn;
    decode_unit(gw, total_units, big_units, prefix, npages, B, H_kv, cur);
    if (cur.unit < 0) {
        check_out();
        return;
    }
    request_unit();
    uint32_t phases = 0u;            // parity bit per buffer
    int slot = 0;
    nxt = cur;
    next_batch(nxt);
    int pid_cur = load_pids(cur);
    int pid_nxt = load_pids(nxt);            // both look-ups and q in flight before the first copy goes out
    load_qraw(cur);
    pid_cur = issue(cur, 0, pid_cur);
    if (nxt.unit >= 0) pid_nxt = issue(nxt, 1, pid_nxt);
    convert_q();
    if (nxt.unit >= 0 && (nxt.r != cur.r || nxt.h != cur.h)) load_qraw(nxt);
    nn = nxt;
    next_batch(nn);
    int pid_nn = load_pids(nn);
    bool failed = false;

    // ldmatrix row address of this lane inside a buffer: matrix (lane>>3) = {pages 0-7 | 8-15} x
    // {first | second 16-byte piece of the k16 step}
    const uint32_t lm_off = (uint32_t)(((lane & 7) + 8 * ((lane >> 3) & 1)) * C::PITCH + (lane >> 4) * 16);
    while (cur.unit >= 0) {
        // wait for the current buffer
        if (!mbar_wait(bar0 + slot * 8, (phases >> slot) & 1u)) {
            failed = true;
            break;
        }
        phases ^= (1u << slot);
        if (pend_slot == slot) {
            reduce_page(kpend, pend_pid, pend_h, buf0 + slot * C::BUF + pend_lane * C::PITCH);
            wrote_generic = true;
            pend_slot = -1;
            __syncwarp();
        }

        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t a_base = buf0 + slot * C::BUF + lm_off;
#pragma unroll
        for (int s = 0; s < C::KSTEPS; ++s) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(a_base + s * 32, a0, a1, a2, a3);
            mma_bf16_16816(acc, a0, a1, a2, a3, bfrag[s][0], bfrag[s][1]);
        }
        // acc[0],acc[1]: page gid, heads 2*tid4, 2*tid4+1;  acc[2],acc[3]: page gid+8, same heads
        const float ninf = -INFINITY;
        float s_lo = fmaxf(2 * tid4 < G ? acc[0] : ninf, 2 * tid4 + 1 < G ? acc[1] : ninf);
        float s_hi = fmaxf(2 * tid4 < G ? acc[2] : ninf, 2 * tid4 + 1 < G ? acc[3] : ninf);
        s_lo = fmaxf(s_lo, __shfl_xor_sync(kFull, s_lo, 1));
        s_hi = fmaxf(s_hi, __shfl_xor_sync(kFull, s_hi, 1));
        s_lo = fmaxf(s_lo, __shfl_xor_sync(kFull, s_lo, 2));
        s_hi = fmaxf(s_hi, __shfl_xor_sync(kFull, s_hi, 2));
        const int pid_lo = __shfl_sync(kFull, pid_cur, gid);
        const int pid_hi = __shfl_sync(kFull, pid_cur, gid + 8);
        if (tid4 == 0) {
            float *dst = scores + ((size_t)cur.r * H_kv + cur.h) * pitch + cur.b0;
            if (cur.b0 + gid < cur.n_r) dst[gid] = (pid_lo >= 0) ? s_lo * scale : ninf;
            if (cur.b0 + gid + 8 < cur.n_r) dst[gid + 8] = (pid_hi >= 0) ? s_hi * scale : ninf;
        }
        __syncwarp();        // every lane is done reading the buffer before it is refilled
        // refill the buffer just consumed with `nn` (its page-table entries arrived long ago)
        if (nn.unit >= 0) pid_nn = issue(nn, slot, pid_nn);
        // advance: cur <- nxt <- nn <- the batch after
        const bool pair_changed = nxt.unit >= 0 && (nxt.r != cur.r || nxt.h != cur.h);
        cur = nxt;
        pid_cur = pid_nxt;
        if (pair_changed) convert_q();                 // qraw holds q of the pair that is now current
        nxt = nn;
        pid_nxt = pid_nn;
        if (nxt.unit >= 0 && (nxt.r != cur.r || nxt.h != cur.h)) load_qraw(nxt);
        next_batch(nn);
        pid_nn = load_pids(nn);
        slot ^= 1;
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        // give the copy that may still be in flight a bounded chance to land before leaving
        mbar_wait(bar0 + (slot ^ 1) * 8, (phases >> (slot ^ 1)) & 1u);
    }
    check_out();
}

// ---------------------------------------------------------------------------------
// top-k kernel: one CTA per (request, kv-head) runs cta_topk (se_topk.cuh) on the pair's score row;
// the keys live in dynamic shared memory (cta_topk_key_words(max_pages) words).
// ---------------------------------------------------------------------------------
constexpr int kTopkThreads = 256;

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float *__restrict__ scores, int pitch, const int32_t *__restrict__ seq_lens, int H_kv,
            int max_pages, int k_pages, int k_max, int sink_pages, int recent_pages,
            int32_t *__restrict__ sel_idx, int32_t *__restrict__ sel_cnt) {
    extern __shared__ __align__(16) uint32_t topk_keys[];
    __shared__ TopkScratch S;
    const int pair = blockIdx.x;
    const int len = seq_lens[pair / H_kv];
    int n = len > 0 ? (len + kPage - 1) / kPage : 0;
    if (n > max_pages) n = max_pages;
    const int total = cta_topk<kTopkThreads>(scores + (size_t)pair * pitch, n, k_pages, k_max, sink_pages,
                                             recent_pages, topk_keys, S, nullptr, sel_idx + (size_t)pair * k_max);
    if (threadIdx.x == 0) sel_cnt[pair] = total;
}

// Dense-layer mode (budget >= context): every present page is selected, so there is nothing to
// score.  One warp per (request, kv-head) writes the present logical pages in ascending order.
__global__ void __launch_bounds__(256)
select_all_kernel(const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens, int pairs,
                  int H_kv, int max_pages, int k_max, int32_t *__restrict__ sel_idx,
                  int32_t *__restrict__ sel_cnt) {
    const int lane = threadIdx.x & 31;
    const int pair = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (pair >= pairs) return;
    const int r = pair / H_kv;
    const int len = seq_lens[r];
    int n = len > 0 ? (len + kPage - 1) / kPage : 0;
    if (n > max_pages) n = max_pages;
    int32_t *out = sel_idx + (size_t)pair * k_max;
    int count = 0;
    for (int b0 = 0; b0 < n; b0 += 32) {
        const int b = b0 + lane;
        const bool ok = b < n && __ldg(page_table + (size_t)r * max_pages + b) >= 0;
        const unsigned m = __ballot_sync(kFull, ok);
        const int pos = count + __popc(m & ((1u << lane) - 1u));
        if (ok && pos < k_max) out[pos] = b;
        count += __popc(m);
    }
    count = min(count, k_max);
    for (int i = count + lane; i < k_max; i += 32) out[i] = -1;
    if (lane == 0) sel_cnt[pair] = count;
}

template <int D>
cudaError_t launch_score(const se_params &p, const void *q, const void *meta, const void *k_cache,
                         const int32_t *page_table, const int32_t *seq_lens, float *scores, uint32_t *status,
                         cudaStream_t stream) {
    using C = ScoreCfg<D>;
    const size_t smem = (size_t)kScoreWarps * 2 * C::BUF + kScoreWarps * 2 * 8 +
                        (size_t)(3 * p.B + 1) * sizeof(int);
    auto kern = score_kernel<D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long units_ub = (long long)p.B * p.H_kv * ((p.max_pages + kUnitPages - 1) / kUnitPages);
    int ctas_per_sm = (int)((220 * 1024) / (smem + 1024));
    if (ctas_per_sm > 6) ctas_per_sm = 6;
    if (ctas_per_sm < 1) ctas_per_sm = 1;
    long long grid = (units_ub + kScoreWarps - 1) / kScoreWarps;
    const long long cap = (long long)device_sm_count() * ctas_per_sm;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    kern<<<(unsigned)grid, kScoreWarps * 32, smem, stream>>>(
        (const uint16_t *)q, (const uint8_t *)meta, (const uint8_t *)k_cache, (uint8_t *)const_cast<void *>(meta),
        page_table, seq_lens, scores, score_pitch(p), p.B, p.H_kv,
        p.H_q / p.H_kv, p.max_pages, p.num_phys_pages, effective_scale(p), status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_page_select(const se_params &p, const void *q, const void *meta, const void *k_cache,
                               const int32_t *page_table, const int32_t *seq_lens, int k_pages,
                               int32_t *sel_idx, int32_t *sel_cnt, void *workspace,
                               const WorkspaceLayout &L, cudaStream_t stream, int stages) {
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    float *scores = reinterpret_cast<float *>(ws + L.scores);
    uint32_t *status = reinterpret_cast<uint32_t *>(ws + L.status);
    if (stages == 3 && k_pages >= p.max_pages && p.k_max >= p.max_pages) {
        // dense layer: the budget covers any context this shape can hold
        if (k_cache != nullptr) {           // the fused call still owes the newest page's summary
            cudaError_t em = launch_meta_update(p, k_cache, page_table, seq_lens, nullptr, const_cast<void *>(meta), stream);
            if (em != cudaSuccess) return em;
        }
        const int pairs_all = p.B * p.H_kv;
        select_all_kernel<<<(pairs_all + 7) / 8, 256, 0, stream>>>(page_table, seq_lens, pairs_all, p.H_kv,
                                                                    p.max_pages, p.k_max, sel_idx, sel_cnt);
        return cudaGetLastError();
    }
    if (stages & 1) {
        cudaError_t e = (p.D == 128)
                            ? launch_score<128>(p, q, meta, k_cache, page_table, seq_lens, scores, status, stream)
                            : launch_score<64>(p, q, meta, k_cache, page_table, seq_lens, scores, status, stream);
        if (e != cudaSuccess) return e;
    }
    if (!(stages & 2)) return cudaSuccess;
    const int pairs = p.B * p.H_kv;
    const size_t key_bytes = (size_t)cta_topk_key_words(p.max_pages, kTopkThreads) * sizeof(uint32_t);
    topk_kernel<<<pairs, kTopkThreads, key_bytes, stream>>>(scores, score_pitch(p), seq_lens, p.H_kv, p.max_pages,
                                                            k_pages, p.k_max, p.sink_pages, p.recent_pages, sel_idx,
                                                            sel_cnt);
    return cudaGetLastError();
}

}  // namespace se

// ---------------------------------------------------------------------------------
// se_page_select_static: page selection for callers that cannot allocate device memory.
// The fp32 page scores (the only scratch the selection needs) live in the array below, which
// every GPU that loads this library holds from load to exit.
// ---------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_select_scratch[SE_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// device address of g_select_scratch, per device ordinal (nullptr = not looked up yet).  Host threads may
// race on the first call of a device: the look-up is idempotent, the slot is written atomically.
std::atomic<void *> g_scratch_ptr[kMaxDevices];

// The array's name is only a host-side handle: the address kernels can use has to be asked for,
// once per device, with that device current (the caller's buffers and stream belong to the current
// device, as with every other entry point).
int static_scratch(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SE_ERR_CUDA;
    void *ptr = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || ptr == nullptr) return SE_ERR_CUDA;
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return SE_OK;
}

}  // namespace

extern "C" int se_page_select_static(const se_params *p, const void *q, const void *meta,
                                     const int32_t *page_table, const int32_t *seq_lens,
                                     int32_t budget_tokens, int32_t *sel_idx, int32_t *sel_cnt,
                                     int32_t *dev_status, void *stream) {
    const int vrc = se::validate_params(p);                             // same shape rules and codes as every call
    if (vrc != SE_OK) return vrc;
    if (!q || !meta || !page_table || !seq_lens || !sel_idx || !sel_cnt) return SE_ERR_NULL_POINTER;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(meta) |
                           reinterpret_cast<uintptr_t>(page_table) | reinterpret_cast<uintptr_t>(seq_lens) |
                           reinterpret_cast<uintptr_t>(sel_idx) | reinterpret_cast<uintptr_t>(sel_cnt);
    if ((bits & 15u) || (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return SE_ERR_MISALIGNED;
    if (budget_tokens < se::kPage || budget_tokens / se::kPage + p->sink_pages + p->recent_pages > p->k_max)
        return SE_ERR_INVALID_ARG;
    // scratch layout: [status word, padded to 256 bytes][fp32 scores, B*H_kv rows of max_pages rounded up to 4]
    const size_t need = 256 + (size_t)p->B * p->H_kv * se::score_pitch(*p) * sizeof(float);
    if (need > SE_STATIC_SCRATCH_BYTES) return SE_ERR_SCRATCH_TOO_SMALL;
    void *scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != SE_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the last call left: the status word has to start at zero, the
    // scores are rewritten for every page before they are read
    if (cudaMemsetAsync(scratch, 0, 256, s) != cudaSuccess) return SE_ERR_CUDA;
    se::WorkspaceLayout L = {};
    L.status = 0;
    L.scores = 256;
    L.total = need;
    cudaError_t e = se::launch_page_select(*p, q, meta, nullptr, page_table, seq_lens, budget_tokens / se::kPage,
                                           sel_idx, sel_cnt, scratch, L, s);
    if (e != cudaSuccess) return SE_ERR_CUDA;
    if (dev_status &&
        cudaMemcpyAsync(dev_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return SE_ERR_CUDA;
    return SE_OK;
}

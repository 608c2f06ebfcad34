// Page scoring and top-k page selection (Appendix A, Quest score equation; TopK entry of
// the notation table).
//
// score_kernel   streams the page summaries.  Every warp is an autonomous pipeline: it owns
//                two shared-memory buffers of PB page summaries, fills them with 1-D bulk
//                asynchronous copies (one per page and head, completion on an mbarrier) and
//                computes on one buffer while the other is in flight.  The bound
//                    sum_c max(q_c*m_c, q_c*M_c)
//                is evaluated exactly as  sum_c (q_c^- * m_c + q_c^+ * M_c)  with
//                q^+ = max(q,0), q^- = min(q,0): because M >= m one of the two products is the
//                maximum and the other factor is zero.  Products of bf16 values are exact in
//                fp32, accumulation is fp32 with packed two-wide FMAs, the G query heads of a
//                kv-head share every summary load, and the per-page sums over the lanes that
//                share a page are formed by a transposing shuffle reduction.
// topk_kernel    one CTA per (request, kv-head): most-significant-digit radix select over
//                order-preserving integer keys, then an index-ordered compaction, so equal
//                scores go to the lower page and the list comes out ascending.
#include "se_internal.h"

namespace se {

namespace {

constexpr int kScoreWarps = 4;     // warps per CTA of the score kernel
constexpr int kPB = 16;            // pages per warp batch
constexpr int kNBU = 4;            // batches per work unit  -> 64 pages per (pair, unit)
constexpr int kUnitPages = kPB * kNBU;

template <int D, int G>
struct ScoreCfg {
    static constexpr int GP = next_pow2(G);
    static constexpr int CPL = (G > 4) ? 4 : 8;         // channels per lane and row
    static constexpr int LPP = D / CPL;                 // lanes sharing one (page, head)
    static constexpr int PPP = 32 / LPP;                // pages per warp pass
    static constexpr int NPS = kPB / PPP;               // passes per batch
    static constexpr int RB = (NPS < 32 / GP) ? NPS : 32 / GP;   // passes per reduction block
    static constexpr int NV = RB * GP;                  // partial sums per lane and block
    static constexpr int NF = (NV / LPP) > 1 ? (NV / LPP) : 1;
    static constexpr int LPG = LPP / RB;                // lanes that end up holding one page
    static constexpr int PHB = 2 * D * 2;               // bytes of one page summary
    static_assert(NPS % RB == 0, "reduction blocks tile the batch");
    static_assert(LPG >= 1, "");
};

struct Batch {
    int r, h, b0, n_r;      // request, kv-head, first logical page, pages of the request
    int unit;               // flat unit index this batch belongs to (-1 = end of stream)
    int k;                  // batch number inside the unit
};

// Flat unit u -> (request, head, first page); prefix[r] = units before request r.
__device__ __forceinline__ bool decode_unit(int u, int total_units, const int *prefix, const int *npages,
                                            int B, int H_kv, Batch &d) {
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
    d.b0 = (local / H_kv) * kUnitPages;
    d.n_r = npages[lo];
    d.unit = u;
    d.k = 0;
    return true;
}

template <int D, int G>
__global__ void __launch_bounds__(kScoreWarps * 32)
score_kernel(const uint16_t *__restrict__ q, const uint8_t *__restrict__ meta,
             const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens,
             float *__restrict__ scores, int B, int H_kv, int max_pages, int P_phys, float scale,
             uint32_t *status) {
    using C = ScoreCfg<D, G>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // layout: [buffers: warps*2*PB*PHB] [mbarriers: warps*2*8] [prefix: B+1 ints] [npages: B ints]
    uint8_t *bufs = smem_raw;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)kScoreWarps * 2 * kPB * C::PHB);
    int *prefix = reinterpret_cast<int *>(bars + kScoreWarps * 2);
    int *npages = prefix + (B + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H_q = H_kv * G;

    // ---- per-CTA: units before each request (exclusive prefix over ceil(n_r/64)*H_kv)
    if (warp == 0) {
        int run = 0;
        for (int base = 0; base < B; base += 32) {
            const int r = base + lane;
            int n = 0;
            if (r < B) {
                const int len = seq_lens[r];
                n = len > 0 ? (len + kPage - 1) / kPage : 0;
                if (n > max_pages) n = max_pages;
                npages[r] = n;
            }
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
    const int gw = blockIdx.x * kScoreWarps + warp;
    const int tw = gridDim.x * kScoreWarps;

    uint8_t *my_buf = bufs + (size_t)warp * 2 * kPB * C::PHB;
    const uint32_t bar0 = smem_u32(&bars[warp * 2]);
    const int pp = lane / C::LPP, lg = lane % C::LPP;

    // q registers of the current pair: q^- multiplies the min row, q^+ the max row
    float2 qn[G][C::CPL / 2], qp[G][C::CPL / 2];
    uint32_t qraw[G][C::CPL / 2];            // raw bf16 pairs of the pair whose batch was issued last
    int q_r = -1, q_h = -1;                  // pair the converted registers belong to

    auto load_qraw = [&](const Batch &d) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint16_t *src = q + ((size_t)d.r * H_q + d.h * G + g) * D + lg * C::CPL;
            if constexpr (C::CPL == 8) {
                const uint4 w = __ldg(reinterpret_cast<const uint4 *>(src));
                qraw[g][0] = w.x; qraw[g][1] = w.y; qraw[g][2] = w.z; qraw[g][3] = w.w;
            } else {
                const uint2 w = __ldg(reinterpret_cast<const uint2 *>(src));
                qraw[g][0] = w.x; qraw[g][1] = w.y;
            }
        }
    };
    auto convert_q = [&]() {
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int j = 0; j < C::CPL / 2; ++j) {
                const float2 f = bf16x2_to_f2(qraw[g][j]);
                qp[g][j] = make_float2(fmaxf(f.x, 0.f), fmaxf(f.y, 0.f));
                qn[g][j] = make_float2(fminf(f.x, 0.f), fminf(f.y, 0.f));
            }
    };

    // advance a descriptor to the next batch of this warp's stream
    auto next_batch = [&](Batch &d) {
        if (d.unit < 0) return;
        if (d.k + 1 < kNBU && d.b0 + kPB < d.n_r) {
            d.k += 1;
            d.b0 += kPB;
            return;
        }
        decode_unit(d.unit + tw, total_units, prefix, npages, B, H_kv, d);
    };

    // issue the copies of one batch into buffer `slot`; returns this lane's physical page (or -1)
    auto issue = [&](const Batch &d, int slot) -> int {
        int pid = -1;
        if (lane < kPB) {
            const int b = d.b0 + lane;
            if (b < d.n_r) {
                pid = page_table[(size_t)d.r * max_pages + b];
                if (pid >= P_phys) {
                    atomicOr(status, SE_DEV_BAD_PAGE_ID);
                    pid = -1;
                }
            }
        }
        const unsigned valid = __ballot_sync(kFull, pid >= 0);
        const uint32_t bar = bar0 + slot * 8;
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(valid) * C::PHB);
        __syncwarp();
        if (pid >= 0) {
            const uint8_t *src = meta + ((size_t)pid * H_kv + d.h) * C::PHB;
            bulk_g2s(smem_u32(my_buf + ((size_t)slot * kPB + lane) * C::PHB), src, C::PHB, bar);
        }
        return pid;
    };

    Batch cur, nxt;
    decode_unit(gw, total_units, prefix, npages, B, H_kv, cur);
    if (cur.unit < 0) return;
    uint32_t phases = 0u;            // parity bit per buffer
    int slot = 0;
    int pid_cur = issue(cur, slot);
    load_qraw(cur);
    int pid_nxt = -1;
    bool failed = false;

    while (cur.unit >= 0) {
        nxt = cur;
        next_batch(nxt);
        // the pair of `cur` may differ from the converted registers: convert before qraw is reused
        if (cur.r != q_r || cur.h != q_h) {
            convert_q();
            q_r = cur.r;
            q_h = cur.h;
        }
        if (nxt.unit >= 0) {
            pid_nxt = issue(nxt, slot ^ 1);
            if (nxt.r != cur.r || nxt.h != cur.h) load_qraw(nxt);
        }
        // wait for the current buffer
        if (!mbar_wait(bar0 + slot * 8, (phases >> slot) & 1u)) {
            failed = true;
            break;
        }
        phases ^= (1u << slot);

        const uint8_t *buf = my_buf + (size_t)slot * kPB * C::PHB;
        float *dst = scores + ((size_t)cur.r * H_kv + cur.h) * max_pages + cur.b0;
#pragma unroll
        for (int rb = 0; rb < C::NPS / C::RB; ++rb) {
            float v[C::NV];
#pragma unroll
            for (int ip = 0; ip < C::RB; ++ip) {
                const int j = (rb * C::RB + ip) * C::PPP + pp;          // page inside the batch
                const uint8_t *pg = buf + (size_t)j * C::PHB + lg * (C::CPL * 2);
                uint32_t mnw[C::CPL / 2], mxw[C::CPL / 2];
                if constexpr (C::CPL == 8) {
                    const uint4 a = *reinterpret_cast<const uint4 *>(pg);
                    const uint4 b = *reinterpret_cast<const uint4 *>(pg + D * 2);
                    mnw[0] = a.x; mnw[1] = a.y; mnw[2] = a.z; mnw[3] = a.w;
                    mxw[0] = b.x; mxw[1] = b.y; mxw[2] = b.z; mxw[3] = b.w;
                } else {
                    const uint2 a = *reinterpret_cast<const uint2 *>(pg);
                    const uint2 b = *reinterpret_cast<const uint2 *>(pg + D * 2);
                    mnw[0] = a.x; mnw[1] = a.y;
                    mxw[0] = b.x; mxw[1] = b.y;
                }
                float2 mnf[C::CPL / 2], mxf[C::CPL / 2];
#pragma unroll
                for (int c = 0; c < C::CPL / 2; ++c) {
                    mnf[c] = bf16x2_to_f2(mnw[c]);
                    mxf[c] = bf16x2_to_f2(mxw[c]);
                }
#pragma unroll
                for (int g = 0; g < C::GP; ++g) {
                    if (g < G) {
                        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
                        for (int c = 0; c < C::CPL / 2; ++c) {
                            acc = ffma2(mnf[c], qn[g < G ? g : 0][c], acc);
                            acc = ffma2(mxf[c], qp[g < G ? g : 0][c], acc);
                        }
                        v[ip * C::GP + g] = acc.x + acc.y;
                    } else {
                        v[ip * C::GP + g] = 0.f;
                    }
                }
            }
            transpose_reduce<C::NV, C::LPP>(v, lane);
            // lane lg now holds NF sums of page ip = lg / LPG; fold the group's heads by max
            const int i0 = (C::NV >= C::LPP) ? lg * C::NF : lg / (C::LPP / C::NV);
            float s = -INFINITY;
#pragma unroll
            for (int j = 0; j < C::NF; ++j) {
                const int g = (i0 + j) % C::GP;
                if (g < G) s = fmaxf(s, v[j]);
            }
#pragma unroll
            for (int m = 1; m < C::LPG; m <<= 1) s = fmaxf(s, __shfl_xor_sync(kFull, s, m));
            const int ip = lg / C::LPG;
            const int j = (rb * C::RB + ip) * C::PPP + pp;
            const int pid_j = __shfl_sync(kFull, pid_cur, j);
            if ((lg % C::LPG) == 0 && cur.b0 + j < cur.n_r)
                dst[j] = (pid_j >= 0) ? s * scale : -INFINITY;
        }
        __syncwarp();        // every lane is done reading the buffer before it is refilled
        cur = nxt;
        pid_cur = pid_nxt;
        slot ^= 1;
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        // give the copy that may still be in flight a bounded chance to land before leaving
        mbar_wait(bar0 + (slot ^ 1) * 8, (phases >> (slot ^ 1)) & 1u);
    }
}

// ---------------------------------------------------------------------------------
// top-k: one CTA per (request, kv-head)
// ---------------------------------------------------------------------------------
constexpr int kTopkThreads = 256;

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float *__restrict__ scores, const int32_t *__restrict__ seq_lens, int H_kv,
            int max_pages, int k_pages, int k_max, int32_t *__restrict__ sel_idx,
            int32_t *__restrict__ sel_cnt) {
    __shared__ int hist[256];
    __shared__ int s_present, s_digit, s_above, s_inbin;
    __shared__ int warp_eq[kTopkThreads / 32], warp_sel[kTopkThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair = blockIdx.x;
    const int r = pair / H_kv;
    const int len = seq_lens[r];
    int n = len > 0 ? (len + kPage - 1) / kPage : 0;
    if (n > max_pages) n = max_pages;
    const float *row = scores + (size_t)pair * max_pages;
    int32_t *out = sel_idx + (size_t)pair * k_max;

    uint32_t prefix = 0;          // digits fixed so far (higher bits), lower bits zero
    int remaining = 0;            // how many still to take among keys matching the prefix
    int k_eff = 0;
    bool ge_mode = false;         // take every key >= prefix (the whole bin is wanted)

    if (tid == 0) s_present = 0;
    for (int shift = 24; shift >= 0 && !ge_mode; shift -= 8) {
        hist[tid] = 0;
        __syncthreads();
        int present = 0;
        for (int i = tid; i < n; i += kTopkThreads) {
            const uint32_t key = f32_key(row[i]);
            if (shift == 24) {
                present += (key != kKeyAbsent);
                atomicAdd(&hist[key >> 24], 1);
            } else if ((key >> (shift + 8)) == (prefix >> (shift + 8))) {
                atomicAdd(&hist[(key >> shift) & 255u], 1);
            }
        }
        if (shift == 24 && present) atomicAdd(&s_present, present);
        __syncthreads();
        if (shift == 24) {
            k_eff = min(min(k_pages, k_max), s_present);
            remaining = k_eff;
            if (k_eff == 0) break;
        }
        // find the digit d with  #(digits > d) < remaining <= #(digits >= d)
        if (warp == 0) {
            int loc[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                loc[j] = hist[lane * 8 + j];
                sum += loc[j];
            }
            int suf = sum;          // inclusive suffix sum over lanes (higher lanes = higher digits)
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_down_sync(kFull, suf, o);
                if (lane + o < 32) suf += t;
            }
            const int above_lane = suf - sum;      // digits in higher lanes
            if (above_lane < remaining && remaining <= suf) {
                int above = above_lane;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (above < remaining && remaining <= above + loc[j]) {
                        s_digit = lane * 8 + j;
                        s_above = above;
                        s_inbin = loc[j];
                    }
                    above += loc[j];
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)s_digit << shift;
        remaining -= s_above;
        if (s_inbin == remaining) ge_mode = true;      // the whole bin is taken: no ties to break
        __syncthreads();
    }

    if (k_eff == 0) {
        for (int i = tid; i < k_max; i += kTopkThreads) out[i] = -1;
        if (tid == 0) sel_cnt[pair] = 0;
        return;
    }
    // keys > T are taken; keys == T are taken in index order until `need` of them are in.
    // In ge_mode every key >= prefix is taken (T = prefix, need = unlimited).
    const uint32_t T = prefix;
    const int need = ge_mode ? 0x7fffffff : remaining;

    int run_eq = 0, run_sel = 0;
    for (int base = 0; base < n; base += kTopkThreads) {
        const int i = base + tid;
        uint32_t key = 0;
        bool gt = false, eq = false;
        if (i < n) {
            key = f32_key(row[i]);
            gt = ge_mode ? (key >= T) : (key > T);
            eq = !ge_mode && (key == T);
        }
        const unsigned beq = __ballot_sync(kFull, eq);
        if (lane == 0) warp_eq[warp] = __popc(beq);
        __syncthreads();
        int eq_before = run_eq, eq_total = 0;
#pragma unroll
        for (int w = 0; w < kTopkThreads / 32; ++w) {
            const int c = warp_eq[w];
            if (w < warp) eq_before += c;
            eq_total += c;
        }
        eq_before += __popc(beq & ((1u << lane) - 1u));
        const bool take = gt || (eq && eq_before < need);
        const unsigned bsel = __ballot_sync(kFull, take);
        if (lane == 0) warp_sel[warp] = __popc(bsel);
        __syncthreads();
        int pos = run_sel, sel_total = 0;
#pragma unroll
        for (int w = 0; w < kTopkThreads / 32; ++w) {
            const int c = warp_sel[w];
            if (w < warp) pos += c;
            sel_total += c;
        }
        pos += __popc(bsel & ((1u << lane) - 1u));
        if (take && pos < k_max) out[pos] = i;
        run_eq += eq_total;
        run_sel += sel_total;
        __syncthreads();
    }
    for (int i = k_eff + tid; i < k_max; i += kTopkThreads) out[i] = -1;
    if (tid == 0) sel_cnt[pair] = k_eff;
}

template <int D, int G>
cudaError_t launch_score(const se_params &p, const void *q, const void *meta, const int32_t *page_table,
                         const int32_t *seq_lens, float *scores, uint32_t *status, cudaStream_t stream) {
    using C = ScoreCfg<D, G>;
    const size_t smem = (size_t)kScoreWarps * 2 * kPB * C::PHB + kScoreWarps * 2 * 8 +
                        (size_t)(2 * p.B + 1) * sizeof(int);
    auto kern = score_kernel<D, G>;
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
        (const uint16_t *)q, (const uint8_t *)meta, page_table, seq_lens, scores, p.B, p.H_kv,
        p.max_pages, p.num_phys_pages, effective_scale(p), status);
    return cudaGetLastError();
}

template <int D>
cudaError_t dispatch_score(const se_params &p, const void *q, const void *meta, const int32_t *page_table,
                           const int32_t *seq_lens, float *scores, uint32_t *status, cudaStream_t stream) {
    switch (p.H_q / p.H_kv) {
        case 1: return launch_score<D, 1>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 2: return launch_score<D, 2>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 3: return launch_score<D, 3>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 4: return launch_score<D, 4>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 5: return launch_score<D, 5>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 6: return launch_score<D, 6>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 7: return launch_score<D, 7>(p, q, meta, page_table, seq_lens, scores, status, stream);
        case 8: return launch_score<D, 8>(p, q, meta, page_table, seq_lens, scores, status, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_page_select(const se_params &p, const void *q, const void *meta,
                               const int32_t *page_table, const int32_t *seq_lens, int k_pages,
                               int32_t *sel_idx, int32_t *sel_cnt, void *workspace,
                               const WorkspaceLayout &L, cudaStream_t stream) {
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    float *scores = reinterpret_cast<float *>(ws + L.scores);
    uint32_t *status = reinterpret_cast<uint32_t *>(ws + L.status);
    cudaError_t e = (p.D == 128)
                        ? dispatch_score<128>(p, q, meta, page_table, seq_lens, scores, status, stream)
                        : dispatch_score<64>(p, q, meta, page_table, seq_lens, scores, status, stream);
    if (e != cudaSuccess) return e;
    topk_kernel<<<p.B * p.H_kv, kTopkThreads, 0, stream>>>(scores, seq_lens, p.H_kv, p.max_pages,
                                                         k_pages, p.k_max, sel_idx, sel_cnt);
    return cudaGetLastError();
}

}  // namespace se

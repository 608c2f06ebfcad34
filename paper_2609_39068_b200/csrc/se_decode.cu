// Paged attention over the selected pages, log-sum-exp merge and the H2O epilogue
// (Appendix A, selected-attention equation and H2O accumulated-score equation).
//
// Three attention kernels share the per-page arithmetic (WarpAttn) and the per-warp copy pipeline
// (attend_range); which one runs follows from the shape alone (make_decode_plan):
//
// decode_kernel      many (request, kv-head) pairs.  Persistent grid, every warp an autonomous
//                    pipeline working through (pair, split) units; with more than four pairs per SM
//                    a pair is one unit and its warp writes out/lse itself, with fewer than two the
//                    pair is cut into splits whose partials (acc, m, l) combine_kernel merges.
// decode_duo_kernel  two to four pairs per SM.  Two adjacent warps share a pair (the two halves of
//                    its list) and merge through the shared memory of their drained rings: twice
//                    the busy warps per SM of the one-warp form, no partials in global memory.
// decode_cta_kernel  at most one pair per SM.  A CTA is one (pair, CTA-split); its eight warps share
//                    the CTA's pages and their partials are merged through shared memory.  The CTAs
//                    of a pair (up to 8) form a thread-block cluster: after a cluster barrier each
//                    of them merges a share of the CTAs' partials and applies the H2O update to the
//                    tokens it attended - no merge kernel, no partials of single warps.
//
// decode_cta_kernel can take the selection from the page scores themselves (kSelect): the CTA runs
// the top-k in its prologue (se_topk.cuh: cta_topk), while the shared-memory ring is still empty and
// serves as its scratch; the list is also written to sel_idx / sel_cnt.  That removes the top-k
// kernel and the selection's round trip from the step.  (With warp units a warp would have to run the
// top-k alone, which is slower than the top-k kernel: those shapes keep it.)  With kFused the CTAs of the
// pair's cluster first score the pair's pages themselves (cta_score_range: the page summaries stream
// through the same ring, the scores go to the workspace, a cluster barrier ends the phase), so the
// whole step - summary of the newest page, scores, top-k, attention, merge, H2O update - is one launch.
//
// Per page, for the G query heads of the kv-head at once:
//     S^T[head, token] = Q[head, :] . K[token, :]^T      (m16n8k16, fp32 accumulate)
//     online softmax in base 2 on the accumulator fragments
//     O[head, :]      += P[head, token] . V[token, :]    (P split into two bf16 terms)
// K and V pages ([16 tokens, D] bf16, contiguous per head) arrive by one 3-D TMA tensor copy each
// (64 channels x 16 rows x D/64 halves, 128-byte swizzle, one mbarrier per ring stage), so ldmatrix
// reads them without bank conflicts.  The accumulator layout of S^T is the A-operand layout of P, so
// the probabilities never leave registers.
//
// combine_kernel     merges split partials where the attention kernel did not (one warp per query
//                    head) and adds exp(z - lse), summed over the query heads of the kv-head, to the
//                    accumulated score of every attended token slot (the H2O epilogue).
#include <cuda.h>

#include "se_internal.h"
#include "se_topk.cuh"

namespace se {

namespace {

constexpr int kDecWarps = 8;
constexpr int kChunk = 128;              // selected pages looked up at once
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTileBytes = kPage * 128;  // one TMA box: 16 rows x 64 bf16

template <int D>
struct DecCfg {
    static constexpr int PAGEB = kPage * D * 2;                // bytes of one K (or V) page
    static constexpr int STAGEB = 2 * PAGEB;                   // K tiles then V tiles
    static constexpr int MAXST = 8;                            // most stages one warp can hold
    // Stages a CTA of decode_kernel shares out among its busy warps.  More copies in flight than
    // this made that kernel slower, not faster (measured: 24 pages in flight per SM lose 3 %
    // against 16 to 20).
    static constexpr int CTA_STAGES = 20 * (128 / D);
    // decode_cta_kernel: three stages for each of the eight warps
    static constexpr int CTA_STAGES_SPLIT = 24 * (128 / D);
    static constexpr int KSTEPS = D / 16;
    static constexpr int NTILES = D / 8;                       // n8 tiles of the output
    static constexpr int PSTRIDE = D + 4;                      // floats per partial row
};

// TMA: one page = 3-D box (64 channels, 16 token rows, D/64 channel halves) of the cache viewed as
// [half][row][64 channels]; it lands as D/64 swizzled 16x128-byte tiles, one after the other.
__device__ __forceinline__ void tma_load_page(uint32_t dst, const CUtensorMap *map, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(0), "r"(y), "r"(0), "r"(bar)
        : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------------------------
// Per-warp attention state: Q fragments, output accumulators and the running softmax statistics
// of the G query heads of one kv-head.  Lane (gid = lane >> 2, tid4 = lane & 3) holds head row gid.
// ---------------------------------------------------------------------------------
template <int D>
struct WarpAttn {
    using C = DecCfg<D>;
    uint32_t qa[C::KSTEPS][2];       // Q as the A operand: row gid = query head gid (rows >= G and 8..15 zero)
    float o_acc[C::NTILES][4];       // elements 0,1: p_hi products, 2,3: p_lo products (added in finish())
    float m_run, l_run;              // of head gid; l is this lane's share (its 4 token columns) until finish()
    // ldmatrix lane offsets inside a 16x128-byte swizzled tile (byte offset of the lane's row, its row & 7,
    // and which of the two 16-byte chunks of a pair it addresses)
    int k_rowoff, k_swz, k_chunk_add;    // K (B operand, not transposed): matrices {tok 0-7 | 8-15} x {chunk c | c+1}
    int v_rowoff, v_swz, v_chunk_add, v_row;   // V (transposed): matrices {tok 0-7 | 8-15} fastest, then {chunk c | c+1}
    int t0;                              // first token column of this lane

    __device__ __forceinline__ void init_lane(int lane) {
        const int k_row = (lane & 7) + 8 * (lane >> 4);
        k_rowoff = k_row * 128;
        k_swz = k_row & 7;
        k_chunk_add = (lane >> 3) & 1;
        v_row = (lane & 7) + 8 * ((lane >> 3) & 1);
        v_rowoff = v_row * 128;
        v_swz = v_row & 7;
        v_chunk_add = lane >> 4;
        t0 = 2 * (lane & 3);
    }

    __device__ __forceinline__ void load_q(const uint16_t *__restrict__ q, size_t head0, int lane, int G) {
        const int gid = lane >> 2, tid4 = lane & 3;
        const bool head_ok = gid < G;
        const uint16_t *src = q + (head0 + (head_ok ? gid : 0)) * D + 2 * tid4;
#pragma unroll
        for (int s = 0; s < C::KSTEPS; ++s) {
            const uint32_t w0 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16));
            const uint32_t w1 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16 + 8));
            qa[s][0] = head_ok ? w0 : 0u;
            qa[s][1] = head_ok ? w1 : 0u;
        }
    }
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int nt = 0; nt < C::NTILES; ++nt) {
            o_acc[nt][0] = 0.f; o_acc[nt][1] = 0.f; o_acc[nt][2] = 0.f; o_acc[nt][3] = 0.f;
        }
        m_run = -INFINITY;
        l_run = 0.f;
    }
    // Logits (base 2, scaled) of head gid for tokens 2*tid4, 2*tid4+1, 8+2*tid4, 9+2*tid4 of the page
    // whose K tiles sit at Ks; tokens >= nv are masked to -inf.
    __device__ __forceinline__ void logits(uint32_t Ks, int nv, float scale_log2, float (&z)[4]) const {
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        float s0b[4] = {0.f, 0.f, 0.f, 0.f}, s1b[4] = {0.f, 0.f, 0.f, 0.f};   // odd k-steps: shorter chains
#pragma unroll
        for (int s = 0; s < C::KSTEPS; ++s) {
            const int hf = s >> 2;
            const int chunk = 2 * (s & 3) + k_chunk_add;
            uint32_t b00, b01, b10, b11;     // {tok 0-7: k lo, k hi}, {tok 8-15: k lo, k hi}
            ldmatrix_x4(Ks + hf * kTileBytes + k_rowoff + ((chunk ^ k_swz) << 4), b00, b01, b10, b11);
            if (s & 1) {
                mma_bf16_16816(s0b, qa[s][0], 0u, qa[s][1], 0u, b00, b01);
                mma_bf16_16816(s1b, qa[s][0], 0u, qa[s][1], 0u, b10, b11);
            } else {
                mma_bf16_16816(s0, qa[s][0], 0u, qa[s][1], 0u, b00, b01);
                mma_bf16_16816(s1, qa[s][0], 0u, qa[s][1], 0u, b10, b11);
            }
        }
        s0[0] += s0b[0]; s0[1] += s0b[1]; s1[0] += s1b[0]; s1[1] += s1b[1];
        z[0] = (t0 < nv) ? s0[0] * scale_log2 : -INFINITY;
        z[1] = (t0 + 1 < nv) ? s0[1] * scale_log2 : -INFINITY;
        z[2] = (t0 + 8 < nv) ? s1[0] * scale_log2 : -INFINITY;
        z[3] = (t0 + 9 < nv) ? s1[1] * scale_log2 : -INFINITY;
    }
    // Online-softmax update with the page's logits and O += P . V for the V tiles at Vs.
    __device__ __forceinline__ void accumulate(uint32_t Vs, int nv, const float (&z)[4], uint32_t zero_chunk) {
        float pmax = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
        pmax = fmaxf(pmax, __shfl_xor_sync(kFull, pmax, 1));
        pmax = fmaxf(pmax, __shfl_xor_sync(kFull, pmax, 2));
        const float m_new = fmaxf(m_run, pmax);           // finite: token 0 of a page is always valid
        const float corr = exp2f(m_run - m_new);          // 0 on the first page (m_run = -inf)
        if (__any_sync(kFull, m_new != m_run)) {
            l_run *= corr;
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt) {
                o_acc[nt][0] *= corr;
                o_acc[nt][1] *= corr;
                o_acc[nt][2] *= corr;
                o_acc[nt][3] *= corr;
            }
            m_run = m_new;
        }
        float p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) p[e] = exp2f(z[e] - m_run);    // exp2(-inf) = 0 for masked tokens
        l_run += (p[0] + p[1]) + (p[2] + p[3]);
        // P as the A operand, split into two bf16 terms so that p_hi + p_lo carries 16 bits.  The
        // group has at most 8 heads, so rows 8-15 of the m16 tile are free: p_hi goes into rows
        // 0-7 and p_lo into rows 8-15, and one MMA yields both products (accumulator elements
        // 0,1 and 2,3 of this lane); they are added in finish().
        const uint32_t ph0 = pack_bf16(p[0], p[1]), ph1 = pack_bf16(p[2], p[3]);
        const float2 f0 = bf16x2_to_f2(ph0), f1 = bf16x2_to_f2(ph1);
        const uint32_t pl0 = pack_bf16(p[0] - f0.x, p[1] - f0.y), pl1 = pack_bf16(p[2] - f1.x, p[3] - f1.y);
#pragma unroll
        for (int c2 = 0; c2 < C::NTILES / 2; ++c2) {
            const int hf = c2 >> 2;
            const int chunk = 2 * (c2 & 3) + v_chunk_add;
            uint32_t v00, v01, v10, v11;     // {chunk c: tok 0-7, tok 8-15}, {chunk c+1: ...}
            // token rows past the request's length may hold anything (NaN included) and their
            // weights are zero: their lanes read a zeroed chunk instead
            const uint32_t va = Vs + hf * kTileBytes + v_rowoff + ((chunk ^ v_swz) << 4);
            ldmatrix_x4_trans(v_row < nv ? va : zero_chunk, v00, v01, v10, v11);
            mma_bf16_16816(o_acc[2 * c2], ph0, pl0, ph1, pl1, v00, v01);
            mma_bf16_16816(o_acc[2 * c2 + 1], ph0, pl0, ph1, pl1, v10, v11);
        }
    }
    // The four lanes of a head hold disjoint token columns: fold their l; add the p_hi and p_lo products.
    __device__ __forceinline__ void finish() {
        l_run += __shfl_xor_sync(kFull, l_run, 1);
        l_run += __shfl_xor_sync(kFull, l_run, 2);
#pragma unroll
        for (int nt = 0; nt < C::NTILES; ++nt) {
            o_acc[nt][0] += o_acc[nt][2];
            o_acc[nt][1] += o_acc[nt][3];
        }
    }
};

// ---------------------------------------------------------------------------------
// Per-warp copy pipeline: a ring of `nstage` stages (one stage = K page + V page of one head), one
// mbarrier per stage, and the list of the pages of the current chunk of selection entries.
// ---------------------------------------------------------------------------------
struct WarpPipe {
    uint32_t ring0, bar0;    // shared-memory addresses of the warp's first stage / first barrier
    int nstage;
    uint32_t phases;         // parity bit per stage
    int stage_c, stage_i;    // next stage to consume / to fill
    int *ent_y;              // row of the page's first token in the [pages*heads*16, D] view of the cache
    int *ent_info;           // valid tokens (bits 0-4) | selection index i (bits 5..)
    int *ent_b;              // logical page (only read by an observation layer)
};

struct AttendArgs {
    const CUtensorMap *k_map, *v_map;
    const int32_t *page_table;
    int max_pages, H_kv, P_phys, G, GP;
    float *zrow;             // H2O: logits of this pair, [k_max][16][GP] (nullptr = off)
    uint32_t *keys_row;      // observation layer: token keys of this request (nullptr = off)
    float scale_log2;
    uint32_t zero_chunk;
    uint32_t *status;
};

// Attends the selection entries [i_lo, i_hi) of one (request r, kv-head hh) pair; sel_at(i) is the
// logical page of entry i.  The valid pages of up to kChunk entries are looked up at once (selection
// -> page table, two dependent loads for the whole chunk) and kept in shared memory; the copy
// pipeline then runs over that list without further global look-ups.  Returns false when a bounded
// wait gave up.  `first` (when kFirst) holds the entries i_lo + rep*32 + lane of the first chunk, loaded by
// the caller ahead of time so that they travel together with the lengths instead of after them.
template <int D, bool kObserve, bool kFirst, typename SelAt>
__device__ __forceinline__ bool attend_range(WarpPipe &P, WarpAttn<D> &A, const AttendArgs &a, SelAt sel_at,
                                             const int (&first)[kChunk / 32], int i_lo, int i_hi, int r, int hh, int len,
                                             int n_r, int lane, bool use_first = true) {
    using C = DecCfg<D>;
    const int gid = lane >> 2, tid4 = lane & 3;
    const float scale_log2 = a.scale_log2;
    const uint32_t zero_chunk = a.zero_chunk;
    float *const zrow = a.zrow;
    const int GP = a.GP;
    const bool head_ok = gid < a.G;
    int chunk_end = i_lo;
    int n_ent = 0, ce = 0, pe = 0;               // entries, next to consume, next to issue

    auto fill_chunk = [&](int base) {
        const int end = min(i_hi, base + kChunk);
        int sl_pid[kChunk / 32], sl_meta[kChunk / 32], sl_b[kObserve ? kChunk / 32 : 1];
#pragma unroll
        for (int rep = 0; rep < kChunk / 32; ++rep) {
            const int i = base + rep * 32 + lane;
            int pid = -1, meta = 0, lb = 0;
            if (i < end) {
                const int b = (kFirst && use_first && base == i_lo) ? first[rep] : sel_at(i);
                if (b < 0 || b >= n_r) {
                    atomicOr(a.status, SE_DEV_BAD_SELECTION);
                } else {
                    pid = __ldg(a.page_table + (size_t)r * a.max_pages + b);
                    lb = b;
                    meta = min(kPage, len - b * kPage) | (i << 5);
                }
            }
            sl_pid[rep] = pid;
            sl_meta[rep] = meta;
            if (kObserve) sl_b[rep] = lb;
        }
        int count = 0;
#pragma unroll
        for (int rep = 0; rep < kChunk / 32; ++rep) {
            int pid = sl_pid[rep];
            const bool looked_up = sl_meta[rep] != 0;
            if (looked_up && pid >= a.P_phys) {
                atomicOr(a.status, SE_DEV_BAD_PAGE_ID);
                pid = -1;
            } else if (looked_up && pid < 0) {
                atomicOr(a.status, SE_DEV_BAD_SELECTION);
            }
            const unsigned vm = __ballot_sync(kFull, pid >= 0);
            if (pid >= 0) {
                const int pos = count + __popc(vm & ((1u << lane) - 1u));
                P.ent_y[pos] = (pid * a.H_kv + hh) * kPage;
                P.ent_info[pos] = sl_meta[rep];
                if (kObserve) P.ent_b[pos] = sl_b[rep];
            }
            count += __popc(vm);
        }
        __syncwarp();
        chunk_end = end;
        n_ent = count;
        ce = 0;
        pe = 0;
    };
    // called between pages, when no stage is being read: fill every free stage.  Lane 0 fetches the
    // K page, lane 1 the V page; each arms the stage's barrier with its own byte count (the barrier
    // expects two arrivals, so the lanes need no ordering between themselves).
    auto top_up = [&]() {
        while (pe < n_ent && pe < ce + P.nstage) {
            if (lane < 2) {
                const uint32_t bar = P.bar0 + P.stage_i * 8;
                const uint32_t dst = P.ring0 + P.stage_i * C::STAGEB + lane * C::PAGEB;
                mbar_expect_tx(bar, C::PAGEB);
                tma_load_page(dst, lane ? a.v_map : a.k_map, P.ent_y[pe], bar);
            }
            P.stage_i = (P.stage_i + 1 == P.nstage) ? 0 : P.stage_i + 1;
            ++pe;
        }
    };

    fill_chunk(i_lo);
    top_up();
    for (;;) {
        if (ce == n_ent) {                       // list exhausted: more entries left?
            if (chunk_end >= i_hi) break;
            fill_chunk(chunk_end);
            top_up();
            continue;
        }
        const int info = P.ent_info[ce];
        const int nv_j = info & 31;
        const int i_j = info >> 5;
        if (!mbar_wait(P.bar0 + P.stage_c * 8, (P.phases >> P.stage_c) & 1u)) return false;
        P.phases ^= (1u << P.stage_c);
        const uint32_t Ks = P.ring0 + P.stage_c * C::STAGEB;
        const uint32_t Vs = Ks + C::PAGEB;
        P.stage_c = (P.stage_c + 1 == P.nstage) ? 0 : P.stage_c + 1;

        float z[4];
        A.logits(Ks, nv_j, scale_log2, z);
        const int t0 = 2 * tid4;
        if (zrow != nullptr && head_ok) {
            float *zp = zrow + ((size_t)i_j * kPage) * GP + gid;
            zp[(t0) * GP] = z[0];
            zp[(t0 + 1) * GP] = z[1];
            zp[(t0 + 8) * GP] = z[2];
            zp[(t0 + 9) * GP] = z[3];
        }
        A.accumulate(Vs, nv_j, z, zero_chunk);
        const int page_b = kObserve ? P.ent_b[ce] : 0;
        __syncwarp();     // all lanes are done with this stage before it is refilled
        ++ce;
        top_up();
        if (kObserve) {
            // (after the stage has been handed back for refilling: the scores only need z)
            // observation layer: s(j) = max over every query head of the logit (Appendix A, OmniKV
            // selection equation).  Here: max over the group's heads (rows gid; rows past the group
            // hold zero queries and are left out), then an atomic max over the kv-heads on the
            // order-preserving integer image of the score.
            float m4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = head_ok ? z[e] : -INFINITY;
                v = fmaxf(v, __shfl_xor_sync(kFull, v, 4));
                v = fmaxf(v, __shfl_xor_sync(kFull, v, 8));
                v = fmaxf(v, __shfl_xor_sync(kFull, v, 16));
                m4[e] = v;
            }
            // after the butterfly every row holds the maxima; rows 0-3 send one token each, so the 16 tokens
            // of the page leave as ONE atomic instruction over 64 contiguous bytes
            if (gid < 4) {
                const float mv = gid == 0 ? m4[0] : gid == 1 ? m4[1] : gid == 2 ? m4[2] : m4[3];
                const int tok = t0 + (gid & 1) + 8 * (gid >> 1);
                if (mv > -INFINITY) atomicMax(a.keys_row + page_b * kPage + tok, f32_key(mv * kLn2));
            }
        }
    }
    return true;
}

// Where a unit's selection comes from: the list the caller passes (sel_idx / sel_cnt are read) or,
// with kSelect, the page scores in the workspace (the top-k runs here and sel_idx / sel_cnt are written).
struct SelectArgs {
    int32_t *sel_idx;        // [pairs][k_max]
    int32_t *sel_cnt;        // [pairs]
    const float *scores;     // [pairs][pitch]
    int pitch, k_pages, sink, recent;
};

// ---------------------------------------------------------------------------------
// decode_kernel: persistent warps over (pair, split) units.
// ---------------------------------------------------------------------------------
template <int D, bool kObserve>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
decode_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
              const uint16_t *__restrict__ q, const int32_t *__restrict__ page_table,
              const int32_t *__restrict__ seq_lens, const SelectArgs sa, float *__restrict__ out,
              float *__restrict__ lse, float *__restrict__ partials, float *__restrict__ zbuf,
              uint32_t *__restrict__ tok_keys, int B, int H_kv, int G, int GP, int max_pages, int P_phys, int k_max,
              int pages_per_split, int max_splits, float scale_log2, uint32_t *status) {
    using C = DecCfg<D>;
    extern __shared__ uint8_t smem_dyn[];
    // tiles must sit on 1024-byte boundaries for the 128-byte swizzle pattern
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The CTA's stages are shared out among the warps that have work: warp w of this CTA is busy iff
    // its first unit w*gridDim.x + blockIdx.x exists, so the busy warps are the lowest ones.  Every
    // busy warp of the GRID gets the same number of stages - that of the fullest CTAs - so that the
    // bytes a CTA keeps in flight, and with them its share of the memory bandwidth, follow its
    // number of units: a CTA with three units and deeper pipelines would finish well before the CTAs
    // with four, which then decide the kernel's time at less than full bandwidth.
    int busy = (B * H_kv * max_splits - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    busy = busy < 1 ? 1 : (busy > kDecWarps ? kDecWarps : busy);
    int busy_max = (B * H_kv * max_splits + (int)gridDim.x - 1) / (int)gridDim.x;
    busy_max = busy_max > kDecWarps ? kDecWarps : busy_max;
    WarpPipe P;
    P.nstage = warp < busy ? min(C::MAXST, C::CTA_STAGES / busy_max) : 0;
    uint8_t *ring = smem_al + (size_t)(warp * P.nstage) * C::STAGEB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + (size_t)C::CTA_STAGES * C::STAGEB) + warp * C::MAXST;
    if (lane == 0) {
        for (int s = 0; s < P.nstage; ++s) mbar_init(smem_u32(&bars[s]), 2);
        mbar_fence_init();
    }
    __syncwarp();
    P.bar0 = smem_u32(&bars[0]);
    P.ring0 = smem_u32(ring);
    P.phases = 0;
    P.stage_c = 0;
    P.stage_i = 0;
    uint8_t *lists = smem_al + (size_t)C::CTA_STAGES * C::STAGEB + kDecWarps * C::MAXST * 8;
    P.ent_y = reinterpret_cast<int *>(lists) + warp * 3 * kChunk;
    P.ent_info = P.ent_y + kChunk;
    P.ent_b = P.ent_info + kChunk;
    // 16 zero bytes per CTA (behind the page lists)
    uint8_t *zero_bytes = lists + (size_t)kDecWarps * 3 * kChunk * sizeof(int);
    if (threadIdx.x < 4) reinterpret_cast<uint32_t *>(zero_bytes)[threadIdx.x] = 0u;
    __syncthreads();

    AttendArgs a;
    a.k_map = &k_map;
    a.v_map = &v_map;
    a.page_table = page_table;
    a.max_pages = max_pages;
    a.H_kv = H_kv;
    a.P_phys = P_phys;
    a.G = G;
    a.GP = GP;
    a.scale_log2 = scale_log2;
    a.zero_chunk = smem_u32(zero_bytes);
    a.status = status;

    const int H_q = H_kv * G;
    const int gid = lane >> 2, tid4 = lane & 3;
    const bool head_ok = gid < G;
    // Work unit = (pair, split): selection entries [split*pages_per_split, +pages_per_split) of the pair.
    // Units are dealt to warps so that warp w of every CTA is busy before warp w+1 of any CTA.
    const int n_units = B * H_kv * max_splits;
    const int warps_total = kDecWarps * gridDim.x;
    bool failed = false;
    WarpAttn<D> A;
    A.init_lane(lane);

    for (int unit = warp * gridDim.x + blockIdx.x; unit < n_units && !failed; unit += warps_total) {
        const int pair = unit / max_splits;
        const int my_split = unit - pair * max_splits;
        const int i_lo = my_split * pages_per_split;
        if (i_lo >= k_max) continue;
        const int r = pair / H_kv, h = pair % H_kv;
        const size_t head0 = (size_t)r * H_q + h * G;
        int32_t *sel_row = sa.sel_idx + (size_t)pair * k_max;
        // Loads that depend on nothing go out first and travel together: the lengths, the selection
        // count, Q, and (when the caller supplies the list) the first chunk of selection entries.
        int first[kChunk / 32];
        A.load_q(q, head0, lane, G);
#pragma unroll
        for (int rep = 0; rep < kChunk / 32; ++rep) {
            const int i = i_lo + rep * 32 + lane;
            first[rep] = i < min(i_lo + pages_per_split, k_max) ? __ldg(sel_row + i) : -1;
        }
        const int len = __ldg(seq_lens + r);
        const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
        int cnt = __ldg(sa.sel_cnt + pair);
        if (cnt > k_max) {
            if (lane == 0) atomicOr(status, SE_DEV_BAD_SELECTION);
            cnt = k_max;
        }
        if (cnt <= 0 || n_r == 0) {
            if (my_split == 0) {      // the first split of the pair reports "nothing attended"
                for (int g = 0; g < G; ++g) {
                    float *o = out + (head0 + g) * D;
                    for (int c = lane; c < D; c += 32) o[c] = 0.f;
                    if (lane == 0) lse[head0 + g] = -INFINITY;
                }
            }
            continue;
        }
        if (i_lo >= cnt) continue;
        const int i_hi = min(min(i_lo + pages_per_split, k_max), cnt);
        const int n_split = (cnt + pages_per_split - 1) / pages_per_split;   // splits of this pair that hold pages

        A.reset();
        a.zrow = zbuf != nullptr ? zbuf + (size_t)pair * k_max * kPage * GP : nullptr;
        a.keys_row = kObserve ? tok_keys + (size_t)r * max_pages * kPage : nullptr;
        auto sel_at = [&](int i) { return __ldg(sel_row + i); };
        if (!attend_range<D, kObserve, true>(P, A, a, sel_at, first, i_lo, i_hi, r, h, len, n_r, lane)) {
            failed = true;
            break;
        }
        A.finish();

        if (n_split == 1) {
            if (head_ok) {
                const float inv = A.l_run > 0.f ? 1.f / A.l_run : 0.f;
                float *o = out + (head0 + gid) * D + 2 * tid4;
#pragma unroll
                for (int nt = 0; nt < C::NTILES; ++nt)
                    *reinterpret_cast<float2 *>(o + nt * 8) = make_float2(A.o_acc[nt][0] * inv, A.o_acc[nt][1] * inv);
                if (tid4 == 0) lse[head0 + gid] = A.l_run > 0.f ? (A.m_run + log2f(A.l_run)) * kLn2 : -INFINITY;
            }
            continue;
        }
        // ---- store the partial; combine_kernel merges the splits of a pair afterwards
        if (head_ok) {
            float *pr = partials + ((head0 + gid) * max_splits + my_split) * C::PSTRIDE;
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt)
                *reinterpret_cast<float2 *>(pr + nt * 8 + 2 * tid4) = make_float2(A.o_acc[nt][0], A.o_acc[nt][1]);
            if (tid4 == 0) {
                pr[D] = A.m_run;
                pr[D + 1] = A.l_run;
            }
        }
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        // bounded wait for whatever this warp still has in flight before the CTA can retire
        for (int s = 0; s < P.nstage; ++s) mbar_wait(P.bar0 + s * 8, (P.phases >> s) & 1u);
    }
}

// ---------------------------------------------------------------------------------
// decode_duo_kernel: two to four pairs per SM.  Two adjacent warps share a pair: each attends half of
// its selected pages, then the two exchange their statistics and half of their accumulators through
// shared memory (named barriers of 64 threads) and each writes half of the output channels.  Six to
// eight busy warps per SM with two stages each draw more bandwidth than three or four warps with
// five or six stages (measured with the gather probe on the same page lists: 81.9 us against 87.5 us
// for the 537 MB of config 3), and the halves even out the 4-against-3 pairs imbalance between CTAs.
// Slot s = warp / 2 of CTA b holds the pairs b + s*gridDim.x (+ 4*gridDim.x ...).
// ---------------------------------------------------------------------------------
constexpr int kDuoStages = 16;           // stages per CTA (D = 128): two per warp; three per warp were 5 % slower

__device__ __forceinline__ void duo_bar(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
decode_duo_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                  const uint16_t *__restrict__ q, const int32_t *__restrict__ page_table,
                  const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ sel_idx,
                  const int32_t *__restrict__ sel_cnt, float *__restrict__ out, float *__restrict__ lse,
                  float *__restrict__ zbuf, int B, int H_kv, int G, int GP, int max_pages, int P_phys, int k_max,
                  float scale_log2, uint32_t *status) {
    using C = DecCfg<D>;
    constexpr int STAGES = kDuoStages * (128 / D);
    constexpr int XPITCH = D / 2 + 8;            // floats per head row of the exchange area
    extern __shared__ uint8_t smem_dyn[];
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot = warp >> 1, half = warp & 1;
    const int pairs = B * H_kv;
    // every busy warp of the grid gets the same number of stages (that of the fullest CTAs)
    const int slots_max = min(kDecWarps / 2, (pairs + (int)gridDim.x - 1) / (int)gridDim.x);
    const bool busy = slot * (int)gridDim.x + (int)blockIdx.x < pairs;
    WarpPipe P;
    P.nstage = busy ? min(C::MAXST, STAGES / (2 * slots_max)) : 0;
    const int nst = min(C::MAXST, STAGES / (2 * slots_max));
    uint8_t *ring = smem_al + (size_t)(warp * nst) * C::STAGEB;
    uint8_t *ring_partner = smem_al + (size_t)((warp ^ 1) * nst) * C::STAGEB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + (size_t)STAGES * C::STAGEB) + warp * C::MAXST;
    if (lane == 0) {
        for (int s = 0; s < P.nstage; ++s) mbar_init(smem_u32(&bars[s]), 2);
        mbar_fence_init();
    }
    __syncwarp();
    P.bar0 = smem_u32(&bars[0]);
    P.ring0 = smem_u32(ring);
    P.phases = 0;
    P.stage_c = 0;
    P.stage_i = 0;
    uint8_t *lists = smem_al + (size_t)STAGES * C::STAGEB + kDecWarps * C::MAXST * 8;
    P.ent_y = reinterpret_cast<int *>(lists) + warp * 3 * kChunk;
    P.ent_info = P.ent_y + kChunk;
    P.ent_b = P.ent_info + kChunk;
    uint8_t *zero_bytes = lists + (size_t)kDecWarps * 3 * kChunk * sizeof(int);
    if (threadIdx.x < 4) reinterpret_cast<uint32_t *>(zero_bytes)[threadIdx.x] = 0u;
    __syncthreads();

    AttendArgs a;
    a.k_map = &k_map;
    a.v_map = &v_map;
    a.page_table = page_table;
    a.max_pages = max_pages;
    a.H_kv = H_kv;
    a.P_phys = P_phys;
    a.G = G;
    a.GP = GP;
    a.scale_log2 = scale_log2;
    a.zero_chunk = smem_u32(zero_bytes);
    a.status = status;
    a.keys_row = nullptr;

    const int H_q = H_kv * G;
    const int gid = lane >> 2, tid4 = lane & 3;
    const bool head_ok = gid < G;
    const int hs = (k_max + 1) / 2;              // where the second half starts when the whole row is selected
    bool failed = false;
    WarpAttn<D> A;
    A.init_lane(lane);
    float *xme = reinterpret_cast<float *>(ring), *xpa = reinterpret_cast<float *>(ring_partner);

    for (int pair = slot * gridDim.x + blockIdx.x; pair < pairs && !failed; pair += (kDecWarps / 2) * gridDim.x) {
        const int r = pair / H_kv, h = pair % H_kv;
        const size_t head0 = (size_t)r * H_q + h * G;
        const int32_t *sel_row = sel_idx + (size_t)pair * k_max;
        // loads that depend on nothing travel together: Q, the lengths, the count and the first chunk of this
        // half's entries - where the half starts if the whole row is selected (the usual case)
        const int i_sp = half * hs;
        int first[kChunk / 32];
        A.load_q(q, head0, lane, G);
#pragma unroll
        for (int rep = 0; rep < kChunk / 32; ++rep) {
            const int i = i_sp + rep * 32 + lane;
            first[rep] = i < min(i_sp + hs, k_max) ? __ldg(sel_row + i) : -1;
        }
        const int len = __ldg(seq_lens + r);
        const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
        int cnt = __ldg(sel_cnt + pair);
        if (cnt > k_max) {
            if (lane == 0) atomicOr(status, SE_DEV_BAD_SELECTION);
            cnt = k_max;
        }
        if (cnt <= 0 || n_r == 0) {               // both warps of the pair take this branch
            if (half == 0) {
                for (int g = 0; g < G; ++g) {
                    float *o = out + (head0 + g) * D;
                    for (int c = lane; c < D; c += 32) o[c] = 0.f;
                    if (lane == 0) lse[head0 + g] = -INFINITY;
                }
            }
            continue;
        }
        const int hc = (cnt + 1) / 2;
        const int i_lo = half ? hc : 0, i_hi = half ? cnt : hc;
        A.reset();
        a.zrow = zbuf != nullptr ? zbuf + (size_t)pair * k_max * kPage * GP : nullptr;
        if (i_lo < i_hi) {
            auto sel_at = [&](int i) { return __ldg(sel_row + i); };
            if (!attend_range<D, false, true>(P, A, a, sel_at, first, i_lo, i_hi, r, h, len, n_r, lane, i_lo == i_sp))
                failed = true;                    // still goes through the pair's barriers below
        }
        A.finish();

        // ---- the two halves meet: statistics, then the accumulators of the channels the partner finishes
        const int bar_id = 1 + slot;
        if (tid4 == 0) {
            xme[gid] = A.m_run;
            xme[8 + gid] = A.l_run;
        }
        duo_bar(bar_id);
        const float mo = xpa[gid], lo = xpa[8 + gid];
        const float mstar = fmaxf(A.m_run, mo);
        const float ws = (A.m_run == -INFINITY) ? 0.f : exp2f(A.m_run - mstar);
        const float wo = (mo == -INFINITY) ? 0.f : exp2f(mo - mstar);
        const float lsum = ws * A.l_run + wo * lo;
        constexpr int HT = C::NTILES / 2;        // half 0 finishes the n-tiles [0, HT), half 1 the others
        float *dst = xme + 16 + gid * XPITCH + 2 * tid4;
        if (half == 0) {
#pragma unroll
            for (int t = 0; t < HT; ++t)
                *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(A.o_acc[HT + t][0] * ws, A.o_acc[HT + t][1] * ws);
        } else {
#pragma unroll
            for (int t = 0; t < HT; ++t)
                *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(A.o_acc[t][0] * ws, A.o_acc[t][1] * ws);
        }
        duo_bar(bar_id);
        if (head_ok) {
            const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
            const float *src = xpa + 16 + gid * XPITCH + 2 * tid4;
            float *o = out + (head0 + gid) * D + 2 * tid4;
            if (half == 0) {
#pragma unroll
                for (int t = 0; t < HT; ++t) {
                    const float2 v = *reinterpret_cast<const float2 *>(src + t * 8);
                    *reinterpret_cast<float2 *>(o + t * 8) = make_float2((A.o_acc[t][0] * ws + v.x) * inv, (A.o_acc[t][1] * ws + v.y) * inv);
                }
                if (tid4 == 0) lse[head0 + gid] = lsum > 0.f ? (mstar + log2f(lsum)) * kLn2 : -INFINITY;
            } else {
#pragma unroll
                for (int t = 0; t < HT; ++t) {
                    const float2 v = *reinterpret_cast<const float2 *>(src + t * 8);
                    *reinterpret_cast<float2 *>(o + (HT + t) * 8) =
                        make_float2((A.o_acc[HT + t][0] * ws + v.x) * inv, (A.o_acc[HT + t][1] * ws + v.y) * inv);
                }
            }
        }
        duo_bar(bar_id);          // the partner has read this warp's area: the ring may be refilled
        fence_proxy_async();      // ... by tensor copies, after these ordinary stores
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        for (int s = 0; s < P.nstage; ++s) mbar_wait(P.bar0 + s * 8, (P.phases >> s) & 1u);
    }
}

// ---------------------------------------------------------------------------------
// Scoring phase of the fused step (Appendix A, Quest summary and score equations): the CTA scores the
// logical pages [b_lo, b_hi) of its pair and writes the fp32 scores to the pair's score row.  Same
// arithmetic as score_kernel (se_select.cu): sum_c max(q m, q M) = sum_c (q^- m + q^+ M) as a dense
// [16 pages x 2D] . [2D x G] contraction per batch of 16 summaries, which arrive by 1-D bulk copies
// into two padded buffers per warp (the warp's share of the still empty ring).  Warp w takes the
// batches w, w+8, ... of the CTA's range, eight of them at a time: their page-table entries are
// fetched together, then the batches run through the double buffer.  The summary of the request's
// newest page is recomputed from K on the spot and written back, as se_meta_update would.
// Returns false when a bounded wait gave up.
// ---------------------------------------------------------------------------------
struct FusedScoreArgs {
    const uint8_t *meta;     // [P_phys][H_kv][2][D] bf16 (read; the newest page's entry is written)
    const uint8_t *k_cache;  // [P_phys][H_kv][16][D] bf16
    float *scores;           // [pairs][pitch]
    int pitch;
    float scale;
};

template <int D>
__device__ __forceinline__ bool cta_score_range(uint8_t *wbuf, uint32_t bar0, int *pids, const uint16_t *__restrict__ q,
                                                size_t head0, int G, const FusedScoreArgs &fs,
                                                const int32_t *__restrict__ pt_row, int n_r, int len, int b_lo, int b_hi,
                                                int hh, int H_kv, int P_phys, float *score_row, uint32_t *status,
                                                int warp, int lane) {
    constexpr int PHB = 4 * D;                   // bytes of one page summary (min row, max row)
    constexpr int PITCH = PHB + 16;              // padded: conflict-free ldmatrix
    constexpr int BUF = kPage * PITCH;
    constexpr int KSTEPS = 2 * D / 16;
    constexpr int NBC = 8;                       // batches whose page-table entries are fetched together
    const int gid = lane >> 2, tid4 = lane & 3;
    const uint32_t buf0 = smem_u32(wbuf);
    const int nb = (b_hi - b_lo + kPage - 1) / kPage;            // batches of the CTA
    const int nbw = nb > warp ? (nb - warp + kDecWarps - 1) / kDecWarps : 0;   // batches of this warp
    if (nbw == 0) return true;

    // B operand: column n = query head n of the group (zero for n >= G); rows k < D carry q^- (they meet
    // the min row), rows k >= D carry q^+ (they meet the max row)
    uint32_t bfrag[KSTEPS][2];
    {
        const uint16_t *src = q + (head0 + (gid < G ? gid : 0)) * D + 2 * tid4;
#pragma unroll
        for (int sidx = 0; sidx < D / 16; ++sidx) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(src + sidx * 16 + 8 * j));
                if (gid >= G) w = 0u;
                const uint32_t negmask = ((w >> 15) & 0x00010001u) * 0xffffu;   // all-ones per negative half
                bfrag[sidx][j] = w & negmask;
                bfrag[D / 16 + sidx][j] = w & ~negmask;
            }
        }
    }
    const uint32_t lm_off = (uint32_t)(((lane & 7) + 8 * ((lane >> 3) & 1)) * PITCH + (lane >> 4) * 16);
    uint32_t phases = 0u;
    const int newest = n_r - 1;                  // the page whose summary is recomputed from K
    const int nv_newest = min(kPage, len - newest * kPage);

    for (int j0 = 0; j0 < nbw; j0 += NBC) {
        const int nc = min(NBC, nbw - j0);
        // page-table entries of this chunk of batches: entry e = batch (e >> 4), page offset (e & 15)
#pragma unroll
        for (int rep = 0; rep < NBC * kPage / 32; ++rep) {
            const int e = rep * 32 + lane;
            const int page = b_lo + (warp + kDecWarps * (j0 + (e >> 4))) * kPage + (e & 15);
            int pid = -1;
            if ((e >> 4) < nc && page < b_hi) pid = __ldg(pt_row + page);
            if (pid >= P_phys) {
                atomicOr(status, SE_DEV_BAD_PAGE_ID);
                pid = -1;
            }
            pids[e] = pid;
        }
        __syncwarp();
        auto issue = [&](int j) {                // batch j of the chunk into buffer j & 1
            const int page = b_lo + (warp + kDecWarps * (j0 + j)) * kPage + lane;
            int pid = lane < kPage ? pids[j * kPage + lane] : -1;
            if (page == newest) pid = -1;        // summarised from K instead of copied
            const unsigned valid = __ballot_sync(kFull, pid >= 0);
            const uint32_t bar = bar0 + (j & 1) * 8;
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(valid) * PHB);
            __syncwarp();
            if (pid >= 0)
                bulk_g2s(buf0 + (j & 1) * BUF + lane * PITCH, fs.meta + ((size_t)pid * H_kv + hh) * PHB, PHB, bar);
        };
        issue(0);
        if (nc > 1) issue(1);
        for (int j = 0; j < nc; ++j) {
            const int slot = j & 1;
            const int page0 = b_lo + (warp + kDecWarps * (j0 + j)) * kPage;
            if (!mbar_wait(bar0 + slot * 8, (phases >> slot) & 1u)) return false;
            phases ^= 1u << slot;
            const int my_pid = lane < kPage ? pids[j * kPage + lane] : -1;
            if (newest >= page0 && newest < page0 + kPage) {
                // the newest page of the request: summary from K (all kv-heads' pages are contiguous per head)
                const int fl = newest - page0;
                const int fpid = __shfl_sync(kFull, my_pid, fl);
                if (fpid >= 0) {
                    constexpr int LPR = D / 8, TPP = 32 / LPR, KROWS = kPage / TPP;
                    const int tg = lane / LPR, lr = lane % LPR;
                    const uint4 *kp = reinterpret_cast<const uint4 *>(fs.k_cache) + ((size_t)fpid * H_kv + hh) * (kPage * D / 8);
                    uint4 w[KROWS];
#pragma unroll
                    for (int i = 0; i < KROWS; ++i) {
                        const int t = i * TPP + tg;
                        w[i] = __ldg(kp + (t < nv_newest ? t : 0) * LPR + lr);      // rows past the length repeat row 0
                    }
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
                    if (tg < 2) {
                        const uint4 val = tg == 0 ? mn : mx;
                        uint4 *gp = reinterpret_cast<uint4 *>(const_cast<uint8_t *>(fs.meta)) + ((size_t)fpid * H_kv + hh) * (2 * D / 8);
                        gp[tg * LPR + lr] = val;
                        sts128(buf0 + slot * BUF + fl * PITCH + (tg * LPR + lr) * 16, val);
                    }
                    __syncwarp();
                }
            }
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t a_base = buf0 + slot * BUF + lm_off;
#pragma unroll
            for (int sidx = 0; sidx < KSTEPS; ++sidx) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4(a_base + sidx * 32, a0, a1, a2, a3);
                mma_bf16_16816(acc, a0, a1, a2, a3, bfrag[sidx][0], bfrag[sidx][1]);
            }
            // acc[0],acc[1]: page gid, heads 2*tid4, 2*tid4+1;  acc[2],acc[3]: page gid+8, same heads
            const float ninf = -INFINITY;
            float s_lo = fmaxf(2 * tid4 < G ? acc[0] : ninf, 2 * tid4 + 1 < G ? acc[1] : ninf);
            float s_hi = fmaxf(2 * tid4 < G ? acc[2] : ninf, 2 * tid4 + 1 < G ? acc[3] : ninf);
            s_lo = fmaxf(s_lo, __shfl_xor_sync(kFull, s_lo, 1));
            s_hi = fmaxf(s_hi, __shfl_xor_sync(kFull, s_hi, 1));
            s_lo = fmaxf(s_lo, __shfl_xor_sync(kFull, s_lo, 2));
            s_hi = fmaxf(s_hi, __shfl_xor_sync(kFull, s_hi, 2));
            const int pid_lo = __shfl_sync(kFull, my_pid, gid);
            const int pid_hi = __shfl_sync(kFull, my_pid, gid + 8);
            if (tid4 == 0) {
                if (page0 + gid < b_hi) score_row[page0 + gid] = (pid_lo >= 0) ? s_lo * fs.scale : ninf;
                if (page0 + gid + 8 < b_hi) score_row[page0 + gid + 8] = (pid_hi >= 0) ? s_hi * fs.scale : ninf;
            }
            __syncwarp();        // every lane is done reading the buffer before it is refilled
            if (j + 2 < nc) {
                fence_proxy_async();             // the newest page's summary may have been stored with ordinary stores
                issue(j + 2);
            }
        }
        __syncwarp();
    }
    return true;
}

// ---------------------------------------------------------------------------------
// decode_cta_kernel: one CTA per (pair, CTA-split); gridDim.x = pairs * cpp.
//   1. selection list of the pair in shared memory: the caller's, or (kSelect) the CTA's own top-k of
//      the score row (every CTA of a pair computes the same list; CTA-split 0 writes it out);
//   2. the cnt selected pages are cut into n_active = ceil(cnt / ceil(cnt / cpp)) equal CTA slices, a
//      slice into eight warp ranges; each warp attends its range (attend_range);
//   3. the warps' partials are merged through shared memory (weights 2^(m_w - m*));
//   4. one active CTA: out / lse are final.  Several: every CTA stores its partial; with merge_here (the
//      CTAs are a cluster) they meet at a cluster barrier, after which each computes the pair's final
//      log-sum-exp, its share of the final output and the H2O update of its own tokens; without it
//      combine_kernel merges the partials.
// ---------------------------------------------------------------------------------
template <int D>
struct CtaCfg {
    using C = DecCfg<D>;
    static constexpr int STAGES_PER_WARP = C::CTA_STAGES_SPLIT / kDecWarps;
    static constexpr int RED_PITCH = D + 8;                    // floats per (warp, head) row of the merge buffer
    static constexpr size_t kStages = (size_t)C::CTA_STAGES_SPLIT * C::STAGEB;
    static constexpr size_t kBars = kStages;
    static constexpr size_t kLists = kBars + (size_t)kDecWarps * C::MAXST * 8;
    static constexpr size_t kZero = kLists + (size_t)kDecWarps * 3 * kChunk * sizeof(int);
    static constexpr size_t kSmall = kZero + 16;               // merge statistics: 4 * 64 floats
    static constexpr size_t kSel = kSmall + 4 * 64 * sizeof(float);
    static_assert(sizeof(TopkScratch) + cta_topk_key_words(8192, kDecWarps * 32) * 4 <= kStages,
                  "the top-k keys and scratch live in the empty ring");
    static_assert((size_t)kDecWarps * 8 * RED_PITCH * sizeof(float) <= kStages, "merge buffer lives in the drained ring");
    static size_t smem_bytes(int k_max) { return kSel + (size_t)k_max * sizeof(int) + 1024; }
};

// kFused (implies kSelect): the CTAs of a pair form a thread-block cluster and score the pair's pages
// first (cta_score_range), each its share; a cluster barrier later every CTA reads the whole score row.
template <int D, bool kSelect, bool kFused>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
decode_cta_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                  const uint16_t *__restrict__ q, const int32_t *__restrict__ page_table,
                  const int32_t *__restrict__ seq_lens, const SelectArgs sa, const FusedScoreArgs fs,
                  float *__restrict__ out, float *__restrict__ lse, float *partials, float *zbuf,
                  float *__restrict__ score_accum, int H_kv, int G, int GP, int max_pages, int P_phys, int k_max,
                  int cpp, int merge_here, float scale_log2, uint32_t *status) {
    using C = DecCfg<D>;
    using L = CtaCfg<D>;
    extern __shared__ uint8_t smem_dyn[];
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gid = lane >> 2, tid4 = lane & 3;
    const int pair = blockIdx.x / cpp, cs = blockIdx.x - pair * cpp;
    const int r = pair / H_kv, h = pair - r * H_kv;
    const int H_q = H_kv * G;
    const size_t head0 = (size_t)r * H_q + h * G;

    WarpPipe P;
    P.nstage = L::STAGES_PER_WARP;
    uint8_t *ring = smem_al + (size_t)(warp * L::STAGES_PER_WARP) * C::STAGEB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + L::kBars) + warp * C::MAXST;
    if (lane == 0) {
        for (int s = 0; s < P.nstage; ++s) mbar_init(smem_u32(&bars[s]), 2);
        if (kFused) {                             // the scoring phase has two buffers with a barrier each
            mbar_init(smem_u32(&bars[C::MAXST - 2]), 1);
            mbar_init(smem_u32(&bars[C::MAXST - 1]), 1);
        }
        mbar_fence_init();
    }
    __syncwarp();
    P.bar0 = smem_u32(&bars[0]);
    P.ring0 = smem_u32(ring);
    P.phases = 0;
    P.stage_c = 0;
    P.stage_i = 0;
    P.ent_y = reinterpret_cast<int *>(smem_al + L::kLists) + warp * 3 * kChunk;
    P.ent_info = P.ent_y + kChunk;
    P.ent_b = P.ent_info + kChunk;
    if (tid < 4) reinterpret_cast<uint32_t *>(smem_al + L::kZero)[tid] = 0u;
    float *s_m = reinterpret_cast<float *>(smem_al + L::kSmall);      // [warp][head]
    float *s_l = s_m + 64;                                            // [warp][head]
    float *s_M = s_l + 64;                                            // [head] merged maximum
    float *s_L = s_M + 64;                                            // [head] merged sum
    int *list = reinterpret_cast<int *>(smem_al + L::kSel);

    const int len = __ldg(seq_lens + r);
    const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
    int32_t *sel_row = sa.sel_idx + (size_t)pair * k_max;
    if (kFused) {
        // this CTA's share of the pair's pages, in whole batches of 16
        const int per = ((n_r + cpp - 1) / cpp + kPage - 1) / kPage * kPage;
        const int b_lo = min(n_r, cs * per), b_hi = min(n_r, b_lo + per);
        const bool ok = cta_score_range<D>(ring, smem_u32(&bars[C::MAXST - 2]), P.ent_y, q, head0, G, fs,
                                           page_table + (size_t)r * max_pages, n_r, len, b_lo, b_hi, h, H_kv, P_phys,
                                           fs.scores + (size_t)pair * fs.pitch, status, warp, lane);
        if (!ok && lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        // every CTA of the pair has written its scores before any of them reads the row
        __threadfence();
        if (cpp > 1) {
            asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
            asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        } else {
            __syncthreads();
        }
        fence_proxy_async();
    }
    int cnt;
    if (kSelect) {
        TopkScratch &S = *reinterpret_cast<TopkScratch *>(smem_al);
        uint32_t *keys = reinterpret_cast<uint32_t *>(smem_al + ((sizeof(TopkScratch) + 15) & ~(size_t)15));
        cnt = cta_topk<kDecWarps * 32>(sa.scores + (size_t)pair * sa.pitch, n_r, sa.k_pages, k_max, sa.sink, sa.recent,
                                       keys, S, list, cs == 0 ? sel_row : nullptr);
        if (cs == 0 && tid == 0) sa.sel_cnt[pair] = cnt;
        fence_proxy_async();          // the scratch was written with ordinary stores; tensor copies refill it
    } else {
        cnt = __ldg(sa.sel_cnt + pair);
        if (cnt > k_max) {
            if (tid == 0) atomicOr(status, SE_DEV_BAD_SELECTION);
            cnt = k_max;
        }
        for (int i = tid; i < cnt; i += kDecWarps * 32) list[i] = __ldg(sel_row + i);
    }
    __syncthreads();
    if (cnt <= 0 || n_r == 0) {
        if (cs == 0) {
            for (int e = tid; e < G * D; e += kDecWarps * 32) out[head0 * D + e] = 0.f;
            if (tid < G) lse[head0 + tid] = -INFINITY;
        }
        return;
    }
    const int per_cta = (cnt + cpp - 1) / cpp;
    const int n_active = (cnt + per_cta - 1) / per_cta;
    const bool single = n_active == 1;
    // merge_here: the CTAs of the pair are a cluster and meet at a cluster barrier below, so a CTA without
    // pages (cs >= n_active) stays until then; otherwise (partials merged by combine_kernel) it is done.
    const bool active = cs < n_active;
    if (!active && (single || !merge_here)) return;
    const int c_lo = min(cnt, cs * per_cta), c_hi = min(cnt, c_lo + per_cta);
    float *s_lse2 = s_l;                  // final log2-sum-exp per head (the per-warp sums are dead by then)

    if (active) {
        const int per_warp = (c_hi - c_lo + kDecWarps - 1) / kDecWarps;
        const int i_lo = min(c_hi, c_lo + warp * per_warp), i_hi = min(c_hi, i_lo + per_warp);

        AttendArgs a;
        a.k_map = &k_map;
        a.v_map = &v_map;
        a.page_table = page_table;
        a.max_pages = max_pages;
        a.H_kv = H_kv;
        a.P_phys = P_phys;
        a.G = G;
        a.GP = GP;
        a.scale_log2 = scale_log2;
        a.zero_chunk = smem_u32(smem_al + L::kZero);
        a.status = status;
        a.zrow = zbuf != nullptr ? zbuf + (size_t)pair * k_max * kPage * GP : nullptr;
        a.keys_row = nullptr;

        WarpAttn<D> A;
        A.init_lane(lane);
        A.reset();
        bool ok = true;
        if (i_lo < i_hi) {
            A.load_q(q, head0, lane, G);
            const int none[kChunk / 32] = {};
            ok = attend_range<D, false, false>(P, A, a, [&](int i) { return list[i]; }, none, i_lo, i_hi, r, h, len,
                                               n_r, lane);
        }
        if (!ok) {
            if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
            for (int s = 0; s < P.nstage; ++s) mbar_wait(P.bar0 + s * 8, (P.phases >> s) & 1u);
        }
        A.finish();

        // ---- merge of the eight warps through shared memory.  Rows past the group hold zero queries:
        // finite values that nobody reads.
        if (tid4 == 0) {
            s_m[warp * 8 + gid] = A.m_run;
            s_l[warp * 8 + gid] = A.l_run;
        }
        __syncthreads();                  // every warp has drained its ring: it becomes the merge buffer
        float mstar = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) mstar = fmaxf(mstar, s_m[w * 8 + gid]);
        float lsum = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) {
            const float mw = s_m[w * 8 + gid];
            lsum += (mw == -INFINITY) ? 0.f : exp2f(mw - mstar) * s_l[w * 8 + gid];
        }
        const float wgt = (A.m_run == -INFINITY) ? 0.f : exp2f(A.m_run - mstar);
        float *red = reinterpret_cast<float *>(smem_al);
        {
            float *dst = red + (size_t)(warp * 8 + gid) * L::RED_PITCH + 2 * tid4;
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt)
                *reinterpret_cast<float2 *>(dst + nt * 8) = make_float2(A.o_acc[nt][0] * wgt, A.o_acc[nt][1] * wgt);
        }
        if (warp == 0 && tid4 == 0) {
            s_M[gid] = mstar;
            s_L[gid] = lsum;
        }
        __syncthreads();
        for (int e = tid; e < G * D; e += kDecWarps * 32) {
            const int g = e / D, c = e - g * D;
            float acc = 0.f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) acc += red[(size_t)(w * 8 + g) * L::RED_PITCH + c];
            if (single) {
                const float lg = s_L[g];
                out[(head0 + g) * D + c] = lg > 0.f ? acc / lg : 0.f;
            } else {
                partials[((head0 + g) * cpp + cs) * C::PSTRIDE + c] = acc;
            }
        }
        if (tid < G) {
            const float lg = s_L[tid], mg = s_M[tid];
            if (single) {
                const float l2 = lg > 0.f ? mg + log2f(lg) : -INFINITY;
                lse[head0 + tid] = l2 * kLn2;
                s_lse2[tid] = l2;
            } else {
                float *pr = partials + ((head0 + tid) * cpp + cs) * C::PSTRIDE;
                pr[D] = mg;
                pr[D + 1] = lg;
            }
        }
    }
    if (!single) {
        if (!merge_here) return;          // combine_kernel merges the partials (and applies the H2O update)
        // ---- several CTAs share the pair: after a cluster barrier every one of them knows all partials.
        // Each computes the pair's final statistics (cheap), a share of the final output, and - below -
        // the H2O update of the tokens it attended itself.
        __threadfence();
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (!active) return;
        // (the partials are in L2; every thread issues all the loads it needs before it uses one, so the
        // merge costs one round trip and not one per CTA of the pair)
        constexpr int MAXC = 8;                  // a cluster has at most 8 CTAs
        if (tid < G) {
            const float *pr = partials + ((head0 + tid) * cpp) * C::PSTRIDE;
            float ms[MAXC], ls[MAXC];
#pragma unroll
            for (int s = 0; s < MAXC; ++s) {
                ms[s] = -INFINITY;
                ls[s] = 0.f;
                if (s < n_active) {
                    ms[s] = __ldcg(pr + (size_t)s * C::PSTRIDE + D);
                    ls[s] = __ldcg(pr + (size_t)s * C::PSTRIDE + D + 1);
                }
            }
            float mg = -INFINITY, lg = 0.f;
#pragma unroll
            for (int s = 0; s < MAXC; ++s) mg = fmaxf(mg, ms[s]);
#pragma unroll
            for (int s = 0; s < MAXC; ++s)
                if (ms[s] != -INFINITY) lg += exp2f(ms[s] - mg) * ls[s];
            const float l2 = lg > 0.f ? mg + log2f(lg) : -INFINITY;
            s_lse2[tid] = l2;
            if (cs == 0) lse[head0 + tid] = l2 * kLn2;
        }
        for (int e = cs * (kDecWarps * 32) + tid; e < G * D; e += n_active * kDecWarps * 32) {
            const int g = e / D, c = e - g * D;
            const float *pr = partials + ((head0 + g) * cpp) * C::PSTRIDE;
            float ms[MAXC], ls[MAXC], vs[MAXC];
#pragma unroll
            for (int s = 0; s < MAXC; ++s) {
                ms[s] = -INFINITY;
                ls[s] = 0.f;
                vs[s] = 0.f;
                if (s < n_active) {
                    ms[s] = __ldcg(pr + (size_t)s * C::PSTRIDE + D);
                    ls[s] = __ldcg(pr + (size_t)s * C::PSTRIDE + D + 1);
                    vs[s] = __ldcg(pr + (size_t)s * C::PSTRIDE + c);
                }
            }
            float mg = -INFINITY, lg = 0.f, acc = 0.f;
#pragma unroll
            for (int s = 0; s < MAXC; ++s) mg = fmaxf(mg, ms[s]);
#pragma unroll
            for (int s = 0; s < MAXC; ++s) {
                if (ms[s] != -INFINITY) {
                    const float wgt = exp2f(ms[s] - mg);
                    lg += wgt * ls[s];
                    acc += wgt * vs[s];
                }
            }
            out[(head0 + g) * D + c] = lg > 0.f ? acc / lg : 0.f;
        }
        __syncthreads();                  // s_lse2
    } else {
        __syncthreads();                  // s_lse2
    }
    if (score_accum == nullptr || !merge_here) return;

    // ---- H2O epilogue (Appendix A, H2O accumulated-score equation) for the tokens this CTA attended:
    // score_accum[slot] += sum over the group's heads of 2^(z - lse2); their logits were written by this
    // CTA's own warps.
    // Four tokens per thread and round: their page-table entries and logits are fetched together, and
    // the sum goes out as a reduction (nothing waits for the old value).
    constexpr int EU = 4;
    for (int e0 = tid; e0 < (c_hi - c_lo) * kPage; e0 += EU * kDecWarps * 32) {
        int pid[EU], tt[EU];
        float zz[EU][8];
#pragma unroll
        for (int u = 0; u < EU; ++u) {
            const int e = e0 + u * kDecWarps * 32;
            pid[u] = -1;
            tt[u] = 0;
#pragma unroll
            for (int gg = 0; gg < 8; ++gg) zz[u][gg] = -INFINITY;
            if (e < (c_hi - c_lo) * kPage) {
                const int i = c_lo + e / kPage, t = e % kPage;
                const int b = list[i];
                if (b >= 0 && b < n_r && t < min(kPage, len - b * kPage)) {
                    pid[u] = __ldg(page_table + (size_t)r * max_pages + b);
                    tt[u] = t;
                    const float *z = zbuf + (((size_t)pair * k_max + i) * kPage + t) * GP;
#pragma unroll
                    for (int gg = 0; gg < 8; ++gg)
                        if (gg < G) zz[u][gg] = __ldcg(z + gg);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < EU; ++u) {
            if (pid[u] < 0 || pid[u] >= P_phys) continue;
            float add = 0.f;
#pragma unroll
            for (int gg = 0; gg < 8; ++gg)
                if (zz[u][gg] != -INFINITY) add += exp2f(zz[u][gg] - s_lse2[gg]);
            atomicAdd(score_accum + ((size_t)pid[u] * H_kv + h) * kPage + tt[u], add);
        }
    }
}

// combine_kernel: one CTA per (request, kv-head) pair, one warp per query head of the group.
//   1. LSE merge of the pair's split partials (skipped when the pair had a single split, whose
//      warp already wrote out/lse): m* = max_s m_s, L = sum_s 2^(m_s-m*) l_s,
//      out = sum_s 2^(m_s-m*) acc_s / L, lse = (m* + log2 L) ln 2.  Lane s fetches (m_s, l_s),
//      the weights follow from warp reductions, then each lane sums four channels with the
//      loads of eight splits in flight together.
//      cpp > 0: the partials come from decode_cta_kernel, whose split count follows from the pair's
//      page count (n_split = ceil(cnt / ceil(cnt / cpp))); merged != 0: out/lse are final already.
//   2. H2O epilogue (zbuf != NULL): score_accum[pid,h,t] += sum_g 2^(z2[g] - lse_g*log2e) for
//      every attended token slot of the pair.  The slots of a pair are spread over gridDim.y
//      CTAs; each of them recomputes the pair's lse (the cheap half of the merge), only
//      blockIdx.y == 0 sums the accumulators and writes out/lse.
template <int D>
__global__ void __launch_bounds__(256)
combine_kernel(const float *__restrict__ partials, const float *__restrict__ zbuf,
               const int32_t *__restrict__ page_table, const int32_t *__restrict__ seq_lens,
               const int32_t *__restrict__ sel_idx, const int32_t *__restrict__ sel_cnt,
               float *__restrict__ out, float *__restrict__ lse, float *__restrict__ score_accum,
               int H_kv, int G, int GP, int max_pages, int P_phys, int k_max, int pages_per_split,
               int max_splits, const int32_t *__restrict__ tok_cnt, int cpp, int merged) {
    constexpr int PSTRIDE = D + 4;
    __shared__ float s_lse2[8];
    const int pair = blockIdx.x;
    const int r = pair / H_kv, h = pair % H_kv;
    const int H_q = H_kv * G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // token-granular decode (tok_cnt != NULL): the units are 16-token tiles of the request's token list
    const int cnt = tok_cnt ? min((tok_cnt[r] + kPage - 1) / kPage, k_max) : min(sel_cnt[pair], k_max);
    const int len = seq_lens[r];
    const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
    const bool nothing = cnt <= 0 || n_r == 0;
    if (cpp > 0 && !nothing) pages_per_split = (cnt + cpp - 1) / cpp;
    const int n_split = (nothing || merged) ? 0 : (cnt + pages_per_split - 1) / pages_per_split;
    const int g = warp;                               // query head of the group handled by this warp
    const bool writer = blockIdx.y == 0;
    if (g < G) {
        const size_t head = (size_t)r * H_q + h * G + g;
        if (n_split > 1) {
            const float *pr0 = partials + head * max_splits * PSTRIDE;
            float mg = -INFINITY, lg = 0.f;
            float4 og = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s0 = 0; s0 < n_split; s0 += 32) {
                const int ns = min(32, n_split - s0);
                float ms = -INFINITY, ls = 0.f;
                if (lane < ns) {
                    ms = __ldcg(pr0 + (size_t)(s0 + lane) * PSTRIDE + D);
                    ls = __ldcg(pr0 + (size_t)(s0 + lane) * PSTRIDE + D + 1);
                }
                float mb = ms;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(kFull, mb, o));
                const float m_new = fmaxf(mg, mb);
                const float wl = (ms == -INFINITY) ? 0.f : exp2f(ms - m_new);      // weight of split s0+lane
                float lb = wl * ls;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lb += __shfl_xor_sync(kFull, lb, o);
                const float keep = (mg == -INFINITY) ? 0.f : exp2f(mg - m_new);
                lg = lg * keep + lb;
                og.x *= keep; og.y *= keep; og.z *= keep; og.w *= keep;
                mg = m_new;
                if (!writer) continue;                    // the other CTAs of the pair only need the lse
                for (int s = 0; s < ns; s += 8) {
                    float4 a[8];
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        a[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (s + t < ns && lane * 4 < D)
                            a[t] = __ldcg(reinterpret_cast<const float4 *>(pr0 + (size_t)(s0 + s + t) * PSTRIDE) + lane);
                    }
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const float ws = __shfl_sync(kFull, wl, (s + t) & 31);
                        og.x += ws * a[t].x; og.y += ws * a[t].y; og.z += ws * a[t].z; og.w += ws * a[t].w;
                    }
                }
            }
            const float inv = lg > 0.f ? 1.f / lg : 0.f;
            if (writer && lane * 4 < D)
                reinterpret_cast<float4 *>(out + head * D)[lane] = make_float4(og.x * inv, og.y * inv, og.z * inv, og.w * inv);
            const float l2 = lg > 0.f ? mg + log2f(lg) : -INFINITY;
            if (lane == 0) {
                if (writer) lse[head] = l2 * kLn2;
                s_lse2[g] = l2;
            }
        } else if (lane == 0) {
            s_lse2[g] = lse[head] * kLog2e;           // written by the decode kernel (single split / nothing)
        }
    }
    if (zbuf == nullptr || nothing) return;
    __syncthreads();
    for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < cnt * kPage; e += gridDim.y * blockDim.x) {
        const int i = e / kPage, t = e % kPage;
        const int b = sel_idx[(size_t)pair * k_max + i];
        if (b < 0 || b >= n_r) continue;
        const int pid = page_table[(size_t)r * max_pages + b];
        if (pid < 0 || pid >= P_phys) continue;
        if (t >= min(kPage, len - b * kPage)) continue;
        const float *z = zbuf + (((size_t)pair * k_max + i) * kPage + t) * GP;
        float add = 0.f;
        for (int gg = 0; gg < G; ++gg) {
            const float zz = z[gg];
            if (zz != -INFINITY) add += exp2f(zz - s_lse2[gg]);
        }
        score_accum[((size_t)pid * H_kv + h) * kPage + t] += add;
    }
}

// ---- tensor maps -------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// The cache viewed as a 3-D bf16 tensor [D/64 halves][P_phys*H_kv*16 rows][64 channels] (the half
// index is the slowest box dimension although its stride, 128 bytes, is the smaller one);
// box = 64 channels x 16 rows x all halves = one page of one head.
bool make_page_map(CUtensorMap *map, const void *base, const se_params &p) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)p.num_phys_pages * p.H_kv * kPage, (cuuint64_t)(p.D / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)p.D * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)kPage, (cuuint32_t)(p.D / 64)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t launch_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                          const int32_t *page_table, const int32_t *seq_lens, int32_t *sel_idx, int32_t *sel_cnt,
                          const SelectFromScores *from_scores, float *out, float *lse, float *score_accum,
                          uint32_t *tok_keys, void *workspace, const WorkspaceLayout &L, int stages,
                          cudaStream_t stream) {
    using C = DecCfg<D>;
    // an observation layer always runs on the warp-unit kernel (the only one that scores tokens)
    const DecodePlan plan = make_decode_plan(p, tok_keys != nullptr);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const int G = p.H_q / p.H_kv, GP = next_pow2(G);
    float *zbuf = score_accum ? reinterpret_cast<float *>(ws + L.zbuf) : nullptr;
    float *partials = reinterpret_cast<float *>(ws + L.partials);
    uint32_t *status = reinterpret_cast<uint32_t *>(ws + L.status);
    const bool select = from_scores != nullptr;
    SelectArgs sa = {};
    sa.sel_idx = sel_idx;
    sa.sel_cnt = sel_cnt;
    if (select) {
        sa.scores = reinterpret_cast<const float *>(ws + L.scores);
        sa.pitch = score_pitch(p);
        sa.k_pages = from_scores->k_pages;
        sa.sink = p.sink_pages;
        sa.recent = p.recent_pages;
    }
    cudaError_t e = cudaSuccess;
    if (stages & 1) {
        CUtensorMap k_map, v_map;
        if (!make_page_map(&k_map, k_cache, p) || !make_page_map(&v_map, v_cache, p)) return cudaErrorInvalidValue;
        const float scale_log2 = effective_scale(p) * kLog2e;
        if (plan.cta_units) {
            const size_t smem = CtaCfg<D>::smem_bytes(p.k_max);
            const bool fused = select && from_scores->meta != nullptr;
            auto kern = fused ? decode_cta_kernel<D, true, true>
                              : (select ? decode_cta_kernel<D, true, false> : decode_cta_kernel<D, false, false>);
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            FusedScoreArgs fs = {};
            if (fused) {
                fs.meta = static_cast<const uint8_t *>(from_scores->meta);
                fs.k_cache = static_cast<const uint8_t *>(k_cache);
                fs.scores = reinterpret_cast<float *>(ws + L.scores);
                fs.pitch = score_pitch(p);
                fs.scale = effective_scale(p);
            }
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(plan.grid);
            cfg.blockDim = dim3(kDecWarps * 32);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            if (plan.merge_in_kernel && plan.max_splits > 1) {   // the CTAs of a pair form a cluster (they share barriers)
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = plan.max_splits;
                attr[0].val.clusterDim.y = 1;
                attr[0].val.clusterDim.z = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
            }
            e = cudaLaunchKernelEx(&cfg, kern, k_map, v_map, (const uint16_t *)q, page_table, seq_lens, sa, fs, out, lse,
                                   partials, zbuf, plan.merge_in_kernel ? score_accum : (float *)nullptr, p.H_kv, G, GP,
                                   p.max_pages, p.num_phys_pages, p.k_max, plan.max_splits,
                                   plan.merge_in_kernel ? 1 : 0, scale_log2, status);
            if (e != cudaSuccess) return e;
        } else if (plan.duo) {
            if (select) return cudaErrorInvalidValue;         // only CTA units select in the kernel
            const size_t smem = (size_t)kDuoStages * (128 / D) * C::STAGEB + (size_t)kDecWarps * C::MAXST * 8 +
                                (size_t)kDecWarps * 3 * kChunk * sizeof(int) + 16 + 1024;
            auto kern = decode_duo_kernel<D>;
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            kern<<<plan.grid, kDecWarps * 32, smem, stream>>>(
                k_map, v_map, (const uint16_t *)q, page_table, seq_lens, sel_idx, sel_cnt, out, lse, zbuf, p.B, p.H_kv,
                G, GP, p.max_pages, p.num_phys_pages, p.k_max, scale_log2, status);
        } else {
            const size_t smem = (size_t)C::CTA_STAGES * C::STAGEB + (size_t)kDecWarps * C::MAXST * 8 +
                                (size_t)kDecWarps * 3 * kChunk * sizeof(int) + 16 + 1024;
            if (select) return cudaErrorInvalidValue;         // only CTA units select in the kernel
            auto kern = tok_keys ? decode_kernel<D, true> : decode_kernel<D, false>;
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            kern<<<plan.grid, kDecWarps * 32, smem, stream>>>(
                k_map, v_map, (const uint16_t *)q, page_table, seq_lens, sa, out, lse, partials, zbuf, tok_keys,
                p.B, p.H_kv, G, GP, p.max_pages, p.num_phys_pages, p.k_max, plan.pages_per_split, plan.max_splits,
                scale_log2, status);
        }
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (!(stages & 2)) return e;
    const bool merged = plan.max_splits == 1 || (plan.cta_units && plan.merge_in_kernel);
    if (plan.cta_units && plan.merge_in_kernel) return e;     // out/lse are final, the H2O epilogue ran in the kernel
    if (merged && !score_accum) return e;                     // out/lse are final and there is no epilogue
    // with the H2O epilogue the token slots of a pair (16 per selected page) are spread over
    // several CTAs, two slots per thread
    const int slot_ctas = score_accum ? (p.k_max * kPage + 511) / 512 : 1;
    combine_kernel<D><<<dim3(p.B * p.H_kv, slot_ctas), 256, 0, stream>>>(
        partials, zbuf, page_table, seq_lens, sel_idx, sel_cnt, out, lse, score_accum, p.H_kv, G, GP, p.max_pages,
        p.num_phys_pages, p.k_max, plan.pages_per_split, plan.max_splits, nullptr, plan.cta_units ? plan.max_splits : 0,
        merged ? 1 : 0);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------
// token_decode_kernel: attention of a sparse layer over a token set handed down by an observation
// layer (Appendix A, OmniKV reuse equation): all kv-heads of request r read the tokens
// tok_idx[r, 0..tok_cnt[r]) of this layer's own cache.  Same structure as decode_kernel - one
// (pair, split) unit per warp, stages shared out among the busy warps, MMA on ldmatrix fragments,
// online softmax - but a tile is 16 tokens from anywhere: 16 K rows and 16 V rows of D*2 bytes,
// fetched with one 1-D bulk copy each (lanes 0-15 the K rows, lanes 16-31 the V rows) into rows
// padded by 16 bytes (conflict-free ldmatrix without hardware swizzle).  Tokens that are out of
// range or whose page is absent are skipped (their columns are masked, their V rows cleared).
// ---------------------------------------------------------------------------------
constexpr int kTokChunk = 512;           // tokens whose rows are looked up at once (32 tiles)

template <int D>
struct TokCfg {
    static constexpr int ROWB = D * 2;                         // bytes of one K or V row
    static constexpr int PITCH = ROWB + 16;
    static constexpr int TILEB = kPage * PITCH;                // K (or V) rows of one tile
    static constexpr int STAGEB = 2 * TILEB;
    static constexpr int MAXST = 8;
    static constexpr int CTA_STAGES = 20 * (128 / D);
    static constexpr int KSTEPS = D / 16;
    static constexpr int NTILES = D / 8;
    static constexpr int PSTRIDE = D + 4;
};

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
token_decode_kernel(const uint16_t *__restrict__ q, const uint8_t *__restrict__ k_cache,
                    const uint8_t *__restrict__ v_cache, const int32_t *__restrict__ page_table,
                    const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ tok_idx,
                    const int32_t *__restrict__ tok_cnt, float *__restrict__ out, float *__restrict__ lse,
                    float *__restrict__ partials, int B, int H_kv, int G, int max_pages, int P_phys, int n_out,
                    int tiles_per_split, int max_splits, float scale_log2, uint32_t *status) {
    using C = TokCfg<D>;
    extern __shared__ __align__(128) uint8_t smem_tok[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_units = B * H_kv * max_splits;
    int busy = (n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    busy = busy < 1 ? 1 : (busy > kDecWarps ? kDecWarps : busy);
    const int nstage = warp < busy ? min(C::MAXST, C::CTA_STAGES / busy) : 0;
    uint8_t *ring = smem_tok + (size_t)(warp * nstage) * C::STAGEB;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_tok + (size_t)C::CTA_STAGES * C::STAGEB) + warp * C::MAXST;
    int *ent_row = reinterpret_cast<int *>(smem_tok + (size_t)C::CTA_STAGES * C::STAGEB + kDecWarps * C::MAXST * 8) +
                   warp * kTokChunk;
    if (lane == 0) {
        for (int s = 0; s < nstage; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_fence_init();
    }
    __syncwarp();
    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t ring0 = smem_u32(ring);
    const int H_q = H_kv * G;
    const int gid = lane >> 2, tid4 = lane & 3;
    const bool head_ok = gid < G;
    const int gw = warp * gridDim.x + blockIdx.x;
    const int warps_total = kDecWarps * gridDim.x;
    const int k_row = (lane & 7) + 8 * (lane >> 4);
    const int k_chunk_add = (lane >> 3) & 1;
    const int v_row = (lane & 7) + 8 * ((lane >> 3) & 1);
    const int v_chunk_add = lane >> 4;
    uint32_t phases = 0;
    int stage_c = 0, stage_i = 0;
    bool failed = false;

    for (int unit = gw; unit < n_units && !failed; unit += warps_total) {
        const int pair = unit / max_splits;
        const int my_split = unit - pair * max_splits;
        const int r = pair / H_kv, h = pair % H_kv;
        const int len = min(__ldg(seq_lens + r), max_pages * kPage);
        int cnt = __ldg(tok_cnt + r);
        if (cnt > n_out) {
            if (lane == 0) atomicOr(status, SE_DEV_BAD_SELECTION);
            cnt = n_out;
        }
        const int tiles = cnt > 0 ? (cnt + kPage - 1) / kPage : 0;
        const int n_split = (tiles + tiles_per_split - 1) / tiles_per_split;
        if (tiles == 0 || len <= 0) {
            if (my_split == 0) {
                for (int g = 0; g < G; ++g) {
                    float *o = out + ((size_t)r * H_q + h * G + g) * D;
                    for (int c = lane; c < D; c += 32) o[c] = 0.f;
                    if (lane == 0) lse[(size_t)r * H_q + h * G + g] = -INFINITY;
                }
            }
            continue;
        }
        if (my_split >= n_split) continue;
        const int e_lo = my_split * tiles_per_split * kPage;                       // entries of this unit
        const int e_hi = min(cnt, (my_split + 1) * tiles_per_split * kPage);

        uint32_t qa[C::KSTEPS][2];
        {
            const uint16_t *src = q + ((size_t)r * H_q + h * G + (head_ok ? gid : 0)) * D + 2 * tid4;
#pragma unroll
            for (int s = 0; s < C::KSTEPS; ++s) {
                const uint32_t w0 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16));
                const uint32_t w1 = __ldg(reinterpret_cast<const uint32_t *>(src + s * 16 + 8));
                qa[s][0] = head_ok ? w0 : 0u;
                qa[s][1] = head_ok ? w1 : 0u;
            }
        }
        float o_acc[C::NTILES][4];
#pragma unroll
        for (int nt = 0; nt < C::NTILES; ++nt) {
            o_acc[nt][0] = 0.f; o_acc[nt][1] = 0.f; o_acc[nt][2] = 0.f; o_acc[nt][3] = 0.f;
        }
        float m_run = -INFINITY, l_run = 0.f;

        for (int c_lo = e_lo; c_lo < e_hi && !failed; c_lo += kTokChunk) {
            // ---- row list of up to kTokChunk tokens: token -> page table -> row of the [pages*heads*16, D] view
            const int c_hi = min(e_hi, c_lo + kTokChunk);
            const int n_tiles = (c_hi - c_lo + kPage - 1) / kPage;
            // (all token loads first, then all page-table loads: two round trips for the whole chunk)
            int tk[kTokChunk / 32], pd[kTokChunk / 32];
#pragma unroll
            for (int rep = 0; rep < kTokChunk / 32; ++rep) {
                const int off = rep * 32 + lane;
                tk[rep] = (c_lo + off < c_hi) ? __ldg(tok_idx + (size_t)r * n_out + c_lo + off) : -2;
            }
#pragma unroll
            for (int rep = 0; rep < kTokChunk / 32; ++rep) {
                pd[rep] = -1;
                if (tk[rep] >= 0 && tk[rep] < len) pd[rep] = __ldg(page_table + (size_t)r * max_pages + (tk[rep] >> 4));
            }
#pragma unroll
            for (int rep = 0; rep < kTokChunk / 32; ++rep) {
                int row = -1;
                if (tk[rep] != -2 && (tk[rep] < 0 || tk[rep] >= len)) atomicOr(status, SE_DEV_BAD_SELECTION);
                else if (pd[rep] >= P_phys) atomicOr(status, SE_DEV_BAD_PAGE_ID);
                else if (pd[rep] >= 0) row = (pd[rep] * H_kv + h) * kPage + (tk[rep] & 15);
                ent_row[rep * 32 + lane] = row;
            }
            __syncwarp();
            int ce = 0, pe = 0;                      // tiles of this chunk consumed / issued
            auto top_up = [&]() {
                while (pe < n_tiles && pe < ce + nstage) {
                    const int row = ent_row[pe * kPage + (lane & 15)];
                    const unsigned vm = __ballot_sync(kFull, row >= 0);
                    const uint32_t bar = bar0 + stage_i * 8;
                    if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(vm) * C::ROWB);
                    __syncwarp();
                    if (row >= 0) {
                        const uint32_t dst = ring0 + stage_i * C::STAGEB + (lane >> 4) * C::TILEB + (lane & 15) * C::PITCH;
                        bulk_g2s(dst, (lane < 16 ? k_cache : v_cache) + (size_t)row * C::ROWB, C::ROWB, bar);
                    }
                    stage_i = (stage_i + 1 == nstage) ? 0 : stage_i + 1;
                    ++pe;
                }
            };
            top_up();
            while (ce < n_tiles) {
                if (!mbar_wait(bar0 + stage_c * 8, (phases >> stage_c) & 1u)) {
                    failed = true;
                    break;
                }
                phases ^= (1u << stage_c);
                const uint32_t Ks = ring0 + stage_c * C::STAGEB;
                const uint32_t Vs = Ks + C::TILEB;
                stage_c = (stage_c + 1 == nstage) ? 0 : stage_c + 1;
                const unsigned vmask = __ballot_sync(kFull, ent_row[ce * kPage + (lane & 15)] >= 0) & 0xffffu;
                if (vmask == 0u) {                        // nothing to attend in this tile
                    ++ce;
                    top_up();
                    continue;
                }
                if (vmask != 0xffffu) {
                    // skipped tokens: whatever the stage held before must not reach the product
                    for (int idx = lane; idx < kPage * (C::ROWB / 16); idx += 32) {
                        const int row = idx / (C::ROWB / 16);
                        if (!((vmask >> row) & 1u))
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(Vs + row * C::PITCH + (idx % (C::ROWB / 16)) * 16), "r"(0u) : "memory");
                    }
                    __syncwarp();
                }
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                float s0b[4] = {0.f, 0.f, 0.f, 0.f}, s1b[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int s = 0; s < C::KSTEPS; ++s) {
                    uint32_t b00, b01, b10, b11;
                    ldmatrix_x4(Ks + k_row * C::PITCH + ((2 * s + k_chunk_add) << 4), b00, b01, b10, b11);
                    if (s & 1) {
                        mma_bf16_16816(s0b, qa[s][0], 0u, qa[s][1], 0u, b00, b01);
                        mma_bf16_16816(s1b, qa[s][0], 0u, qa[s][1], 0u, b10, b11);
                    } else {
                        mma_bf16_16816(s0, qa[s][0], 0u, qa[s][1], 0u, b00, b01);
                        mma_bf16_16816(s1, qa[s][0], 0u, qa[s][1], 0u, b10, b11);
                    }
                }
                s0[0] += s0b[0]; s0[1] += s0b[1]; s1[0] += s1b[0]; s1[1] += s1b[1];
                const int t0 = 2 * tid4;
                float z[4];
                z[0] = ((vmask >> t0) & 1u) ? s0[0] * scale_log2 : -INFINITY;
                z[1] = ((vmask >> (t0 + 1)) & 1u) ? s0[1] * scale_log2 : -INFINITY;
                z[2] = ((vmask >> (t0 + 8)) & 1u) ? s1[0] * scale_log2 : -INFINITY;
                z[3] = ((vmask >> (t0 + 9)) & 1u) ? s1[1] * scale_log2 : -INFINITY;
                float pmax = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
                pmax = fmaxf(pmax, __shfl_xor_sync(kFull, pmax, 1));
                pmax = fmaxf(pmax, __shfl_xor_sync(kFull, pmax, 2));
                const float m_new = fmaxf(m_run, pmax);           // finite: the tile has a valid token
                const float corr = exp2f(m_run - m_new);
                if (__any_sync(kFull, m_new != m_run)) {
                    l_run *= corr;
#pragma unroll
                    for (int nt = 0; nt < C::NTILES; ++nt) {
                        o_acc[nt][0] *= corr; o_acc[nt][1] *= corr; o_acc[nt][2] *= corr; o_acc[nt][3] *= corr;
                    }
                    m_run = m_new;
                }
                float pw[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) pw[e] = exp2f(z[e] - m_run);
                l_run += (pw[0] + pw[1]) + (pw[2] + pw[3]);
                const uint32_t ph0 = pack_bf16(pw[0], pw[1]), ph1 = pack_bf16(pw[2], pw[3]);
                const float2 f0 = bf16x2_to_f2(ph0), f1 = bf16x2_to_f2(ph1);
                const uint32_t pl0 = pack_bf16(pw[0] - f0.x, pw[1] - f0.y), pl1 = pack_bf16(pw[2] - f1.x, pw[3] - f1.y);
#pragma unroll
                for (int c2 = 0; c2 < C::NTILES / 2; ++c2) {
                    uint32_t v00, v01, v10, v11;
                    ldmatrix_x4_trans(Vs + v_row * C::PITCH + ((2 * c2 + v_chunk_add) << 4), v00, v01, v10, v11);
                    mma_bf16_16816(o_acc[2 * c2], ph0, pl0, ph1, pl1, v00, v01);
                    mma_bf16_16816(o_acc[2 * c2 + 1], ph0, pl0, ph1, pl1, v10, v11);
                }
                __syncwarp();
                // rows cleared with ordinary stores come before the bulk copies that refill the stage
                if (vmask != 0xffffu) fence_proxy_async();
                ++ce;
                top_up();
            }
        }
        if (failed) break;

        l_run += __shfl_xor_sync(kFull, l_run, 1);
        l_run += __shfl_xor_sync(kFull, l_run, 2);
#pragma unroll
        for (int nt = 0; nt < C::NTILES; ++nt) {
            o_acc[nt][0] += o_acc[nt][2];
            o_acc[nt][1] += o_acc[nt][3];
        }
        if (n_split == 1) {
            if (head_ok) {
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                float *o = out + ((size_t)r * H_q + h * G + gid) * D + 2 * tid4;
#pragma unroll
                for (int nt = 0; nt < C::NTILES; ++nt)
                    *reinterpret_cast<float2 *>(o + nt * 8) = make_float2(o_acc[nt][0] * inv, o_acc[nt][1] * inv);
                if (tid4 == 0)
                    lse[(size_t)r * H_q + h * G + gid] = l_run > 0.f ? (m_run + log2f(l_run)) * kLn2 : -INFINITY;
            }
            continue;
        }
        if (head_ok) {
            float *pr = partials + (((size_t)r * H_q + h * G + gid) * max_splits + my_split) * C::PSTRIDE;
#pragma unroll
            for (int nt = 0; nt < C::NTILES; ++nt)
                *reinterpret_cast<float2 *>(pr + nt * 8 + 2 * tid4) = make_float2(o_acc[nt][0], o_acc[nt][1]);
            if (tid4 == 0) {
                pr[D] = m_run;
                pr[D + 1] = l_run;
            }
        }
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        for (int s = 0; s < nstage; ++s) mbar_wait(bar0 + s * 8, (phases >> s) & 1u);
    }
}

template <int D>
cudaError_t launch_token_decode_t(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                                  const int32_t *page_table, const int32_t *seq_lens, const int32_t *tok_idx,
                                  const int32_t *tok_cnt, int n_out, float *out, float *lse, void *workspace,
                                  const WorkspaceLayout &L, cudaStream_t stream) {
    using C = TokCfg<D>;
    const DecodePlan plan = make_decode_plan(p, true);  // warp units; a unit of the plan = one 16-token tile
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const int G = p.H_q / p.H_kv, GP = next_pow2(G);
    const size_t smem = (size_t)C::CTA_STAGES * C::STAGEB + (size_t)kDecWarps * C::MAXST * 8 +
                        (size_t)kDecWarps * kTokChunk * sizeof(int);
    auto kern = token_decode_kernel<D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<plan.grid, kDecWarps * 32, smem, stream>>>(
        (const uint16_t *)q, (const uint8_t *)k_cache, (const uint8_t *)v_cache, page_table, seq_lens, tok_idx,
        tok_cnt, out, lse, reinterpret_cast<float *>(ws + L.partials), p.B, p.H_kv, G, p.max_pages,
        p.num_phys_pages, n_out, plan.pages_per_split, plan.max_splits, effective_scale(p) * kLog2e,
        reinterpret_cast<uint32_t *>(ws + L.status));
    e = cudaGetLastError();
    if (e != cudaSuccess || plan.max_splits == 1) return e;
    combine_kernel<D><<<dim3(p.B * p.H_kv, 1), 256, 0, stream>>>(
        reinterpret_cast<const float *>(ws + L.partials), nullptr, page_table, seq_lens, nullptr, nullptr, out, lse,
        nullptr, p.H_kv, G, GP, p.max_pages, p.num_phys_pages, p.k_max, plan.pages_per_split, plan.max_splits,
        tok_cnt, 0, 0);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_token_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                                const int32_t *page_table, const int32_t *seq_lens, const int32_t *tok_idx,
                                const int32_t *tok_cnt, int n_out, float *out, float *lse, void *workspace,
                                const WorkspaceLayout &L, cudaStream_t stream) {
    return (p.D == 128) ? launch_token_decode_t<128>(p, q, k_cache, v_cache, page_table, seq_lens, tok_idx,
                                                     tok_cnt, n_out, out, lse, workspace, L, stream)
                        : launch_token_decode_t<64>(p, q, k_cache, v_cache, page_table, seq_lens, tok_idx,
                                                    tok_cnt, n_out, out, lse, workspace, L, stream);
}


int decode_warps_per_cta() { return kDecWarps; }

cudaError_t launch_sparse_decode(const se_params &p, const void *q, const void *k_cache,
                                 const void *v_cache, const int32_t *page_table,
                                 const int32_t *seq_lens, int32_t *sel_idx, int32_t *sel_cnt,
                                 const SelectFromScores *from_scores, float *out, float *lse, float *score_accum,
                                 uint32_t *tok_keys, void *workspace, const WorkspaceLayout &L, int stages,
                                 cudaStream_t stream) {
    return (p.D == 128) ? launch_decode<128>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                             from_scores, out, lse, score_accum, tok_keys, workspace, L, stages, stream)
                        : launch_decode<64>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                            from_scores, out, lse, score_accum, tok_keys, workspace, L, stages, stream);
}

}  // namespace se

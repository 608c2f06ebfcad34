// Split-K paged attention over the selected pages, log-sum-exp merge and the H2O epilogue
// (Appendix A, selected-attention equation and H2O accumulated-score equation).
//
// decode_kernel  Every warp is an autonomous pipeline.  The selected pages of all
//                (request, kv-head) pairs form one flat list of pairs*k_max slots; each warp
//                owns an equal contiguous slice of it, so a pair is split over as many
//                warps as its slots span (split-K) and all warps carry the same load.
//                A K page and a V page of one head are contiguous [16, D] bf16 tiles; the warp
//                streams them through a ring of shared-memory stages with 1-D bulk
//                asynchronous copies (completion on mbarriers) and computes, for the G query
//                heads of the kv-head at once, z = q.K (packed fp32 FMAs, transposing shuffle
//                reduction), an online softmax in base 2 and acc += p.V.  A warp that holds
//                all pages of a pair writes out/lse itself; otherwise it stores a partial
//                (acc, m, l) and the warp that finishes last merges them (an atomic ticket,
//                no waiting).
// h2o_kernel     adds exp(z - lse), summed over the query heads of the kv-head, to the
//                accumulated score of every attended token slot.
#include "se_internal.h"

namespace se {

namespace {

constexpr int kDecWarps = 8;
constexpr int kWin = 32;                 // selected pages looked up at once
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D, int G>
struct DecCfg {
    static constexpr int GP = next_pow2(G);
    static constexpr int LPR = (D == 128 && G > 4) ? 16 : 8;   // lanes per token row
    static constexpr int NCH = D / (LPR * 8);                  // 16-byte pieces per lane and row
    static constexpr int CPL = NCH * 8;                        // channels per lane
    static constexpr int TPP = 32 / LPR;                       // token rows per warp pass
    static constexpr int NP = kPage / TPP;                     // passes per page
    static constexpr int RB = (NP < 32 / GP) ? NP : 32 / GP;   // passes per reduction block
    static constexpr int NV = RB * GP;
    static constexpr int NF = (NV / LPR) > 1 ? (NV / LPR) : 1;
    static constexpr int PAGEB = kPage * D * 2;                // bytes of one K (or V) page
    static constexpr int NSTAGE = (D == 128) ? 3 : 4;
    static constexpr int ZS = kPage * GP;                      // floats of the logit tile
    static constexpr int WARP_SMEM = NSTAGE * 2 * PAGEB + ZS * 4;
    static constexpr int PSTRIDE = D + 4;                      // floats per partial row
    static_assert(NP % RB == 0, "");
    static_assert(NCH >= 1, "");
};

template <int D, int G>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
decode_kernel(const uint16_t *__restrict__ q, const uint8_t *__restrict__ k_cache,
              const uint8_t *__restrict__ v_cache, const int32_t *__restrict__ page_table,
              const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ sel_idx,
              const int32_t *__restrict__ sel_cnt, float *__restrict__ out, float *__restrict__ lse,
              float *__restrict__ partials, uint32_t *__restrict__ tickets, float *__restrict__ zbuf,
              int B, int H_kv, int max_pages, int P_phys, int k_max, int pages_per_warp,
              int max_splits, float scale_log2, uint32_t *status) {
    using C = DecCfg<D, G>;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = smem_raw + (size_t)warp * C::WARP_SMEM;
    float *zs = reinterpret_cast<float *>(ring + C::NSTAGE * 2 * C::PAGEB);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)kDecWarps * C::WARP_SMEM) + warp * C::NSTAGE;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < C::NSTAGE; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_fence_init();
    }
    __syncwarp();
    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t ring0 = smem_u32(ring);

    const int H_q = H_kv * G;
    const int tg = lane / C::LPR, lg = lane % C::LPR;
    const long long X = (long long)B * H_kv * k_max;                 // flat slots
    const long long gw = (long long)blockIdx.x * kDecWarps + warp;
    long long x = gw * pages_per_warp;
    const long long x_end = min(X, x + (long long)pages_per_warp);

    uint32_t phases = 0;          // parity bit per stage
    int stage_c = 0, stage_i = 0; // next stage to consume / to fill
    bool failed = false;

    while (x < x_end && !failed) {
        // ---- the part of one pair that lies in this warp's slice
        const int pair = (int)(x / k_max);
        const int i_lo = (int)(x - (long long)pair * k_max);
        const int i_hi_slot = (int)min((long long)k_max, x_end - (long long)pair * k_max);
        x = (long long)pair * k_max + i_hi_slot;                      // next pair starts here
        const int r = pair / H_kv, h = pair % H_kv;
        int cnt = sel_cnt[pair];
        if (cnt > k_max) {
            if (lane == 0) atomicOr(status, SE_DEV_BAD_SELECTION);
            cnt = k_max;
        }
        const int len = seq_lens[r];
        const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
        if (cnt <= 0 || n_r == 0) {
            if (i_lo == 0) {          // the warp holding the pair's first slot reports "nothing attended"
                for (int g = 0; g < G; ++g) {
                    float *o = out + ((size_t)r * H_q + h * G + g) * D;
                    for (int c = lane; c < D; c += 32) o[c] = 0.f;
                    if (lane == 0) lse[(size_t)r * H_q + h * G + g] = -INFINITY;
                }
            }
            continue;
        }
        if (i_lo >= cnt) continue;
        const int i_hi = min(i_hi_slot, cnt);
        const int w_first = (int)(((long long)pair * k_max) / pages_per_warp);
        const int w_last = (int)(((long long)pair * k_max + cnt - 1) / pages_per_warp);
        const int n_split = w_last - w_first + 1;
        const int my_split = (int)(gw - w_first);

        // ---- q of the G heads, pre-scaled by sm_scale*log2(e)
        float2 q2[G][C::CPL / 2];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int ch = 0; ch < C::NCH; ++ch) {
                const uint4 w = __ldg(reinterpret_cast<const uint4 *>(
                    q + ((size_t)r * H_q + h * G + g) * D + (ch * C::LPR + lg) * 8));
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 f = bf16x2_to_f2(ww[c]);
                    q2[g][ch * 4 + c] = make_float2(f.x * scale_log2, f.y * scale_log2);
                }
            }
        float2 acc[G][C::CPL / 2];
        float m_run[G], l_run[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            m_run[g] = -INFINITY;
            l_run[g] = 0.f;
#pragma unroll
            for (int c = 0; c < C::CPL / 2; ++c) acc[g][c] = make_float2(0.f, 0.f);
        }

        for (int win = i_lo; win < i_hi && !failed; win += kWin) {
            // ---- look up up to 32 selected pages
            const int i_me = win + lane;
            int pid = -1, nv = 0;
            if (i_me < i_hi) {
                const int b = sel_idx[(size_t)pair * k_max + i_me];
                if (b < 0 || b >= n_r) {
                    atomicOr(status, SE_DEV_BAD_SELECTION);
                } else {
                    pid = page_table[(size_t)r * max_pages + b];
                    if (pid >= P_phys) {
                        atomicOr(status, SE_DEV_BAD_PAGE_ID);
                        pid = -1;
                    } else if (pid < 0) {
                        atomicOr(status, SE_DEV_BAD_SELECTION);
                    }
                    nv = min(kPage, len - b * kPage);
                }
            }
            const unsigned vmask = __ballot_sync(kFull, pid >= 0);
            const int nvalid = __popc(vmask);

            auto issue = [&](int j) {
                const int src_lane = __fns(vmask, 0, j + 1);
                const int pj = __shfl_sync(kFull, pid, src_lane);
                if (lane == 0) {
                    const uint32_t bar = bar0 + stage_i * 8;
                    const uint32_t dst = ring0 + stage_i * (2 * C::PAGEB);
                    mbar_expect_tx(bar, 2 * C::PAGEB);
                    const size_t off = ((size_t)pj * H_kv + h) * C::PAGEB;
                    bulk_g2s(dst, k_cache + off, C::PAGEB, bar);
                    bulk_g2s(dst + C::PAGEB, v_cache + off, C::PAGEB, bar);
                }
                stage_i = (stage_i + 1 == C::NSTAGE) ? 0 : stage_i + 1;
            };

            const int pre = min(C::NSTAGE - 1, nvalid);
            for (int j = 0; j < pre; ++j) issue(j);

            for (int j = 0; j < nvalid; ++j) {
                if (j + C::NSTAGE - 1 < nvalid) issue(j + C::NSTAGE - 1);
                const int src_lane = __fns(vmask, 0, j + 1);
                const int nv_j = __shfl_sync(kFull, nv, src_lane);
                const int i_j = win + src_lane;
                if (!mbar_wait(bar0 + stage_c * 8, (phases >> stage_c) & 1u)) {
                    failed = true;
                    break;
                }
                phases ^= (1u << stage_c);
                const uint8_t *Ks = ring + (size_t)stage_c * (2 * C::PAGEB);
                const uint8_t *Vs = Ks + C::PAGEB;
                stage_c = (stage_c + 1 == C::NSTAGE) ? 0 : stage_c + 1;

                // ---- z = q.K for 16 tokens x G heads
#pragma unroll
                for (int rb = 0; rb < C::NP / C::RB; ++rb) {
                    float v[C::NV];
#pragma unroll
                    for (int ip = 0; ip < C::RB; ++ip) {
                        const int t = (rb * C::RB + ip) * C::TPP + tg;
                        float2 kf[C::CPL / 2];
#pragma unroll
                        for (int ch = 0; ch < C::NCH; ++ch) {
                            const uint4 w = *reinterpret_cast<const uint4 *>(Ks + (size_t)t * (D * 2) + (ch * C::LPR + lg) * 16);
                            kf[ch * 4 + 0] = bf16x2_to_f2(w.x);
                            kf[ch * 4 + 1] = bf16x2_to_f2(w.y);
                            kf[ch * 4 + 2] = bf16x2_to_f2(w.z);
                            kf[ch * 4 + 3] = bf16x2_to_f2(w.w);
                        }
#pragma unroll
                        for (int g = 0; g < C::GP; ++g) {
                            if (g < G) {
                                float2 a = make_float2(0.f, 0.f);
#pragma unroll
                                for (int c = 0; c < C::CPL / 2; ++c) a = ffma2(kf[c], q2[g < G ? g : 0][c], a);
                                v[ip * C::GP + g] = a.x + a.y;
                            } else {
                                v[ip * C::GP + g] = 0.f;
                            }
                        }
                    }
                    transpose_reduce<C::NV, C::LPR>(v, lane);
                    const int i0 = (C::NV >= C::LPR) ? lg * C::NF : lg / (C::LPR / C::NV);
#pragma unroll
                    for (int jj = 0; jj < C::NF; ++jj) {
                        const int idx = i0 + jj;
                        const int g = idx % C::GP;
                        const int t = (rb * C::RB + idx / C::GP) * C::TPP + tg;
                        const float z = (t < nv_j) ? v[jj] : -INFINITY;
                        zs[t * C::GP + g] = z;
                        if (zbuf != nullptr && g < G)
                            zbuf[(((size_t)pair * k_max + i_j) * kPage + t) * C::GP + g] = z;
                    }
                }
                __syncwarp();

                // ---- online softmax (base 2): page maxima of this lane's token rows, then over rows
                float pmax[G];
#pragma unroll
                for (int g = 0; g < G; ++g) pmax[g] = -INFINITY;
#pragma unroll
                for (int tp = 0; tp < C::NP; ++tp) {
                    const int t = tp * C::TPP + tg;
#pragma unroll
                    for (int g = 0; g < G; ++g) pmax[g] = fmaxf(pmax[g], zs[t * C::GP + g]);
                }
#pragma unroll
                for (int mk = C::LPR; mk < 32; mk <<= 1)
#pragma unroll
                    for (int g = 0; g < G; ++g) pmax[g] = fmaxf(pmax[g], __shfl_xor_sync(kFull, pmax[g], mk));
                bool rescale = false;
                float m_use[G];
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float m_new = fmaxf(m_run[g], pmax[g]);
                    rescale |= (m_new != m_run[g]);
                    m_use[g] = m_new;
                }
                if (rescale) {            // warp-uniform: the maxima are identical in every lane
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float corr = (m_use[g] == -INFINITY) ? 1.f : exp2f(m_run[g] - m_use[g]);
                        l_run[g] *= corr;
#pragma unroll
                        for (int c = 0; c < C::CPL / 2; ++c) {
                            acc[g][c].x *= corr;
                            acc[g][c].y *= corr;
                        }
                        m_run[g] = m_use[g];
                    }
                }
                // ---- acc += p.V
#pragma unroll
                for (int tp = 0; tp < C::NP; ++tp) {
                    const int t = tp * C::TPP + tg;
                    float2 vf[C::CPL / 2];
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch) {
                        const uint4 w = *reinterpret_cast<const uint4 *>(Vs + (size_t)t * (D * 2) + (ch * C::LPR + lg) * 16);
                        vf[ch * 4 + 0] = bf16x2_to_f2(w.x);
                        vf[ch * 4 + 1] = bf16x2_to_f2(w.y);
                        vf[ch * 4 + 2] = bf16x2_to_f2(w.z);
                        vf[ch * 4 + 3] = bf16x2_to_f2(w.w);
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float z = zs[t * C::GP + g];
                        const float pz = (z == -INFINITY) ? 0.f : exp2f(z - m_run[g]);
                        l_run[g] += pz;
                        const float2 p2 = make_float2(pz, pz);
#pragma unroll
                        for (int c = 0; c < C::CPL / 2; ++c) acc[g][c] = ffma2(vf[c], p2, acc[g][c]);
                    }
                }
                __syncwarp();     // all lanes are done with this stage and with zs
            }
        }
        if (failed) break;

        // ---- fold the token-row groups: every lane ends with the totals of its channels
#pragma unroll
        for (int mk = C::LPR; mk < 32; mk <<= 1)
#pragma unroll
            for (int g = 0; g < G; ++g) {
                l_run[g] += __shfl_xor_sync(kFull, l_run[g], mk);
#pragma unroll
                for (int c = 0; c < C::CPL / 2; ++c) {
                    acc[g][c].x += __shfl_xor_sync(kFull, acc[g][c].x, mk);
                    acc[g][c].y += __shfl_xor_sync(kFull, acc[g][c].y, mk);
                }
            }

        if (n_split == 1) {
            if (tg == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float inv = l_run[g] > 0.f ? 1.f / l_run[g] : 0.f;
                    float *o = out + ((size_t)r * H_q + h * G + g) * D;
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch) {
                        float4 *dst = reinterpret_cast<float4 *>(o + (ch * C::LPR + lg) * 8);
                        dst[0] = make_float4(acc[g][ch * 4 + 0].x * inv, acc[g][ch * 4 + 0].y * inv,
                                             acc[g][ch * 4 + 1].x * inv, acc[g][ch * 4 + 1].y * inv);
                        dst[1] = make_float4(acc[g][ch * 4 + 2].x * inv, acc[g][ch * 4 + 2].y * inv,
                                             acc[g][ch * 4 + 3].x * inv, acc[g][ch * 4 + 3].y * inv);
                    }
                    if (lg == 0)
                        lse[(size_t)r * H_q + h * G + g] =
                            l_run[g] > 0.f ? (m_run[g] + log2f(l_run[g])) * kLn2 : -INFINITY;
                }
            }
            continue;
        }

        // ---- store the partial, take a ticket, the last one merges
        if (tg == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float *pr = partials + (((size_t)r * H_q + h * G + g) * max_splits + my_split) * C::PSTRIDE;
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
                    float4 *dst = reinterpret_cast<float4 *>(pr + (ch * C::LPR + lg) * 8);
                    dst[0] = make_float4(acc[g][ch * 4 + 0].x, acc[g][ch * 4 + 0].y, acc[g][ch * 4 + 1].x, acc[g][ch * 4 + 1].y);
                    dst[1] = make_float4(acc[g][ch * 4 + 2].x, acc[g][ch * 4 + 2].y, acc[g][ch * 4 + 3].x, acc[g][ch * 4 + 3].y);
                }
                if (lg == 0) {
                    pr[D] = m_run[g];
                    pr[D + 1] = l_run[g];
                }
            }
        }
        __threadfence();
        __syncwarp();
        unsigned old = 0;
        if (lane == 0) old = atomicAdd(&tickets[pair], 1u);
        old = __shfl_sync(kFull, old, 0);
        if ((int)old != n_split - 1) continue;
        __threadfence();
        if (lane == 0) tickets[pair] = 0u;                 // ready for the next launch
        for (int g = 0; g < G; ++g) {
            const float *pr = partials + (((size_t)r * H_q + h * G + g) * max_splits) * C::PSTRIDE;
            float m_all = -INFINITY;
            for (int s = 0; s < n_split; ++s) m_all = fmaxf(m_all, __ldcg(pr + (size_t)s * C::PSTRIDE + D));
            float L = 0.f;
            float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s = 0; s < n_split; ++s) {
                const float ms = __ldcg(pr + (size_t)s * C::PSTRIDE + D);
                const float ls = __ldcg(pr + (size_t)s * C::PSTRIDE + D + 1);
                const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - m_all);
                L += w * ls;
                if (lane * 4 < D) {
                    const float4 a = __ldcg(reinterpret_cast<const float4 *>(pr + (size_t)s * C::PSTRIDE) + lane);
                    o4.x += w * a.x; o4.y += w * a.y; o4.z += w * a.z; o4.w += w * a.w;
                }
            }
            const float inv = L > 0.f ? 1.f / L : 0.f;
            if (lane * 4 < D) {
                float4 *dst = reinterpret_cast<float4 *>(out + ((size_t)r * H_q + h * G + g) * D) + lane;
                *dst = make_float4(o4.x * inv, o4.y * inv, o4.z * inv, o4.w * inv);
            }
            if (lane == 0)
                lse[(size_t)r * H_q + h * G + g] = L > 0.f ? (m_all + log2f(L)) * kLn2 : -INFINITY;
        }
    }
    if (failed) {
        if (lane == 0) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        // bounded wait for whatever this warp still has in flight before the CTA can retire
        for (int s = 0; s < C::NSTAGE; ++s) mbar_wait(bar0 + s * 8, (phases >> s) & 1u);
    }
}

// score_accum[pid,h,t] += sum_g exp2(z2[g] - lse[g]*log2e) for every attended token slot.
template <int GP>
__global__ void __launch_bounds__(256)
h2o_kernel(const float *__restrict__ zbuf, const float *__restrict__ lse, const int32_t *__restrict__ page_table,
           const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ sel_idx,
           const int32_t *__restrict__ sel_cnt, float *__restrict__ score_accum, int B, int H_kv, int G,
           int max_pages, int P_phys, int k_max) {
    const long long total = (long long)B * H_kv * k_max * kPage;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(e % kPage);
        const long long slot = e / kPage;
        const int i = (int)(slot % k_max);
        const int pair = (int)(slot / k_max);
        const int r = pair / H_kv, h = pair % H_kv;
        if (i >= min(sel_cnt[pair], k_max)) continue;
        const int len = seq_lens[r];
        const int n_r = len > 0 ? min(max_pages, (len + kPage - 1) / kPage) : 0;
        const int b = sel_idx[(size_t)pair * k_max + i];
        if (b < 0 || b >= n_r) continue;
        const int pid = page_table[(size_t)r * max_pages + b];
        if (pid < 0 || pid >= P_phys) continue;
        if (t >= min(kPage, len - b * kPage)) continue;
        const float *z = zbuf + (size_t)e * GP;
        float add = 0.f;
        for (int g = 0; g < G; ++g) {
            const float l2 = lse[(size_t)r * (H_kv * G) + h * G + g] * kLog2e;
            const float zz = z[g];
            if (zz != -INFINITY) add += exp2f(zz - l2);
        }
        score_accum[((size_t)pid * H_kv + h) * kPage + t] += add;
    }
}

template <int D, int G>
cudaError_t launch_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                          const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                          const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                          void *workspace, const WorkspaceLayout &L, cudaStream_t stream) {
    using C = DecCfg<D, G>;
    const DecodePlan plan = make_decode_plan(p);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const size_t smem = (size_t)kDecWarps * C::WARP_SMEM + (size_t)kDecWarps * C::NSTAGE * 8;
    auto kern = decode_kernel<D, G>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    float *zbuf = score_accum ? reinterpret_cast<float *>(ws + L.zbuf) : nullptr;
    kern<<<plan.grid, kDecWarps * 32, smem, stream>>>(
        (const uint16_t *)q, (const uint8_t *)k_cache, (const uint8_t *)v_cache, page_table, seq_lens,
        sel_idx, sel_cnt, out, lse, reinterpret_cast<float *>(ws + L.partials),
        reinterpret_cast<uint32_t *>(ws + L.dec_tickets), zbuf, p.B, p.H_kv, p.max_pages,
        p.num_phys_pages, p.k_max, plan.pages_per_warp, plan.max_splits,
        effective_scale(p) * kLog2e, reinterpret_cast<uint32_t *>(ws + L.status));
    e = cudaGetLastError();
    if (e != cudaSuccess || !score_accum) return e;
    const long long total = (long long)p.B * p.H_kv * p.k_max * kPage;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)device_sm_count() * 8;
    if (blocks > cap) blocks = cap;
    h2o_kernel<C::GP><<<(unsigned)blocks, 256, 0, stream>>>(zbuf, lse, page_table, seq_lens, sel_idx, sel_cnt,
                                                          score_accum, p.B, p.H_kv, G, p.max_pages,
                                                          p.num_phys_pages, p.k_max);
    return cudaGetLastError();
}

template <int D>
cudaError_t dispatch_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                            const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                            const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                            void *workspace, const WorkspaceLayout &L, cudaStream_t stream) {
#define SE_CASE(GG)                                                                                      \
    case GG:                                                                                             \
        return launch_decode<D, GG>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt, out, \
                                    lse, score_accum, workspace, L, stream);
    switch (p.H_q / p.H_kv) {
        SE_CASE(1) SE_CASE(2) SE_CASE(3) SE_CASE(4) SE_CASE(5) SE_CASE(6) SE_CASE(7) SE_CASE(8)
    }
#undef SE_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

int decode_warps_per_cta() { return kDecWarps; }

cudaError_t launch_sparse_decode(const se_params &p, const void *q, const void *k_cache,
                                 const void *v_cache, const int32_t *page_table,
                                 const int32_t *seq_lens, const int32_t *sel_idx,
                                 const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                                 void *workspace, const WorkspaceLayout &L, cudaStream_t stream) {
    return (p.D == 128) ? dispatch_decode<128>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                               out, lse, score_accum, workspace, L, stream)
                        : dispatch_decode<64>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                              out, lse, score_accum, workspace, L, stream);
}

}  // namespace se

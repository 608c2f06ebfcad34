// Split-K paged attention over the selected pages, log-sum-exp merge and the H2O epilogue
// (Appendix A, selected-attention equation and H2O accumulated-score equation).
//
// decode_kernel  Every warp is an autonomous pipeline.  The selected pages of all
//                (request, kv-head) pairs form one flat list of pairs*k_max slots; each warp
//                owns an equal contiguous slice of it, so a pair is split over as many
//                warps as its slots span (split-K) and all warps carry the same load.
//                K and V pages ([16 tokens, D] bf16, contiguous per head) are fetched by TMA
//                tensor copies (2-D tiles of 16 rows x 64 channels, 128-byte swizzle, one
//                mbarrier per ring stage) so that ldmatrix reads them without bank conflicts.
//                Per page and for the G query heads of the kv-head at once:
//                    S^T[head, token] = Q[head, :] . K[token, :]^T      (m16n8k16, fp32 accumulate)
//                    online softmax in base 2 on the accumulator fragments
//                    O[head, :]      += P[head, token] . V[token, :]    (P split into two bf16 terms)
//                The accumulator layout of S^T is the A-operand layout of P, so the
//                probabilities never leave registers.  A warp that holds all pages of a pair
//                writes out/lse itself; otherwise it stores a partial (acc, m, l) and the warp
//                that finishes last merges them (an atomic ticket, no waiting).
//                An earlier plain-FMA version of this kernel needed ~1050 warp instructions per
//                page (8 KB) and was issue-bound at 65 % of the copy bandwidth.
// h2o_kernel     adds exp(z - lse), summed over the query heads of the kv-head, to the
//                accumulated score of every attended token slot.
#include <cuda.h>

#include "se_internal.h"

namespace se {

namespace {

constexpr int kDecWarps = 8;
constexpr int kWin = 32;                 // selected pages looked up at once
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTileBytes = kPage * 128;  // one TMA box: 16 rows x 64 bf16

template <int D>
struct DecCfg {
    static constexpr int HALVES = D / 64;                      // 64-channel tiles per page
    static constexpr int PAGEB = kPage * D * 2;                // bytes of one K (or V) page
    static constexpr int STAGEB = 2 * PAGEB;                   // K tiles then V tiles
    static constexpr int NSTAGE = (D == 128) ? 3 : 4;
    static constexpr int KSTEPS = D / 16;
    static constexpr int NTILES = D / 8;                       // n8 tiles of the output
    static constexpr int WARP_SMEM = NSTAGE * STAGEB;
    static constexpr int PSTRIDE = D + 4;                      // floats per partial row
};

// TMA: 2-D tile (x = channel, y = row of the [pages*heads*16, D] view) -> shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
decode_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
              const uint16_t *__restrict__ q, const int32_t *__restrict__ page_table,
              const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ sel_idx,
              const int32_t *__restrict__ sel_cnt, float *__restrict__ out, float *__restrict__ lse,
              float *__restrict__ partials, uint32_t *__restrict__ tickets, float *__restrict__ zbuf,
              int B, int H_kv, int G, int GP, int max_pages, int P_phys, int k_max, int pages_per_warp,
              int max_splits, float scale_log2, uint32_t *status) {
    using C = DecCfg<D>;
    extern __shared__ uint8_t smem_dyn[];
    // tiles must sit on 1024-byte boundaries for the 128-byte swizzle pattern
    uint8_t *smem_al = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = smem_al + (size_t)warp * C::WARP_SMEM;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + (size_t)kDecWarps * C::WARP_SMEM) + warp * C::NSTAGE;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < C::NSTAGE; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_fence_init();
    }
    __syncwarp();
    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t ring0 = smem_u32(ring);

    const int H_q = H_kv * G;
    const int gid = lane >> 2, tid4 = lane & 3;          // fragment coordinates: head row / column pair
    const bool head_ok = gid < G;
    const long long X = (long long)B * H_kv * k_max;     // flat slots
    const long long gw = (long long)blockIdx.x * kDecWarps + warp;
    long long x = gw * pages_per_warp;
    const long long x_end = min(X, x + (long long)pages_per_warp);

    // ldmatrix lane offsets inside a 16x128-byte swizzled tile.
    // K (B operand, not transposed): matrices {tok 0-7 | 8-15} x {chunk c | c+1}
    const int k_row = (lane & 7) + 8 * (lane >> 4);
    const int k_chunk_add = (lane >> 3) & 1;
    // V (B operand, transposed): matrices {tok 0-7 | 8-15} fastest, then {chunk c | c+1}
    const int v_row = (lane & 7) + 8 * ((lane >> 3) & 1);
    const int v_chunk_add = lane >> 4;

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

        // ---- Q as the A operand: row gid = query head gid of the group (rows >= G and 8..15 are zero)
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
        float m_run = -INFINITY, l_run = 0.f;       // of head gid; l is this lane's share (its 4 token columns)

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
                    const uint32_t dst = ring0 + stage_i * C::STAGEB;
                    mbar_expect_tx(bar, C::STAGEB);
                    const int y = (pj * H_kv + h) * kPage;
#pragma unroll
                    for (int hf = 0; hf < C::HALVES; ++hf) {
                        tma_load_2d(dst + hf * kTileBytes, &k_map, hf * 64, y, bar);
                        tma_load_2d(dst + C::PAGEB + hf * kTileBytes, &v_map, hf * 64, y, bar);
                    }
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
                const uint32_t Ks = ring0 + stage_c * C::STAGEB;
                const uint32_t Vs = Ks + C::PAGEB;
                stage_c = (stage_c + 1 == C::NSTAGE) ? 0 : stage_c + 1;

                // ---- S^T[head, token] = Q . K^T : two n8 tiles (tokens 0-7, 8-15)
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int s = 0; s < C::KSTEPS; ++s) {
                    const int hf = s >> 2;
                    const int chunk = 2 * (s & 3) + k_chunk_add;
                    uint32_t b00, b01, b10, b11;     // {tok 0-7: k lo, k hi}, {tok 8-15: k lo, k hi}
                    ldmatrix_x4(Ks + hf * kTileBytes + k_row * 128 + ((chunk ^ (k_row & 7)) << 4), b00, b01, b10, b11);
                    mma_bf16_16816(s0, qa[s][0], 0u, qa[s][1], 0u, b00, b01);
                    mma_bf16_16816(s1, qa[s][0], 0u, qa[s][1], 0u, b10, b11);
                }
                // this lane: head gid, tokens 2*tid4, 2*tid4+1 (s0) and 8+2*tid4, 9+2*tid4 (s1)
                const int t0 = 2 * tid4;
                float z[4];
                z[0] = (t0 < nv_j) ? s0[0] * scale_log2 : -INFINITY;
                z[1] = (t0 + 1 < nv_j) ? s0[1] * scale_log2 : -INFINITY;
                z[2] = (t0 + 8 < nv_j) ? s1[0] * scale_log2 : -INFINITY;
                z[3] = (t0 + 9 < nv_j) ? s1[1] * scale_log2 : -INFINITY;
                if (zbuf != nullptr && head_ok) {
                    float *zp = zbuf + (((size_t)pair * k_max + i_j) * kPage) * GP + gid;
                    zp[(t0) * GP] = z[0];
                    zp[(t0 + 1) * GP] = z[1];
                    zp[(t0 + 8) * GP] = z[2];
                    zp[(t0 + 9) * GP] = z[3];
                }
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
                    }
                    m_run = m_new;
                }
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) p[e] = exp2f(z[e] - m_run);    // exp2(-inf) = 0 for masked tokens
                l_run += (p[0] + p[1]) + (p[2] + p[3]);
                // P as the A operand, split into two bf16 terms so that p_hi + p_lo carries 16 bits
                const uint32_t ph0 = pack_bf16(p[0], p[1]), ph1 = pack_bf16(p[2], p[3]);
                const float2 f0 = bf16x2_to_f2(ph0), f1 = bf16x2_to_f2(ph1);
                const uint32_t pl0 = pack_bf16(p[0] - f0.x, p[1] - f0.y), pl1 = pack_bf16(p[2] - f1.x, p[3] - f1.y);

                // ---- O[head, :] += P . V : n8 tiles over the channels, k16 = the 16 tokens
#pragma unroll
                for (int c2 = 0; c2 < C::NTILES / 2; ++c2) {
                    const int hf = c2 >> 2;
                    const int chunk = 2 * (c2 & 3) + v_chunk_add;
                    uint32_t v00, v01, v10, v11;     // {chunk c: tok 0-7, tok 8-15}, {chunk c+1: ...}
                    ldmatrix_x4_trans(Vs + hf * kTileBytes + v_row * 128 + ((chunk ^ (v_row & 7)) << 4), v00, v01, v10, v11);
                    mma_bf16_16816(o_acc[2 * c2], ph0, 0u, ph1, 0u, v00, v01);
                    mma_bf16_16816(o_acc[2 * c2], pl0, 0u, pl1, 0u, v00, v01);
                    mma_bf16_16816(o_acc[2 * c2 + 1], ph0, 0u, ph1, 0u, v10, v11);
                    mma_bf16_16816(o_acc[2 * c2 + 1], pl0, 0u, pl1, 0u, v10, v11);
                }
                __syncwarp();     // all lanes are done with this stage before it is refilled
            }
        }
        if (failed) break;

        // ---- the four lanes of a head hold disjoint token columns: fold their l
        l_run += __shfl_xor_sync(kFull, l_run, 1);
        l_run += __shfl_xor_sync(kFull, l_run, 2);

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

        // ---- store the partial, take a ticket, the last one merges
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
__global__ void __launch_bounds__(256)
h2o_kernel(const float *__restrict__ zbuf, const float *__restrict__ lse, const int32_t *__restrict__ page_table,
           const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ sel_idx,
           const int32_t *__restrict__ sel_cnt, float *__restrict__ score_accum, int B, int H_kv, int G, int GP,
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

// The cache viewed as a 2-D bf16 tensor [P_phys*H_kv*16 rows, D channels]; box = 16 rows x 64 channels.
bool make_page_map(CUtensorMap *map, const void *base, const se_params &p) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)p.D, (cuuint64_t)p.num_phys_pages * p.H_kv * kPage};
    const cuuint64_t strides[1] = {(cuuint64_t)p.D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t launch_decode(const se_params &p, const void *q, const void *k_cache, const void *v_cache,
                          const int32_t *page_table, const int32_t *seq_lens, const int32_t *sel_idx,
                          const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                          void *workspace, const WorkspaceLayout &L, cudaStream_t stream) {
    using C = DecCfg<D>;
    const DecodePlan plan = make_decode_plan(p);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    CUtensorMap k_map, v_map;
    if (!make_page_map(&k_map, k_cache, p) || !make_page_map(&v_map, v_cache, p)) return cudaErrorInvalidValue;
    const size_t smem = (size_t)kDecWarps * C::WARP_SMEM + (size_t)kDecWarps * C::NSTAGE * 8 + 1024;
    auto kern = decode_kernel<D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int G = p.H_q / p.H_kv, GP = next_pow2(G);
    float *zbuf = score_accum ? reinterpret_cast<float *>(ws + L.zbuf) : nullptr;
    kern<<<plan.grid, kDecWarps * 32, smem, stream>>>(
        k_map, v_map, (const uint16_t *)q, page_table, seq_lens, sel_idx, sel_cnt, out, lse,
        reinterpret_cast<float *>(ws + L.partials), reinterpret_cast<uint32_t *>(ws + L.dec_tickets), zbuf,
        p.B, p.H_kv, G, GP, p.max_pages, p.num_phys_pages, p.k_max, plan.pages_per_warp, plan.max_splits,
        effective_scale(p) * kLog2e, reinterpret_cast<uint32_t *>(ws + L.status));
    e = cudaGetLastError();
    if (e != cudaSuccess || !score_accum) return e;
    const long long total = (long long)p.B * p.H_kv * p.k_max * kPage;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)device_sm_count() * 8;
    if (blocks > cap) blocks = cap;
    h2o_kernel<<<(unsigned)blocks, 256, 0, stream>>>(zbuf, lse, page_table, seq_lens, sel_idx, sel_cnt,
                                                     score_accum, p.B, p.H_kv, G, GP, p.max_pages,
                                                     p.num_phys_pages, p.k_max);
    return cudaGetLastError();
}

}  // namespace

int decode_warps_per_cta() { return kDecWarps; }

cudaError_t launch_sparse_decode(const se_params &p, const void *q, const void *k_cache,
                                 const void *v_cache, const int32_t *page_table,
                                 const int32_t *seq_lens, const int32_t *sel_idx,
                                 const int32_t *sel_cnt, float *out, float *lse, float *score_accum,
                                 void *workspace, const WorkspaceLayout &L, cudaStream_t stream) {
    return (p.D == 128) ? launch_decode<128>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                             out, lse, score_accum, workspace, L, stream)
                        : launch_decode<64>(p, q, k_cache, v_cache, page_table, seq_lens, sel_idx, sel_cnt,
                                            out, lse, score_accum, workspace, L, stream);
}

}  // namespace se

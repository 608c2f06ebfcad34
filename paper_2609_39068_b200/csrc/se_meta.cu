// Quest page summaries: channel-wise min / max of K over the valid tokens of a page
// (Appendix A, Quest summary equation; the incremental mode follows the sentence after the score
// equation: a newly written key only changes the extrema of the page it lands in).
//
// One warp per (request, logical page, kv-head).  A K page of one head is a contiguous
// [16, D] bf16 tile; a row is read with 16-byte loads by D/8 lanes, several rows per warp
// pass, and the row groups are folded with shuffles.  min/max of bf16 pairs is exact.
#include "se_internal.h"

namespace se {

namespace {

template <int D>
__global__ void __launch_bounds__(256)
meta_update_kernel(const uint4 *__restrict__ k_cache, const int32_t *__restrict__ page_table,
                   const int32_t *__restrict__ seq_lens, const int32_t *__restrict__ first_tok,
                   uint4 *__restrict__ meta, int B, int H_kv, int max_pages, int P_phys,
                   uint32_t *status) {
    constexpr int LPR = D / 8;           // lanes per token row (16-byte pieces)
    constexpr int TPP = 32 / LPR;        // token rows per warp pass
    constexpr int NP = kPage / TPP;      // passes per page
    const int lane = threadIdx.x & 31;
    const int tg = lane / LPR, lr = lane % LPR;
    const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    const bool incremental = (first_tok == nullptr);
    const long long items = incremental ? (long long)B * H_kv : (long long)B * max_pages * H_kv;

    for (long long it = warp0; it < items; it += nwarps) {
        int r, b, h;
        h = (int)(it % H_kv);
        if (incremental) {
            r = (int)(it / H_kv);
            b = -1;
        } else {
            long long rb = it / H_kv;
            b = (int)(rb % max_pages);
            r = (int)(rb / max_pages);
        }
        const int len = seq_lens[r];
        if (len <= 0) continue;
        const int n_r = (len + kPage - 1) / kPage;
        if (incremental) {
            b = n_r - 1;
        } else {
            int b0 = first_tok[r] / kPage;
            if (b < b0 || b >= n_r) continue;
        }
        if (b >= max_pages) continue;
        const int pid = page_table[(size_t)r * max_pages + b];
        if (pid < 0) continue;
        if (pid >= P_phys) {
            if (lane == 0 && status) atomicOr(status, SE_DEV_BAD_PAGE_ID);
            continue;
        }
        const int nv = min(kPage, len - b * kPage);
        const uint4 *kp = k_cache + ((size_t)pid * H_kv + h) * (kPage * D / 8);

        uint4 mn = make_uint4(0x7f807f80u, 0x7f807f80u, 0x7f807f80u, 0x7f807f80u);   // +inf pairs
        uint4 mx = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);   // -inf pairs
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const int t = i * TPP + tg;
            if (t < nv) {
                const uint4 w = __ldg(kp + t * LPR + lr);
                mn.x = bmin2(mn.x, w.x); mn.y = bmin2(mn.y, w.y); mn.z = bmin2(mn.z, w.z); mn.w = bmin2(mn.w, w.w);
                mx.x = bmax2(mx.x, w.x); mx.y = bmax2(mx.y, w.y); mx.z = bmax2(mx.z, w.z); mx.w = bmax2(mx.w, w.w);
            }
        }
#pragma unroll
        for (int m = LPR; m < 32; m <<= 1) {
            mn.x = bmin2(mn.x, __shfl_xor_sync(kFull, mn.x, m)); mn.y = bmin2(mn.y, __shfl_xor_sync(kFull, mn.y, m));
            mn.z = bmin2(mn.z, __shfl_xor_sync(kFull, mn.z, m)); mn.w = bmin2(mn.w, __shfl_xor_sync(kFull, mn.w, m));
            mx.x = bmax2(mx.x, __shfl_xor_sync(kFull, mx.x, m)); mx.y = bmax2(mx.y, __shfl_xor_sync(kFull, mx.y, m));
            mx.z = bmax2(mx.z, __shfl_xor_sync(kFull, mx.z, m)); mx.w = bmax2(mx.w, __shfl_xor_sync(kFull, mx.w, m));
        }
        uint4 *mp = meta + ((size_t)pid * H_kv + h) * (2 * D / 8);
        if (tg == 0) mp[lr] = mn;
        if (tg == 1) mp[LPR + lr] = mx;
    }
}

}  // namespace

cudaError_t launch_meta_update(const se_params &p, const void *k_cache, const int32_t *page_table,
                               const int32_t *seq_lens, const int32_t *first_tok, void *meta,
                               cudaStream_t stream) {
    const long long items = first_tok ? (long long)p.B * p.max_pages * p.H_kv : (long long)p.B * p.H_kv;
    const int warps_per_cta = 8;
    long long ctas = (items + warps_per_cta - 1) / warps_per_cta;
    const long long cap = (long long)device_sm_count() * 32;
    if (ctas > cap) ctas = cap;
    if (ctas < 1) ctas = 1;
    // no workspace is passed to this call, so out-of-range page ids are skipped without a report
    if (p.D == 128)
        meta_update_kernel<128><<<(unsigned)ctas, 256, 0, stream>>>(
            (const uint4 *)k_cache, page_table, seq_lens, first_tok, (uint4 *)meta, p.B, p.H_kv,
            p.max_pages, p.num_phys_pages, nullptr);
    else
        meta_update_kernel<64><<<(unsigned)ctas, 256, 0, stream>>>(
            (const uint4 *)k_cache, page_table, seq_lens, first_tok, (uint4 *)meta, p.B, p.H_kv,
            p.max_pages, p.num_phys_pages, nullptr);
    return cudaGetLastError();
}

}  // namespace se

// Read-only gather probe: the practical ceiling of the path's access patterns on a given GPU.
//
// The scoring, attention and token-attention kernels are gathers of fixed-size pieces (512-byte page
// summaries, 4 KB K and V pages, 256-byte token rows) through per-warp rings of shared-memory stages
// filled by bulk asynchronous copies.  This kernel does exactly that and nothing else - no look-ups
// beyond the piece list, no arithmetic - so its time on the same piece list is what the memory system
// allows for that pattern and pipeline shape; a kernel's distance to it is what its own look-ups and
// arithmetic cost.  The paper has no counterpart: it is a measurement aid for the benchmark.
#include "se_internal.h"

namespace se {

namespace {

constexpr int kProbeMaxStages = 24;

// Every warp is an autonomous pipeline over the stage-batches b = gw, gw + warps, ...: a batch is
// `pps` pieces; lane j < pps looks up piece b*pps + j and copies it into slot j of the stage.
__global__ void __launch_bounds__(1024)
gather_probe_kernel(const uint8_t *__restrict__ base0, const uint8_t *__restrict__ base1,
                    const int32_t *__restrict__ piece_idx, long long n_pieces, int piece_bytes, int pps, int nstage,
                    uint32_t *status) {
    extern __shared__ __align__(128) uint8_t smem_probe[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    const size_t stage_bytes = (size_t)pps * piece_bytes;
    uint8_t *ring = smem_probe + (size_t)warp * nstage * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_probe + (size_t)nwarps * nstage * stage_bytes) + warp * kProbeMaxStages;
    if (lane == 0) {
        for (int s = 0; s < nstage; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_fence_init();
    }
    __syncwarp();
    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t ring0 = smem_u32(ring);
    const long long n_batches = (n_pieces + pps - 1) / pps;
    const long long gw = (long long)blockIdx.x * nwarps + warp, tw = (long long)gridDim.x * nwarps;
    uint32_t phases = 0;
    int stage_i = 0, stage_c = 0;
    long long issued = gw, consumed = gw;
    int in_flight = 0;
    // the piece of the batch after the next one to issue is looked up ahead of time
    auto lookup = [&](long long b) -> int {
        const long long e = b * pps + lane;
        return (b < n_batches && lane < pps && e < n_pieces) ? __ldg(piece_idx + e) : -1;
    };
    int next_idx = lookup(issued);
    bool failed = false;
    while (consumed < n_batches) {
        while (issued < n_batches && in_flight < nstage) {
            const int idx = next_idx;
            next_idx = lookup(issued + tw);
            const unsigned valid = __ballot_sync(kFull, idx >= 0);
            const uint32_t bar = bar0 + stage_i * 8;
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)__popc(valid) * piece_bytes);
            __syncwarp();
            if (idx >= 0) {
                const uint8_t *src = ((base1 != nullptr && (lane & 1)) ? base1 : base0) + (size_t)idx * piece_bytes;
                bulk_g2s(ring0 + (uint32_t)(stage_i * stage_bytes) + lane * piece_bytes, src, piece_bytes, bar);
            }
            stage_i = stage_i + 1 == nstage ? 0 : stage_i + 1;
            issued += tw;
            ++in_flight;
        }
        if (!mbar_wait(bar0 + stage_c * 8, (phases >> stage_c) & 1u)) {
            failed = true;
            break;
        }
        phases ^= 1u << stage_c;
        stage_c = stage_c + 1 == nstage ? 0 : stage_c + 1;
        consumed += tw;
        --in_flight;
        __syncwarp();
    }
    if (failed) {
        if (lane == 0 && status) atomicOr(status, SE_DEV_WAIT_TIMEOUT);
        for (int s = 0; s < nstage; ++s) mbar_wait(bar0 + s * 8, (phases >> s) & 1u);
    }
}

}  // namespace

}  // namespace se

extern "C" int se_probe_gather(const void *base0, const void *base1, const int32_t *piece_idx, int64_t n_pieces,
                               int32_t piece_bytes, int32_t pieces_per_stage, int32_t stages_per_warp,
                               int32_t warps_per_cta, int32_t ctas_per_sm, void *stream) {
    if (!base0 || !piece_idx) return SE_ERR_NULL_POINTER;
    if ((reinterpret_cast<uintptr_t>(base0) | reinterpret_cast<uintptr_t>(base1) |
         reinterpret_cast<uintptr_t>(piece_idx)) & 15u)
        return SE_ERR_MISALIGNED;
    if (n_pieces < 1 || piece_bytes < 16 || (piece_bytes & 15) || pieces_per_stage < 1 || pieces_per_stage > 32 ||
        stages_per_warp < 1 || stages_per_warp > se::kProbeMaxStages || warps_per_cta < 1 || warps_per_cta > 32 ||
        ctas_per_sm < 1 || ctas_per_sm > 8)
        return SE_ERR_INVALID_ARG;
    const size_t smem = (size_t)warps_per_cta * stages_per_warp * pieces_per_stage * piece_bytes +
                        (size_t)warps_per_cta * se::kProbeMaxStages * 8;
    if (smem > 227 * 1024) return SE_ERR_INVALID_ARG;
    if (cudaFuncSetAttribute(se::gather_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return SE_ERR_CUDA;
    se::gather_probe_kernel<<<se::device_sm_count() * ctas_per_sm, warps_per_cta * 32, smem,
                              static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t *>(base0), static_cast<const uint8_t *>(base1), piece_idx, n_pieces, piece_bytes,
        pieces_per_stage, stages_per_warp, nullptr);
    return cudaGetLastError() == cudaSuccess ? SE_OK : SE_ERR_CUDA;
}

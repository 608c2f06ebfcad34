// Device-side building blocks shared by the kernels: mbarrier / bulk-copy PTX wrappers
// with bounded waits, bf16 unpacking, packed fp32 FMA, and the transposing warp reduction.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sparse_engine.h"

namespace se {

constexpr int kPage = 16;
constexpr unsigned kFull = 0xffffffffu;

// ---------------------------------------------------------------------------------
// Workspace layout (host and device agree through this struct; all offsets in bytes
// from the workspace base, each a multiple of 256).
// ---------------------------------------------------------------------------------
struct WorkspaceLayout {
    size_t status;          // 256 bytes: uint32 status word, work-queue counters of the score kernel
    size_t pairctl;         // uint32 [B*H_kv] arrival counters (fused top-k, in-kernel merge); zero between calls
    bool   has_pairctl;
    size_t scores;          // float  [B*H_kv][score_pitch]
    size_t partials;        // float  [B*H_q*max_splits*(D+2)]
    size_t zbuf;            // float  [B*H_kv*k_max*16*G]  logits kept for the H2O epilogue
    size_t total;
    int    max_splits;
};

// ---------------------------------------------------------------------------------
// shared-memory addresses, mbarriers, bulk copies
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after kWaitLimitNs of wall-clock time (%globaltimer; far beyond any copy's
// latency) and reports failure instead of spinning forever.
constexpr unsigned long long kWaitLimitNs = 200ull * 1000 * 1000;

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 256; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        if (globaltimer_ns() - t0 > kWaitLimitNs) return false;
    }
}

// One-dimensional bulk asynchronous copy global -> shared of this CTA (no tensor map).
// src, dst 16-byte aligned, bytes a multiple of 16; completion is signalled on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// ---------------------------------------------------------------------------------
// arithmetic helpers
// ---------------------------------------------------------------------------------
// bf16 pair packed in a 32-bit word -> two fp32 (exact).
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t w) {
    float2 r;
    r.x = __uint_as_float(w << 16);
    r.y = __uint_as_float(w & 0xffff0000u);
    return r;
}

__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    return __ffma2_rn(a, b, c);
}

// min / max of two packed bf16 pairs (exact; -0 orders below +0)
__device__ __forceinline__ uint32_t bmin2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}

// Order-preserving map fp32 -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t f32_key(float f) {
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

constexpr uint32_t kKeyAbsent = 0x007fffffu;   // f32_key(-inf): below every finite score
constexpr uint32_t kKeyForced = 0xffffffffu;   // marks a page that is selected regardless of its score

// Exclusive prefix of one int per thread over the CTA (thread order); `tot` is a shared array
// of at least 32 ints that no other scan is using between the surrounding barriers.
template <int NW>
__device__ __forceinline__ int cta_excl_scan(int v, int *tot, int lane, int warp) {
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) tot[warp] = inc;
    __syncthreads();
    const int wt = lane < NW ? tot[lane] : 0;
    int winc = wt;
#pragma unroll
    for (int o = 1; o < NW; o <<= 1) {
        const int t = __shfl_up_sync(kFull, winc, o);
        if (lane >= o) winc += t;
    }
    return __shfl_sync(kFull, winc - wt, warp) + inc - v;
}

// ---------------------------------------------------------------------------------
// warp-level matrix helpers (bf16 inputs, fp32 accumulation)
// ---------------------------------------------------------------------------------
// Four 8x8 b16 matrices from shared memory; lane l supplies the address of row (l & 7) of
// matrix (l >> 3) and receives, from matrix i, elements (row l>>2, columns 2*(l&3), +1).
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}
// Same, each matrix transposed on the way in.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__host__ __device__ constexpr int next_pow2(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

// ---------------------------------------------------------------------------------
// Transposing reduction.  Every lane of a group of LP consecutive lanes (LP a power of
// two, group aligned) holds N0 partial values v[0..N0); the sum over the group of v[i]
// is wanted for every i.  Instead of N0 butterflies, each step exchanges half of the
// values, so a step costs N/2 shuffles.  On return lane `lg` (index in its group) holds
// in v[0..NF), NF = max(1, N0/LP), the complete sums of the indices
//     i = lg*NF + j            (N0 >= LP)
//     i = lg / (LP/N0)         (N0 <  LP; neighbouring lanes hold copies)
// ---------------------------------------------------------------------------------
template <int N, int MASK>
struct TReduce {
    template <int NMAX>
    static __device__ __forceinline__ void run(float (&v)[NMAX], int lane) {
        if constexpr (MASK >= 1) {
            if constexpr (N >= 2) {
                const bool up = (lane & MASK) != 0;
#pragma unroll
                for (int j = 0; j < N / 2; ++j) {
                    const float keep = up ? v[j + N / 2] : v[j];
                    const float send = up ? v[j] : v[j + N / 2];
                    v[j] = keep + __shfl_xor_sync(kFull, send, MASK);
                }
                TReduce<N / 2, MASK / 2>::run(v, lane);
            } else {
                v[0] += __shfl_xor_sync(kFull, v[0], MASK);
                TReduce<1, MASK / 2>::run(v, lane);
            }
        }
    }
};

template <int N0, int LP, int NMAX>
__device__ __forceinline__ void transpose_reduce(float (&v)[NMAX], int lane) {
    static_assert((N0 & (N0 - 1)) == 0 && (LP & (LP - 1)) == 0, "powers of two");
    TReduce<N0, LP / 2>::run(v, lane);
}

}  // namespace se

// Skinny weight-streaming GEMM  out[r, n] += sum_k X[r, k] * W[n, k]   (r < R <= 64 rows).
//
// This is the step that moves almost every byte of a verification pass: each bf16 weight is
// read from HBM exactly once and used for all R rows (the paper's Section "Autoregressive vs
// Speculative Sampling": sampling is memory-bound, so K candidate rows cost about what one
// row costs).  Design:
//   * the weight matrix is cut into tiles of 128 rows x 64 k (16 KB); the stream of
//     (tile, k-chunk) units is split evenly and contiguously over a grid of one CTA per SM
//     (stream-K), so every SM pulls the same number of bytes whatever the matrix shape;
//   * one producer thread per CTA issues tensor-map bulk copies (TMA, 128-byte swizzle) of the
//     weight tile and of the matching activation slices into a deep shared-memory ring guarded
//     by mbarriers -- up to ~200 KB of loads in flight per SM to cover HBM latency;
//   * eight consumer warps run bf16 tensor-core MMAs (m16n8k16, fp32 accumulate) with the
//     weights as the 16-row operand and the token rows padded to multiples of 8 on the narrow
//     side.  Activations are fp32 split into bf16 hi + lo, two MMAs per slice, so the result
//     matches fp32-activation arithmetic to ~2^-17;
//   * partial sums of a tile that several CTAs share are added to the output with fp32
//     reductions in L2 (the output is pre-initialised with bias / residual / zero).
// Every wait on an mbarrier is bounded; on time-out the kernel records SSD_E_TIMEOUT and leaves.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace ssd {

constexpr int kTileN = 128;
constexpr int kTileK = 64;
constexpr int kGemmConsumerWarps = 8;
constexpr int kGemmThreads = (kGemmConsumerWarps + 1) * 32;
constexpr int kWTileBytes = kTileN * kTileK * 2;
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s: far beyond any legitimate wait
constexpr int kTimeoutCode = -5;

struct GemmArgs {
    float *out;   // [R, ldo], accumulated into
    int ldo, N, Kd, R;
    int n_tiles, kchunks, stages;
    int32_t *status;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Non-blocking probe (try_wait may suspend the thread for a while; a thread that polls several
// conditions in turn must not).
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` cycles.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t *bar, uint32_t parity, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}
// ... within kWaitCycles (the drain waits of an error path always use this long bound).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    return mbar_wait_limit(bar, parity, kWaitCycles);
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NT = padded rows / 8 (token rows sit on the 8-wide side of the MMA).
template <int NT>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmXhi,
                 const __grid_constant__ CUtensorMap tmXlo, const GemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);  // swizzle atoms are 1 KB
    constexpr int kXBytes = NT * 8 * kTileK * 2;
    constexpr int kStageBytes = kWTileBytes + 2 * kXBytes;
    const int S = a.stages;
    uint64_t *full = (uint64_t *)(smem + (size_t)S * kStageBytes);
    uint64_t *empty = full + S;
    int *abort_flag = (int *)(empty + S);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = (long long)a.n_tiles * a.kchunks;
    const int c0 = (int)(total * blockIdx.x / gridDim.x);
    const int c1 = (int)(total * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kGemmConsumerWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    int issued = 0;
    if (warp == kGemmConsumerWarps) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmXhi) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmXlo) : "memory");
            uint64_t pol_stream;  // weights are read once: let them leave L2 first
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            int tile = c0 / a.kchunks, kc = c0 % a.kchunks;
            for (int c = c0; c < c1; ++c, ++issued) {
                const int s = issued % S;
                if (issued >= S && !mbar_wait(&empty[s], ((issued / S) - 1) & 1)) {
                    set_status(a.status, kTimeoutCode);
                    *abort_flag = 1;
                    break;
                }
                uint8_t *st = smem + (size_t)s * kStageBytes;
                mbar_expect_tx(&full[s], kStageBytes);
                tma_load_2d_hint(st, &tmW, kc * kTileK, tile * kTileN, &full[s], pol_stream);
                tma_load_2d(st + kWTileBytes, &tmXhi, kc * kTileK, 0, &full[s]);
                tma_load_2d(st + kWTileBytes + kXBytes, &tmXlo, kc * kTileK, 0, &full[s]);
                if (++kc == a.kchunks) { kc = 0; ++tile; }
            }
        }
    } else {
        float acc[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

        auto flush = [&](int tile) {
            const int n = tile * kTileN + warp * 16 + (lane >> 2);
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                const int m0 = 8 * j + (lane & 3) * 2;
                if (n < a.N) {
                    if (m0 < a.R) atomicAdd(a.out + (size_t)m0 * a.ldo + n, acc[j][0]);
                    if (m0 + 1 < a.R) atomicAdd(a.out + (size_t)(m0 + 1) * a.ldo + n, acc[j][1]);
                }
                if (n + 8 < a.N) {
                    if (m0 < a.R) atomicAdd(a.out + (size_t)m0 * a.ldo + n + 8, acc[j][2]);
                    if (m0 + 1 < a.R) atomicAdd(a.out + (size_t)(m0 + 1) * a.ldo + n + 8, acc[j][3]);
                }
                acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
            }
        };

        // ldmatrix lane roles.  A (weights): lanes 0-15 address rows 0-15 of the first 8-k chunk,
        // lanes 16-31 the same rows of the second.  B (tokens): four 8x8 blocks = {hi, lo} x 2 chunks.
        const int arow = lane & 15, achunk = lane >> 4;
        const int brow = lane & 7, bsel = lane >> 3;
        int tile = c0 / a.kchunks, kc = c0 % a.kchunks, it = 0;
        bool ok = true;
        for (int c = c0; c < c1; ++c, ++it) {
            const int s = it % S;
            if (!mbar_wait(&full[s], (it / S) & 1)) {
                set_status(a.status, kTimeoutCode);
                ok = false;
                break;
            }
            const uint32_t st = smem_u32(smem + (size_t)s * kStageBytes);
            const uint32_t wbase = st + (uint32_t)(warp * 16 + arow) * 128u;
            const uint32_t xbase = st + kWTileBytes + (bsel >= 2 ? kXBytes : 0) + (uint32_t)brow * 128u;
#pragma unroll
            for (int ks = 0; ks < kTileK / 16; ++ks) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4(wbase + ((uint32_t)((2 * ks + achunk) ^ (arow & 7)) << 4), a0, a1, a2, a3);
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    uint32_t h0, h1, l0, l1;
                    ldmatrix_x4(xbase + (uint32_t)j * 1024u + ((uint32_t)((2 * ks + (bsel & 1)) ^ brow) << 4), h0, h1,
                                l0, l1);
                    mma_bf16(acc[j], a0, a1, a2, a3, h0, h1);
                    mma_bf16(acc[j], a0, a1, a2, a3, l0, l1);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
            if (++kc == a.kchunks) {
                flush(tile);
                kc = 0;
                ++tile;
            }
        }
        if (ok && kc != 0) flush(tile);
    }

    __syncthreads();
    // Error path only: do not leave while bulk copies may still land in this CTA's shared memory.
    if (warp == kGemmConsumerWarps && lane == 0 && *(volatile int *)abort_flag) {
        for (int i = (issued > S ? issued - S : 0); i < issued; ++i) mbar_wait(&full[i % S], (i / S) & 1);
    }
}

// ---------------------------------------------------------------------------------------------
// fp32-weight variant (small fp32 models only; not a bandwidth path): one warp per output feature.
__global__ void gemm_f32_kernel(const float *__restrict__ W, const float *__restrict__ X, int ldx, float *out,
                                int ldo, int N, int Kd, int R) {
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (n >= N) return;
    const float *w = W + (size_t)n * Kd;
    for (int r = 0; r < R; ++r) {
        const float *x = X + (size_t)r * ldx;
        float acc = 0.f;
        for (int k = lane; k < Kd; k += 32) acc = fmaf(x[k], w[k], acc);
        acc = warp_sum(acc);
        if (lane == 0) out[(size_t)r * ldo + n] += acc;
    }
}

}  // namespace ssd

// Prompt pass over many rows at once (Section "KV Caching", Figure 1: the pass that fills the cache before
// sampling starts).  With hundreds or thousands of rows per forward the linear layers are compute-bound: this
// file holds the two kernels that differ from the few-row path - a tiled tcgen05 GEMM over 128 activation rows
// x 256 weight rows per CTA, and a causal attention over row tiles whose keys / values all sit in the cache -
// the row-wise steps (set-up, embedding, norms, activation, rotary + append) are the stepwise path's kernels,
// which take any number of rows.
//
// prefill_gemm_kernel:  out[r, n] += sum_k (Xhi[r, k] + Xlo[r, k]) * W[n, k]
//   * output tiles of 128 rows x 256 columns, dealt round-robin to one CTA per SM; 192 threads: warp 0 = TMA
//     producer, warp 1 = MMA issuer, warps 2-5 = epilogue (one tensor-memory lane quadrant each); two accumulators
//     in tensor memory (2 x 256 columns), so a tile's epilogue runs under the next tile's products;
//   * a stage of the shared-memory ring = the activation rows' hi tile and lo tile (128 rows x 64 k, bf16) and
//     the weight tile (256 rows x 64 k), all by 2-D tensor-map copies with the 128-byte swizzle, 64 KB;
//   * per stage eight tcgen05.mma (M = 128, N = 256, K = 16): four k-steps with the hi tile, four with the lo
//     tile, into ONE fp32 accumulator in tensor memory: W hi + W lo is the fp32-activation product to ~2^-17,
//     the same arithmetic as the few-row path (the price is half the tensor throughput);
//   * the tile is owned by this CTA alone (no split over k), so the epilogue writes accumulator + bias over the
//     output, or adds them to it (the residual stream), with plain loads and stores.
// Every wait is bounded; on time-out the kernel records SSD_E_TIMEOUT, drains its copies and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm.cuh"
#include "persistent.cuh"
#include "rowops.cuh"

namespace ssd {

constexpr int kPfTileM = 128, kPfTileN = 256, kPfStages = 3;
constexpr int kPfABytes = kPfTileM * kTileK * 2;            // 16 KB: one of hi / lo
constexpr int kPfWBytes = kPfTileN * kTileK * 2;            // 32 KB
constexpr int kPfStageBytes = 2 * kPfABytes + kPfWBytes;    // 64 KB
constexpr int kPfThreads = 192;
constexpr size_t kPfSmem = 1024 + (size_t)kPfStages * kPfStageBytes + 256;  // + barriers, TMEM slot, abort flag

struct PfGemmArgs {
    float *out;         // [R, ldo] fp32
    const float *bias;  // [N] or null
    int accumulate;     // 1: out += X W^T + bias (the residual stream); 0: out = X W^T + bias
    int ldo, N, Kd, R;
    long long wait_cycles;  // bound of every wait that takes work
    int32_t *status;
};

__global__ void __launch_bounds__(kPfThreads, 1)
prefill_gemm_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmXhi,
                    const __grid_constant__ CUtensorMap tmXlo, const PfGemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *full = (uint64_t *)(smem + (size_t)kPfStages * kPfStageBytes);
    uint64_t *empty = full + kPfStages;
    uint64_t *acc_full = empty + kPfStages;  // [2]
    uint64_t *acc_empty = acc_full + 2;      // [2]
    uint32_t *tmem_slot = (uint32_t *)(acc_empty + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kchunks = (a.Kd + kTileK - 1) / kTileK;
    const int tiles_m = (a.R + kPfTileM - 1) / kPfTileM, tiles_n = (a.N + kPfTileN - 1) / kPfTileN;
    const int n_tiles = tiles_m * tiles_n;
    // this CTA's tiles: blockIdx.x, + gridDim.x, ...; row tiles vary fastest, so the CTAs that run together share
    // weight tiles in L2 (the activations of all rows stay there anyway)

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPfStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 4);  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    int issued = 0;  // stage fills issued by the producer thread
    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * kPfTileM, n0 = (tile / tiles_m) * kPfTileN;
                for (int kc = 0; kc < kchunks; ++kc, ++issued) {
                    const int s = issued % kPfStages;
                    if (*abort_flag ||
                        (issued >= kPfStages && !mbar_wait_limit(&empty[s], ((issued / kPfStages) - 1) & 1, a.wait_cycles))) {
                        ok = false;
                        break;
                    }
                    uint8_t *st = smem + (size_t)s * kPfStageBytes;
                    mbar_expect_tx(&full[s], kPfStageBytes);
                    tma_load_2d(st, &tmXhi, kc * kTileK, m0, &full[s]);
                    tma_load_2d(st + kPfABytes, &tmXlo, kc * kTileK, m0, &full[s]);
                    tma_load_2d(st + 2 * kPfABytes, &tmW, kc * kTileK, n0, &full[s]);
                }
            }
            if (!ok) {
                set_status(a.status, kTimeoutCode);
                *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kPfTileM, kPfTileN);
            bool ok = true;
            int it = 0, j = 0;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++j) {
                const int buf = j & 1;
                if (j >= 2 && !mbar_wait_limit(&acc_empty[buf], ((j >> 1) - 1) & 1, 4 * a.wait_cycles)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem + (uint32_t)(buf * kPfTileN);
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const int s = it % kPfStages;
                    if (*abort_flag || !mbar_wait_limit(&full[s], (it / kPfStages) & 1, a.wait_cycles)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t st = smem_u32(smem + (size_t)s * kPfStageBytes);
                    const uint64_t hi = umma_desc_sw128(st), lo = umma_desc_sw128(st + kPfABytes), w = umma_desc_sw128(st + 2 * kPfABytes);
#pragma unroll
                    for (int ks = 0; ks < kTileK / 16; ++ks) tc_mma_bf16(d_tmem, hi + 2 * ks, w + 2 * ks, idesc, (kc | ks) ? 1u : 0u);
#pragma unroll
                    for (int ks = 0; ks < kTileK / 16; ++ks) tc_mma_bf16(d_tmem, lo + 2 * ks, w + 2 * ks, idesc, 1u);
                    tc_commit(&empty[s]);
                }
                if (ok) tc_commit(&acc_full[buf]);
            }
            if (!ok) {
                set_status(a.status, kTimeoutCode);
                *abort_flag = 1;
            }
        }
        __syncwarp();
    } else {
        // epilogue: accumulator row r sits in tensor-memory lane r; warp w reaches lanes 32 (w % 4) ..
        const int quad = warp & 3;
        const bool vec = ((uintptr_t)a.out & 15) == 0 && (a.ldo & 3) == 0 && (!a.bias || ((uintptr_t)a.bias & 15) == 0);
        int j = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++j) {
            const int buf = j & 1;
            const int m0 = (tile % tiles_m) * kPfTileM, n0 = (tile / tiles_m) * kPfTileN;
            const int row = m0 + quad * 32 + lane;
            // (the wait ends early once another role has given up)
            bool landed = false;
            {
                const long long t0 = clock64();
                while (!(landed = mbar_try_wait(&acc_full[buf], (j >> 1) & 1))) {
                    if (*abort_flag || clock64() - t0 > 8 * a.wait_cycles) break;
                }
            }
            if (!__all_sync(0xffffffffu, landed)) {  // (the tensor-memory loads are warp-wide)
                set_status(a.status, kTimeoutCode);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            float *orow = a.out + (size_t)row * a.ldo + n0;
#pragma unroll 1
            for (int cb = 0; cb < kPfTileN / 32; ++cb) {
                if (n0 + cb * 32 >= a.N) break;
                float v[32];
                tc_ld_32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * kPfTileN + cb * 32), v);
                if (row < a.R) {
                    if (vec && n0 + cb * 32 + 31 < a.N) {
                        if (a.bias) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float4 bv = __ldg(reinterpret_cast<const float4 *>(a.bias + n0 + cb * 32 + 4 * i));
                                v[4 * i] += bv.x; v[4 * i + 1] += bv.y; v[4 * i + 2] += bv.z; v[4 * i + 3] += bv.w;
                            }
                        }
                        if (a.accumulate) {
                            float4 o[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) o[i] = *reinterpret_cast<const float4 *>(orow + cb * 32 + 4 * i);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                v[4 * i] += o[i].x; v[4 * i + 1] += o[i].y; v[4 * i + 2] += o[i].z; v[4 * i + 3] += o[i].w;
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            *reinterpret_cast<float4 *>(orow + cb * 32 + 4 * i) = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    } else {
                        for (int i = 0; i < 32; ++i) {
                            const int col = n0 + cb * 32 + i;
                            if (col < a.N) {
                                float y = v[i] + (a.bias ? a.bias[col] : 0.f);
                                if (a.accumulate) y += orow[cb * 32 + i];
                                orow[cb * 32 + i] = y;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);  // this warp has read its quadrant of the buffer
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 0) {
        if (lane == 0 && *abort_flag)  // error path only: copies that may still land in this CTA's shared memory
            for (int i = (issued > kPfStages ? issued - kPfStages : 0); i < issued; ++i) mbar_wait(&full[i % kPfStages], (i / kPfStages) & 1);
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(512) : "memory");
    }
}

// Row norm for the many-row pass: one CTA of 256 threads per row, the row held in registers (float4 per thread,
// up to 8192 columns; wider rows are re-read), statistics in fp64, one or two outputs (bf16 hi + lo, row-major)
// from the same statistics.
struct PfNormArgs {
    const float *x;
    int d, kind;  // 0 LayerNorm, 1 RMSNorm
    float eps;
    int n_norms;
    const float *g[2], *b[2];
    __nv_bfloat16 *hi[2], *lo[2];
};
__device__ __forceinline__ void store_hilo4(__nv_bfloat16 *hi, __nv_bfloat16 *lo, size_t idx, float4 y) {
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(y.x, y.y), h23 = __floats2bfloat162_rn(y.z, y.w);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(y.x - __low2float(h01), y.y - __high2float(h01));
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(y.z - __low2float(h23), y.w - __high2float(h23));
    uint2 hv, lv;
    hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
    lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
    *reinterpret_cast<uint2 *>(hi + idx) = hv;
    *reinterpret_cast<uint2 *>(lo + idx) = lv;
}
__global__ void __launch_bounds__(256) prefill_norm_kernel(const PfNormArgs a) {  // d % 4 == 0
    __shared__ double red[32];
    const int r = blockIdx.x, q4 = a.d >> 2;
    const float4 *x4 = reinterpret_cast<const float4 *>(a.x + (size_t)r * a.d);
    float4 v[8];
    double s = 0.0, ss = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = threadIdx.x + 256 * k;
        v[k] = i < q4 ? x4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        s += ((double)v[k].x + (double)v[k].y) + ((double)v[k].z + (double)v[k].w);
    }
    for (int i = threadIdx.x + 2048; i < q4; i += 256) {
        const float4 w = x4[i];
        s += ((double)w.x + (double)w.y) + ((double)w.z + (double)w.w);
    }
    double mean = 0.0;
    if (a.kind == 0) mean = block_sum(s, red) / a.d;
    auto sq = [&](const float4 &w) {
        const double c0 = w.x - mean, c1 = w.y - mean, c2 = w.z - mean, c3 = w.w - mean;
        return (c0 * c0 + c1 * c1) + (c2 * c2 + c3 * c3);
    };
#pragma unroll
    for (int k = 0; k < 8; ++k)
        if (threadIdx.x + 256 * k < q4) ss += sq(v[k]);
    for (int i = threadIdx.x + 2048; i < q4; i += 256) ss += sq(x4[i]);
    const double rstd = rsqrt(block_sum(ss, red) / a.d + (double)a.eps);
#pragma unroll
    for (int n = 0; n < 2; ++n) {
        if (n >= a.n_norms) break;
        const float4 *g4 = reinterpret_cast<const float4 *>(a.g[n]);
        const float4 *b4 = reinterpret_cast<const float4 *>(a.b[n]);
        auto emit = [&](int i, const float4 &w) {
            const float4 g = __ldg(g4 + i);
            const float4 bb = b4 ? __ldg(b4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            float4 y;
            y.x = (float)(((double)w.x - mean) * rstd * (double)g.x + (double)bb.x);
            y.y = (float)(((double)w.y - mean) * rstd * (double)g.y + (double)bb.y);
            y.z = (float)(((double)w.z - mean) * rstd * (double)g.z + (double)bb.z);
            y.w = (float)(((double)w.w - mean) * rstd * (double)g.w + (double)bb.w);
            store_hilo4(a.hi[n], a.lo[n], (size_t)r * a.d + 4 * (size_t)i, y);
        };
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (threadIdx.x + 256 * k < q4) emit(threadIdx.x + 256 * k, v[k]);
        for (int i = threadIdx.x + 2048; i < q4; i += 256) emit(i, x4[i]);
    }
}

// act[r, i] = GELU(t[r, i])  or  SiLU(t[r, i]) * t[r, F + i], four columns per thread; grid (ceil(F / 1024), R); F % 4 == 0
__global__ void __launch_bounds__(256) prefill_act_kernel(const float *__restrict__ t, int ld_t, int F, int swiglu,
                                                          __nv_bfloat16 *hi, __nv_bfloat16 *lo) {
    const int r = blockIdx.y, i = 4 * (blockIdx.x * 256 + threadIdx.x);
    if (i >= F) return;
    const float *tr = t + (size_t)r * ld_t;
    const float4 u = *reinterpret_cast<const float4 *>(tr + i);
    float4 y;
    if (swiglu) {
        const float4 w = *reinterpret_cast<const float4 *>(tr + F + i);
        y = make_float4(silu(u.x) * w.x, silu(u.y) * w.y, silu(u.z) * w.z, silu(u.w) * w.w);
    } else {
        y = make_float4(gelu_erf(u.x), gelu_erf(u.y), gelu_erf(u.z), gelu_erf(u.w));
    }
    store_hilo4(hi, lo, (size_t)r * F + i, y);
}

// prefill_attn_kernel: causal attention of 64 query rows of one (sequence, head) over the cache, which already
// holds this pass's keys / values (the append kernel has run).  Four warps of 16 rows each; K / V chunks of 64
// positions go through two cp.async buffers shared by the four warps; per warp and chunk
//   S [16 x 64] = Q (bf16 hi + lo) K^T,   running max / sum in registers (base-2 exponentials),
//   O [16 x Dh] += P (bf16 hi + lo) V,
// on mma.sync tiles (m16n8k16): the projections carry ~95 % of a prompt pass's arithmetic, so this step stays on
// the warp-level path.  Row m of the sequence sees positions <= len + m.  The result goes to the out-projection
// operand as bf16 hi + lo, row-major; rows that are not fed get zeros.
constexpr int kPaRows = 64, kPaThreads = 128, kPaChunk = 64;
inline size_t prefill_attn_smem(int Dh) {
    return (size_t)2 * kPaRows * (Dh + 8) * 2 + (size_t)2 * 2 * kPaChunk * (Dh + 8) * 2;
}

struct PfAttnArgs {
    const float *q;              // [B * M, d] position-encoded queries
    const __nv_bfloat16 *cache;  // this layer's slab [B][2][H][S][Dh]
    const int32_t *len;          // [B] committed lengths
    const int32_t *n_eff;        // [B] rows fed per sequence
    __nv_bfloat16 *out_hi, *out_lo;  // [B * M, d]
    int M, H, Dh, S, d;
    float scale;
};

__global__ void __launch_bounds__(kPaThreads) prefill_attn_kernel(const PfAttnArgs a) {
    extern __shared__ __align__(16) uint8_t pa_smem[];
    const int mt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int Dh = a.Dh, pitch = Dh + 8;
    const uint32_t pitchB = (uint32_t)pitch * 2u;
    __nv_bfloat16 *Qhi = reinterpret_cast<__nv_bfloat16 *>(pa_smem);
    __nv_bfloat16 *Qlo = Qhi + kPaRows * pitch;
    __nv_bfloat16 *KV = Qlo + kPaRows * pitch;  // buffer i: K at KV + i * 2 * 64 * pitch, V 64 * pitch later
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int nk = Dh >> 4, vpr = Dh >> 3;
    const int len = a.len[b], n = a.n_eff[b];
    const int m_base = mt * kPaRows, r0 = b * a.M;
    const int rows_fed = max(0, min(kPaRows, n - m_base));
    const int p_end = rows_fed > 0 ? min(len + m_base + rows_fed, a.S) : 0;  // positions any row of this tile sees
    const int n_chunks = (p_end + kPaChunk - 1) / kPaChunk;
    const float sc = a.scale * 1.4426950408889634f;
    const __nv_bfloat16 *kc = a.cache + ((size_t)(b * 2) * a.H + h) * a.S * Dh;
    const __nv_bfloat16 *vc = kc + (size_t)a.H * a.S * Dh;

    auto load_chunk = [&](int c) {
        __nv_bfloat16 *Kb = KV + (size_t)(c & 1) * 2 * kPaChunk * pitch, *Vb = Kb + kPaChunk * pitch;
        const int t0 = c * kPaChunk;
        for (int i = tid; i < kPaChunk * vpr; i += kPaThreads) {
            const int pp = i / vpr, v8 = i % vpr, pos = t0 + pp;
            __nv_bfloat16 *dk = Kb + pp * pitch + v8 * 8, *dv = Vb + pp * pitch + v8 * 8;
            if (pos < p_end) {
                cp_async16(dk, kc + (size_t)pos * Dh + v8 * 8);
                cp_async16(dv, vc + (size_t)pos * Dh + v8 * 8);
            } else {  // masked positions: P is 0 there, and 0 x these zeros stays 0
                *reinterpret_cast<uint4 *>(dk) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4 *>(dv) = make_uint4(0, 0, 0, 0);
            }
        }
        cp_async_commit();
    };
    if (n_chunks > 0) load_chunk(0);
    // Q rows of this tile as bf16 hi / lo
    for (int i = tid; i < kPaRows * vpr; i += kPaThreads) {
        const int ml = i / vpr, v8 = i % vpr, m = m_base + ml;
        float qv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) qv[u] = 0.f;
        if (m < n) {
            const float *src = a.q + (size_t)(r0 + m) * a.d + h * Dh + v8 * 8;
            const float4 x0 = *reinterpret_cast<const float4 *>(src), x1 = *reinterpret_cast<const float4 *>(src + 4);
            qv[0] = x0.x; qv[1] = x0.y; qv[2] = x0.z; qv[3] = x0.w; qv[4] = x1.x; qv[5] = x1.y; qv[6] = x1.z; qv[7] = x1.w;
        }
        __nv_bfloat16 hq[8], lq[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            hq[u] = __float2bfloat16_rn(qv[u]);
            lq[u] = __float2bfloat16_rn(qv[u] - __bfloat162float(hq[u]));
        }
        *reinterpret_cast<uint4 *>(Qhi + ml * pitch + v8 * 8) = *reinterpret_cast<uint4 *>(hq);
        *reinterpret_cast<uint4 *>(Qlo + ml * pitch + v8 * 8) = *reinterpret_cast<uint4 *>(lq);
    }

    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int row_lo = m_base + 16 * warp;           // this warp's rows: row_lo + g, row_lo + g + 8
    const int warp_end = len + row_lo + 15;           // last position any of them sees

    for (int c = 0; c < n_chunks; ++c) {
        if (c + 1 < n_chunks) load_chunk(c + 1); else cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();  // chunk c (and, first time, Q) is in shared memory
        const int t0 = c * kPaChunk;
        if (t0 <= warp_end && row_lo < n) {
            const __nv_bfloat16 *Kb = KV + (size_t)(c & 1) * 2 * kPaChunk * pitch, *Vb = Kb + kPaChunk * pitch;
            float s[8][4];
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
            const uint32_t qa = smem_u32(Qhi) + (uint32_t)(16 * warp + (lane & 15)) * pitchB + (uint32_t)(lane >> 4) * 16u;
            const uint32_t ql = qa + (uint32_t)kPaRows * pitchB;
            const uint32_t ka = smem_u32(Kb) + (uint32_t)((lane & 7) + 8 * (lane >> 4)) * pitchB + (uint32_t)((lane >> 3) & 1) * 16u;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                if (ks < nk) {
                    uint32_t a0, a1, a2, a3, c0, c1, c2, c3;
                    ldmatrix_x4(qa + ks * 32, a0, a1, a2, a3);
                    ldmatrix_x4(ql + ks * 32, c0, c1, c2, c3);
#pragma unroll
                    for (int j2 = 0; j2 < 4; ++j2) {  // 16 positions: (0-7: k lo, k hi), (8-15: k lo, k hi)
                        uint32_t k0, k1, k2, k3;
                        ldmatrix_x4(ka + (uint32_t)(16 * j2) * pitchB + ks * 32, k0, k1, k2, k3);
                        mma_bf16(s[2 * j2], a0, a1, a2, a3, k0, k1);
                        mma_bf16(s[2 * j2], c0, c1, c2, c3, k0, k1);
                        mma_bf16(s[2 * j2 + 1], a0, a1, a2, a3, k2, k3);
                        mma_bf16(s[2 * j2 + 1], c0, c1, c2, c3, k2, k3);
                    }
                }
            }
            // mask, running max / sum (rows g and g + 8)
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
                const int m = row_lo + g + 8 * hrow;
                const int last = m < n ? len + m : -1;  // last visible position
                float mx = -INFINITY;
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int pos = t0 + 8 * j + 2 * t + e;
                        const float v = pos <= last ? s[j][2 * hrow + e] * sc : -INFINITY;
                        s[j][2 * hrow + e] = v;
                        mx = fmaxf(mx, v);
                    }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run[hrow], mx);
                float f = 1.f, sum = 0.f;
                if (m_new > -INFINITY) {
                    f = exp2f(m_run[hrow] - m_new);  // 0 on the first non-empty block
#pragma unroll
                    for (int j = 0; j < 8; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float pv = exp2f(s[j][2 * hrow + e] - m_new);
                            s[j][2 * hrow + e] = pv;
                            sum += pv;
                        }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) s[j][2 * hrow] = s[j][2 * hrow + 1] = 0.f;
                }
                m_run[hrow] = m_new;
                l_run[hrow] = l_run[hrow] * f + sum;  // this thread's share; lanes are summed at the end
#pragma unroll
                for (int j = 0; j < 16; ++j) { o[j][2 * hrow] *= f; o[j][2 * hrow + 1] *= f; }
            }
            // O += P V: k = 16 positions per step, n = the head's columns
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t ph[4], pl[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {  // a0: (row g, k 2t..) a1: (row g+8, ..) a2: (row g, k 8+2t..) a3: (row g+8, ..)
                    const int j = 2 * kk + (q >> 1), hrow = q & 1;
                    const float x0 = s[j][2 * hrow], x1 = s[j][2 * hrow + 1];
                    const __nv_bfloat162 hv = __floats2bfloat162_rn(x0, x1);
                    ph[q] = *reinterpret_cast<const uint32_t *>(&hv);
                    pl[q] = pack_bf16x2(x0 - __low2float(hv), x1 - __high2float(hv));
                }
                const uint32_t va = smem_u32(Vb) + (uint32_t)(16 * kk + (lane & 15)) * pitchB;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < 2 * nk) {
                        uint32_t b0, b1;
                        ldmatrix_x2_trans(va + j * 16, b0, b1);
                        mma_bf16(o[j], ph[0], ph[1], ph[2], ph[3], b0, b1);
                        mma_bf16(o[j], pl[0], pl[1], pl[2], pl[3], b0, b1);
                    }
                }
            }
        }
        __syncthreads();  // everyone is done with this buffer before it is refilled
    }
    cp_async_wait<0>();
    // output: rows g, g + 8 of this warp; columns 8 j + 2 t, + 1
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
        float L = l_run[hrow];
        L += __shfl_xor_sync(0xffffffffu, L, 1);
        L += __shfl_xor_sync(0xffffffffu, L, 2);
        const int m = row_lo + g + 8 * hrow;
        if (m >= a.M) continue;
        const float inv = (m < n && L > 0.f) ? 1.f / L : 0.f;
        const size_t base = (size_t)(r0 + m) * a.d + h * Dh + 2 * t;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (j < 2 * nk) {
                const float y0 = o[j][2 * hrow] * inv, y1 = o[j][2 * hrow + 1] * inv;
                const __nv_bfloat162 hv = __floats2bfloat162_rn(y0, y1);
                const __nv_bfloat162 lv = __floats2bfloat162_rn(y0 - __low2float(hv), y1 - __high2float(hv));
                *reinterpret_cast<__nv_bfloat162 *>(a.out_hi + base + 8 * j) = hv;
                *reinterpret_cast<__nv_bfloat162 *>(a.out_lo + base + 8 * j) = lv;
            }
        }
    }
}

// prefill_attn_tc_kernel (head dim 128): the same causal attention on the 5th-generation tensor core, 128 query rows
// of one (sequence, head) per CTA, 128 positions per chunk, scores, probabilities and output in tensor memory:
//   S [128 rows x 128 positions] = Q (bf16 hi + lo, 128-byte-swizzled tiles in shared memory) x K chunk^T (straight
//                                  from the TMA copy of the cache): 2 x 8 MMAs of K = 16 head dims;
//   thread r of warps 0-3 owns query row r = tensor-memory lane r: it reads its row of S, keeps the row's running
//   maximum and sum in registers (no exchange between threads), and writes P = exp2(S - max) back over the same
//   columns as packed bf16 hi and lo (per group of 32 positions: 16 columns hi, 16 columns lo);
//   O [128 rows x 128 head dims] += P (hi, then lo: the A operand read from tensor memory) x V chunk (the B operand,
//                                  head dims contiguous: MN-major): 2 x 8 MMAs of K = 16 positions.
// S is double-buffered (256 columns) so that the scores of chunk c + 1 are computed while the threads work on chunk
// c; O takes 128 columns.  The running maximum is only raised when a chunk exceeds it by more than 2^8 (the sums and
// O absorb the factor), so that rescaling O - a read and a write of the thread's 128 columns - is rare.
// Warp 4 issues the MMAs, warp 5 the K / V copies (two stages each).  Every wait is bounded.
constexpr int kPtRows = 128, kPtChunk = 128, kPtThreads = 192;
constexpr int kPtQBytes = 2 * 128 * 128;             // one of hi / lo: two 64-column panels of 128 rows x 128 bytes
constexpr int kPtKvBytes = 2 * 128 * 128;            // one K or V chunk, the same shape
constexpr size_t kPtSmem = 1024 + 2 * kPtQBytes + 4 * kPtKvBytes + 256;
constexpr float kPtMaxSlack = 8.f;

struct PtAttnArgs {
    const float *q;              // [B * M, d] position-encoded queries
    const int32_t *len;          // [B] committed lengths
    const int32_t *n_eff;        // [B] rows fed per sequence
    __nv_bfloat16 *out_hi, *out_lo;  // [B * M, d]
    int M, H, S, d;
    int kv_row0;                 // first row of this layer in the cache seen as rows of 128 bf16
    float scale;
    long long wait_cycles;
    int32_t *status;
};

__device__ __forceinline__ void tc_st_16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
        "tcgen05.wait::st.sync.aligned;\n" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
        "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
// 64 consecutive columns of this thread's lane in one round trip
__device__ __forceinline__ void tc_ld_64(uint32_t taddr, float (&v)[64]) {
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%64];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
// 32 columns of this thread's lane; completion is awaited by tc_wait_st
__device__ __forceinline__ void tc_st_32u_nowait(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] x B[smem descriptor]
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__global__ void __launch_bounds__(kPtThreads, 1)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap tmKV, const PtAttnArgs a) {
    extern __shared__ uint8_t pt_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)pt_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *qhi = smem, *qlo = smem + kPtQBytes, *kring = smem + 2 * kPtQBytes, *vring = kring + 2 * kPtKvBytes;
    uint64_t *bars = (uint64_t *)(vring + 2 * kPtKvBytes);
    uint64_t *k_full = bars, *k_free = bars + 2, *v_full = bars + 4, *v_free = bars + 6, *s_full = bars + 8;
    uint64_t *p_ready = bars + 10, *o_done = bars + 11;
    uint32_t *tmem_slot = (uint32_t *)(bars + 12);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    constexpr int Dh = 128;
    const int mt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int len = a.len[b], n = a.n_eff[b];
    const int m_base = mt * kPtRows, r0 = b * a.M;
    const int rows_fed = max(0, min(kPtRows, n - m_base));
    if (rows_fed == 0) {  // nothing fed in this tile: zeros for its rows
        for (int i = tid; i < kPtRows * (Dh / 8); i += kPtThreads) {
            const int m = m_base + i / (Dh / 8);
            if (m < a.M) {
                const size_t off = (size_t)(r0 + m) * a.d + h * Dh + (i % (Dh / 8)) * 8;
                *reinterpret_cast<uint4 *>(a.out_hi + off) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4 *>(a.out_lo + off) = make_uint4(0, 0, 0, 0);
            }
        }
        return;
    }
    const int p_end = min(len + m_base + rows_fed, a.S);  // positions any row of this tile sees
    const int n_chunks = (p_end + kPtChunk - 1) / kPtChunk;
    const int krow0 = a.kv_row0 + ((b * 2) * a.H + h) * a.S, vrow0 = krow0 + a.H * a.S;

    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < 10; ++i) mbar_init(&bars[i], 1);
        mbar_init(p_ready, 128);
        mbar_init(o_done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Q rows of this tile as bf16 hi / lo (warps 0-3): consecutive threads take consecutive 8-column pieces of a row,
    // all sixteen loads of a thread in flight together
    if (tid < kPtRows) {
        float4 x0[16], x1[16];
#pragma unroll
        for (int it = 0; it < 16; ++it) {
            const int u = it * kPtRows + tid, row = u >> 4, g8 = u & 15, m = m_base + row;
            x0[it] = x1[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m < n) {
                const float *src = a.q + (size_t)(r0 + m) * a.d + h * Dh + g8 * 8;
                x0[it] = __ldg(reinterpret_cast<const float4 *>(src));
                x1[it] = __ldg(reinterpret_cast<const float4 *>(src + 4));
            }
        }
#pragma unroll
        for (int it = 0; it < 16; ++it) {
            const int u = it * kPtRows + tid, row = u >> 4, g8 = u & 15;
            const float qv[8] = {x0[it].x, x0[it].y, x0[it].z, x0[it].w, x1[it].x, x1[it].y, x1[it].z, x1[it].w};
            __nv_bfloat16 hq[8], lq[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                hq[e] = __float2bfloat16_rn(qv[e]);
                lq[e] = __float2bfloat16_rn(qv[e] - __bfloat162float(hq[e]));
            }
            const uint32_t off = (uint32_t)(g8 >> 3) * 16384u + sw128(row, g8 & 7);
            *reinterpret_cast<uint4 *>(qhi + off) = *reinterpret_cast<uint4 *>(hq);
            *reinterpret_cast<uint4 *>(qlo + off) = *reinterpret_cast<uint4 *>(lq);
        }
    }
    fence_async_proxy();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tS = tmem, tO = tmem + 256;  // S / P of chunk c at tS + 128 (c & 1)
    auto wait = [&](uint64_t *bar, uint32_t parity) {  // keeps every role's control flow intact once anything has timed out
        if (*abort_flag) return;
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity)) {
            if (*abort_flag) return;
            if (clock64() - t0 > a.wait_cycles) {
                set_status(a.status, kTimeoutCode);
                *abort_flag = 1;
                return;
            }
        }
    };

    if (warp == 5) {
        if (lane == 0) {
            int issued_k = 0, issued_v = 0;
            for (int c = 0; c < n_chunks && !*abort_flag; ++c) {
                const int s = c & 1;
                if (c >= 2) wait(&k_free[s], ((c >> 1) - 1) & 1);
                if (*abort_flag) break;
                mbar_expect_tx(&k_full[s], kPtKvBytes);
                tma_load_2d(kring + s * kPtKvBytes, &tmKV, 0, krow0 + c * kPtChunk, &k_full[s]);
                tma_load_2d(kring + s * kPtKvBytes + 16384, &tmKV, 64, krow0 + c * kPtChunk, &k_full[s]);
                ++issued_k;
                if (c >= 2) wait(&v_free[s], ((c >> 1) - 1) & 1);
                if (*abort_flag) break;
                mbar_expect_tx(&v_full[s], kPtKvBytes);
                tma_load_2d(vring + s * kPtKvBytes, &tmKV, 0, vrow0 + c * kPtChunk, &v_full[s]);
                tma_load_2d(vring + s * kPtKvBytes + 16384, &tmKV, 64, vrow0 + c * kPtChunk, &v_full[s]);
                ++issued_v;
            }
            if (*abort_flag) {  // error path only: copies still in flight into this CTA's shared memory
                for (int c = max(0, issued_k - 2); c < issued_k; ++c) mbar_wait(&k_full[c & 1], (c >> 1) & 1);
                for (int c = max(0, issued_v - 2); c < issued_v; ++c) mbar_wait(&v_full[c & 1], (c >> 1) & 1);
            }
        }
        __syncwarp();
    } else if (warp == 4) {
        if (lane == 0) {
            const uint32_t idS = umma_idesc_bf16(128, 128), idO = umma_idesc_bf16(128, 128) | (1u << 16);  // B of P V: MN-major
            auto issue_s = [&](int c) {
                const int s = c & 1;
                wait(&k_full[s], (c >> 1) & 1);
                if (*abort_flag) return;
                tc_fence_after();
                const uint32_t ka = smem_u32(kring + s * kPtKvBytes), qa = smem_u32(qhi), ql = smem_u32(qlo);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // k = 16 head dims per step; panel ks / 4
                    tc_mma_bf16(tS + 128 * s, umma_desc(qa + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                                umma_desc(ka + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024), idS, ks ? 1u : 0u);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc_mma_bf16(tS + 128 * s, umma_desc(ql + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                                umma_desc(ka + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024), idS, 1u);
                tc_commit(&s_full[s]);
                tc_commit(&k_free[s]);
            };
            issue_s(0);
            for (int c = 0; c < n_chunks && !*abort_flag; ++c) {
                const int s = c & 1;
                if (c + 1 < n_chunks) issue_s(c + 1);
                wait(p_ready, c & 1);
                wait(&v_full[s], (c >> 1) & 1);
                if (*abort_flag) break;
                tc_fence_after();
                const uint32_t va = smem_u32(vring + s * kPtKvBytes), tP = tS + 128 * s;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // k = 16 positions per step: two 8-row groups of the V tile; P hi
                    tc_mma_bf16_ta(tO, tP + 32 * (ks >> 1) + 8 * (ks & 1), umma_desc(va + ks * 2048, 16384, 1024), idO, (c | ks) ? 1u : 0u);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // P lo
                    tc_mma_bf16_ta(tO, tP + 32 * (ks >> 1) + 16 + 8 * (ks & 1), umma_desc(va + ks * 2048, 16384, 1024), idO, 1u);
                tc_commit(o_done);
                tc_commit(&v_free[s]);
            }
        }
        __syncwarp();
    } else {
        // ---------------- softmax and output: thread = query row = tensor-memory lane ----------------
        const int m = m_base + tid;
        const int last = m < n ? len + m : -1;  // last visible position
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        const float sc = a.scale * 1.4426950408889634f;
        float m_run = -INFINITY, l_run = 0.f;
        for (int c = 0; c < n_chunks; ++c) {
            const uint32_t tSc = tS + 128 * (c & 1) + lane_sel;
            const int pos0 = c * kPtChunk;
            wait(&s_full[c & 1], (c >> 1) & 1);
            tc_fence_after();
            // the row's 128 scores in two round trips, kept in registers for both passes
            float v0[64], v1[64];
            tc_ld_64(tSc, v0);
            tc_ld_64(tSc + 64, v1);
            float mc = -INFINITY;
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                v0[i] = pos0 + i <= last ? v0[i] * sc : -INFINITY;
                v1[i] = pos0 + 64 + i <= last ? v1[i] * sc : -INFINITY;
                mc = fmaxf(mc, fmaxf(v0[i], v1[i]));
            }
            const float m_new = (mc > m_run + kPtMaxSlack || m_run == -INFINITY) ? fmaxf(m_run, mc) : m_run;
            const float f = m_new > -INFINITY ? exp2f(m_run - m_new) : 1.f;  // 0 on the first non-empty chunk
            const float m_ref = m_new > -INFINITY ? m_new : 0.f;             // (all masked: every p is exp2(-inf) = 0)
            float sum = 0.f;
            auto emit = [&](const float (&v)[64], int half) {  // P of 64 positions: per 32 of them 16 columns hi, 16 lo
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t w[32];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float p0 = exp2f(v[32 * g + 2 * i] - m_ref), p1 = exp2f(v[32 * g + 2 * i + 1] - m_ref);
                        sum += p0 + p1;
                        const __nv_bfloat162 hv = __floats2bfloat162_rn(p0, p1);
                        w[i] = *reinterpret_cast<const uint32_t *>(&hv);
                        w[16 + i] = pack_bf16x2(p0 - __low2float(hv), p1 - __high2float(hv));
                    }
                    tc_st_32u_nowait(tSc + 64 * half + 32 * g, w);
                }
            };
            emit(v0, 0);
            emit(v1, 1);
            tc_wait_st();
            l_run = l_run * f + sum;
            m_run = m_new;
            // the accumulated O row moves to the new maximum, once P V of the previous chunk has written it; the
            // tensor-memory loads and stores are warp-wide, so the warp goes together (f = 1 where nothing moved)
            if (c > 0 && __any_sync(0xffffffffu, f != 1.f)) {
                wait(o_done, (c - 1) & 1);
                tc_fence_after();
#pragma unroll 1
                for (int g = 0; g < 4; ++g) {
                    float o[32];
                    tc_ld_32(tO + lane_sel + 32 * g, o);
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] *= f;
                    tc_st_32(tO + lane_sel + 32 * g, o);
                }
            }
            tc_fence_before();
            mbar_arrive(p_ready);
        }
        wait(o_done, (n_chunks - 1) & 1);
        tc_fence_after();
        {
            const bool store = m < a.M && !*abort_flag;  // (the loads are warp-wide: every lane takes them)
            const float inv = (m < n && l_run > 0.f) ? 1.f / l_run : 0.f;
            const size_t base = (size_t)(r0 + (store ? m : 0)) * a.d + h * Dh;
#pragma unroll 1
            for (int g = 0; g < 2; ++g) {
                float o[64];
                tc_ld_64(tO + lane_sel + 64 * g, o);
                if (store) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {  // eight head dims: 16 bytes of hi, 16 bytes of lo
                        uint32_t hw[4], lw[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float y0 = o[8 * i + 2 * e] * inv, y1 = o[8 * i + 2 * e + 1] * inv;
                            const __nv_bfloat162 hv = __floats2bfloat162_rn(y0, y1);
                            hw[e] = *reinterpret_cast<const uint32_t *>(&hv);
                            lw[e] = pack_bf16x2(y0 - __low2float(hv), y1 - __high2float(hv));
                        }
                        *reinterpret_cast<uint4 *>(a.out_hi + base + 64 * g + 8 * i) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4 *>(a.out_lo + base + 64 * g + 8 * i) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    }
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(512) : "memory");
    }
}

}  // namespace ssd

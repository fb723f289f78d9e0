// K-query causal attention over the contiguous per-layer KV cache (Section "KV Caching", Figure 1;
// the K+1 verification rows of Figure 2 are the queries).  The position axis is split over CTAs
// (each streams a slice of keys/values once for all of a sequence's rows of one head) and the
// slices are merged with their log-sum-exp statistics.
#pragma once
#include "common.cuh"
#include "rowops.cuh"

namespace ssd {

constexpr int kAttnTile = 64;      // positions per shared-memory tile
constexpr int kAttnThreads = 128;

struct AttnArgs {
    const float *q;     // [R, d] position-encoded queries (fp32)
    const void *cache;  // this layer: [B][2][H][S][Dh]
    const int32_t *len; // [B] committed lengths
    int M, H, Dh, S, d;
    int chunk, n_split; // positions per split (multiple of kAttnTile)
    float scale;
    RowInfo ri;
    float *part_m, *part_l, *part_o;  // [R, H, n_split], ..., [R, H, n_split, Dh]
};

template <typename T>
__device__ __forceinline__ void load8(const T *p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8<float>(const float *p, float (&v)[8]) {
    float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[8]) {
    uint4 u = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// grid (n_split, B*H); MR = compile-time bound on rows per sequence
template <typename T, int MR>
__global__ void __launch_bounds__(kAttnThreads) attn_partial_kernel(AttnArgs a) {
    extern __shared__ __align__(16) uint8_t attn_smem[];
    const int split = blockIdx.x, b = blockIdx.y / a.H, h = blockIdx.y % a.H;
    const int Dh = a.Dh, pitch = Dh + 16 / (int)sizeof(T);  // +16 B per row: conflict-free 16 B reads
    float *Qs = reinterpret_cast<float *>(attn_smem);                  // [MR][Dh]
    float *Ps = Qs + MR * Dh;                                          // [MR][kAttnTile]
    float *fac = Ps + MR * kAttnTile;                                  // [MR]
    float *run_m = fac + MR, *run_l = run_m + MR;                      // [MR] each
    T *Ks = reinterpret_cast<T *>(run_l + MR);                         // [kAttnTile][pitch]
    T *Vs = Ks + kAttnTile * pitch;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_rows = a.ri.n_eff[b];
    const int len = a.len[b];
    const int r0 = b * a.M;
    const int p_begin = split * a.chunk;
    const int p_end = min(p_begin + a.chunk, len + n_rows);

    float o[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m) o[m] = 0.f;
    if (tid < MR) { run_m[tid] = -INFINITY; run_l[tid] = 0.f; }

    if (p_begin < p_end) {
        for (int i = tid; i < n_rows * Dh; i += kAttnThreads) {
            int m = i / Dh, e = i % Dh;
            Qs[m * Dh + e] = a.q[(size_t)(r0 + m) * a.d + h * Dh + e];
        }
        const T *kc = (const T *)a.cache + ((size_t)(b * 2) * a.H + h) * a.S * Dh;
        const T *vc = kc + (size_t)a.H * a.S * Dh;
        const int vec_per_row = Dh / 8;
        for (int t0 = p_begin; t0 < p_end; t0 += kAttnTile) {
            const int np = min(kAttnTile, p_end - t0);
            __syncthreads();  // previous tile fully consumed (and Qs / run_* visible on the first pass)
            for (int i = tid; i < np * vec_per_row; i += kAttnThreads) {
                int p = i / vec_per_row, v8 = i % vec_per_row;
                const size_t g = (size_t)(t0 + p) * Dh + v8 * 8;
                if (sizeof(T) == 2) {
                    *reinterpret_cast<uint4 *>(Ks + p * pitch + v8 * 8) = *reinterpret_cast<const uint4 *>(kc + g);
                    *reinterpret_cast<uint4 *>(Vs + p * pitch + v8 * 8) = *reinterpret_cast<const uint4 *>(vc + g);
                } else {
                    const float4 *ks = reinterpret_cast<const float4 *>(kc + g), *vs = reinterpret_cast<const float4 *>(vc + g);
                    float4 *kd = reinterpret_cast<float4 *>(Ks + p * pitch + v8 * 8), *vd = reinterpret_cast<float4 *>(Vs + p * pitch + v8 * 8);
                    kd[0] = ks[0]; kd[1] = ks[1]; vd[0] = vs[0]; vd[1] = vs[1];
                }
            }
            __syncthreads();
            // scores: thread = (position p, row parity); each key row is read once for its rows
            {
                const int p = tid % kAttnTile, mg = tid / kAttnTile;  // mg in {0,1}
                float s[(MR + 1) / 2];
#pragma unroll
                for (int i = 0; i < (MR + 1) / 2; ++i) s[i] = 0.f;
                if (p < np) {
                    for (int v8 = 0; v8 < vec_per_row; ++v8) {
                        float kv[8];
                        load8<T>(Ks + p * pitch + v8 * 8, kv);
#pragma unroll
                        for (int i = 0; i < (MR + 1) / 2; ++i) {
                            const int m = mg + 2 * i;
                            if (m < n_rows) {
                                const float *qv = Qs + m * Dh + v8 * 8;
#pragma unroll
                                for (int e = 0; e < 8; ++e) s[i] = fmaf(qv[e], kv[e], s[i]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < (MR + 1) / 2; ++i) {
                    const int m = mg + 2 * i;
                    if (m < MR && m < n_rows) {
                        const bool vis = p < np && (t0 + p) <= len + m;  // causal: row m sees positions <= len + m
                        Ps[m * kAttnTile + p] = vis ? s[i] * a.scale : -INFINITY;
                    }
                }
            }
            __syncthreads();
            // running softmax statistics: one warp per row
            for (int m = warp; m < n_rows; m += kAttnThreads / 32) {
                float s0 = Ps[m * kAttnTile + lane], s1 = Ps[m * kAttnTile + lane + 32];
                float tmax = warp_max(fmaxf(s0, s1));
                float m_old = run_m[m], m_new = fmaxf(m_old, tmax);
                float f = 1.f, e0 = 0.f, e1 = 0.f;
                if (m_new > -INFINITY) {
                    f = __expf(m_old - m_new);  // exp(-inf) = 0 on the first non-empty tile
                    e0 = __expf(s0 - m_new);
                    e1 = __expf(s1 - m_new);
                }
                Ps[m * kAttnTile + lane] = e0;
                Ps[m * kAttnTile + lane + 32] = e1;
                float sum = warp_sum(e0 + e1);
                if (lane == 0) {
                    fac[m] = f;
                    run_m[m] = m_new;
                    run_l[m] = run_l[m] * f + sum;
                }
            }
            __syncthreads();
            // o[m][e] = o[m][e] * f[m] + sum_p P[m][p] V[p][e];  thread = column e
            if (tid < Dh) {
#pragma unroll
                for (int m = 0; m < MR; ++m)
                    if (m < n_rows) o[m] *= fac[m];
                for (int p = 0; p < np; ++p) {
                    const float v = to_f32(Vs[p * pitch + tid]);
#pragma unroll
                    for (int m = 0; m < MR; ++m)
                        if (m < n_rows) o[m] = fmaf(Ps[m * kAttnTile + p], v, o[m]);
                }
            }
        }
    }
    __syncthreads();
    for (int m = 0; m < a.M; ++m) {
        const size_t slot = ((size_t)(r0 + m) * a.H + h) * a.n_split + split;
        const bool live = m < n_rows && m < MR;
        if (tid == 0) {
            a.part_m[slot] = live ? run_m[m] : -INFINITY;
            a.part_l[slot] = live ? run_l[m] : 0.f;
        }
        if (tid < Dh) {
            float val = 0.f;
#pragma unroll
            for (int mm = 0; mm < MR; ++mm)
                if (mm == m) val = o[mm];
            a.part_o[slot * Dh + tid] = live ? val : 0.f;
        }
    }
}

struct CombineArgs {
    const float *part_m, *part_l, *part_o;
    int H, Dh, n_split, d;
    Operand out;       // attention output rows as GEMM operand (may be empty)
    float *out_f32;    // optional plain fp32 copy [R, d]
    float *x;          // residual stream for the bias job (may be null)
    BiasJob bias;
};

// grid (H, R)
__global__ void attn_combine_kernel(CombineArgs a) {
    const int h = blockIdx.x, r = blockIdx.y;
    const size_t base = ((size_t)r * a.H + h) * a.n_split;
    float mx = -INFINITY;
    for (int s = 0; s < a.n_split; ++s) mx = fmaxf(mx, a.part_m[base + s]);
    for (int e = threadIdx.x; e < a.Dh; e += blockDim.x) {
        float L = 0.f, acc = 0.f;
        if (mx > -INFINITY) {
            for (int s = 0; s < a.n_split; ++s) {
                const float pm = a.part_m[base + s];
                if (pm == -INFINITY) continue;
                const float w = __expf(pm - mx);
                L = fmaf(a.part_l[base + s], w, L);
                acc = fmaf(a.part_o[(base + s) * a.Dh + e], w, acc);
            }
        }
        const float val = L > 0.f ? acc / L : 0.f;
        const int col = h * a.Dh + e;
        if (a.out.f32 || a.out.hi) store_operand(a.out, r, col, val);
        if (a.out_f32) a.out_f32[(size_t)r * a.d + col] = val;
        if (a.x && (a.bias.b0 || a.bias.b1)) {
            float add = (a.bias.b0 ? a.bias.b0[col] : 0.f) + (a.bias.b1 ? a.bias.b1[col] : 0.f);
            a.x[(size_t)r * a.d + col] += add;
        }
    }
}

}  // namespace ssd

// Row-wise steps between the GEMMs: row bookkeeping + rotary table, embedding gather, norms,
// MLP activation, rotary + KV append.  All tiny next to the weight stream; one CTA per row.
#pragma once
#include "common.cuh"

namespace ssd {

// A buffer to pre-load before a GEMM accumulates into it: dst[r, i] = bias ? bias[i] : 0.
struct InitJob {
    float *dst;
    const float *bias;
    int n, ld;
};
// dst[r, i] += bias[i]  (residual-stream biases of the projections that accumulate into x)
struct BiasJob {
    const float *b0, *b1;
};

struct SetupArgs {
    int B, M;                 // rows per sequence (maximum)
    const int32_t *n_rows;    // [B] or null (= M)
    const int32_t *len;       // [B] committed lengths
    int s_max, pos_limit;     // cache capacity; position-table rows (0 = unlimited)
    int rotary_dim;
    float rotary_base;
    RowInfo ri;
    int32_t *status;
};

// One CTA per row r = b*M + j.
__global__ void setup_rows_kernel(SetupArgs a) {
    const int r = blockIdx.x, b = r / a.M, j = r % a.M;
    int n = a.n_rows ? a.n_rows[b] : a.M;
    n = max(0, min(n, a.M));
    const int len = a.len[b];
    bool fits = len + n <= a.s_max && (a.pos_limit == 0 || len + n <= a.pos_limit);
    if (!fits) {
        n = 0;
        if (threadIdx.x == 0) set_status(a.status, -3 /* capacity */);
    }
    int pos = len + j;
    int lim = a.s_max - 1;
    if (a.pos_limit && a.pos_limit - 1 < lim) lim = a.pos_limit - 1;
    if (pos > lim) pos = lim;  // rows that are not fed still index tables safely
    if (threadIdx.x == 0) {
        a.ri.seq[r] = b;
        a.ri.pos[r] = pos;
        a.ri.valid[r] = j < n;
        if (j == 0) a.ri.n_eff[b] = n;
    }
    const int half = a.rotary_dim / 2;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        // angle = pos * base^(-2i/rd), in double: fp32 loses the low bits of pos * theta at long context
        double theta = (double)pos * exp2(-2.0 * i / a.rotary_dim * log2((double)a.rotary_base));
        double s, c;
        sincos(theta, &s, &c);
        a.ri.rope_cos[(size_t)r * half + i] = (float)c;
        a.ri.rope_sin[(size_t)r * half + i] = (float)s;
    }
}

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// x[r, :] = E[token] (+ P[pos])
template <typename T>
__global__ void embed_kernel(const T *__restrict__ E, const T *__restrict__ P, const int32_t *tokens, int tok_stride,
                             int M, int vocab, int d, RowInfo ri, float *x) {
    const int r = blockIdx.x, b = r / M, j = r % M;
    int tok = ri.valid[r] ? tokens[(size_t)b * tok_stride + j] : 0;  // rows that are not fed read nothing
    tok = max(0, min(tok, vocab - 1));
    const T *e = E + (size_t)tok * d;
    const T *p = P ? P + (size_t)ri.pos[r] * d : nullptr;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = to_f32(e[i]);
        if (p) v = v + to_f32(p[i]);
        x[(size_t)r * d + i] = v;
    }
}

struct NormArgs {
    const float *x;
    int d, kind;  // 0 LayerNorm, 1 RMSNorm
    float eps;
    int n_norms;  // 1 or 2 outputs from the same statistics
    const float *g[2], *b[2];
    Operand out[2];
    InitJob init[3];
    int n_init;
};

__global__ void norm_kernel(NormArgs a) {
    __shared__ double red[32];
    const int r = blockIdx.x;
    const float *x = a.x + (size_t)r * a.d;
    double mean = 0.0, rstd;
    if (a.kind == 0) {
        double s = 0.0;
        for (int i = threadIdx.x; i < a.d; i += blockDim.x) s += x[i];
        mean = block_sum(s, red) / a.d;
        double v = 0.0;
        for (int i = threadIdx.x; i < a.d; i += blockDim.x) {
            double c = x[i] - mean;
            v += c * c;
        }
        v = block_sum(v, red) / a.d;
        rstd = rsqrt(v + (double)a.eps);
    } else {
        double s = 0.0;
        for (int i = threadIdx.x; i < a.d; i += blockDim.x) s += (double)x[i] * x[i];
        s = block_sum(s, red) / a.d;
        rstd = rsqrt(s + (double)a.eps);
    }
    for (int k = 0; k < a.n_norms; ++k) {
        const float *g = a.g[k], *bb = a.b[k];
        for (int i = threadIdx.x; i < a.d; i += blockDim.x) {
            double y = ((double)x[i] - mean) * rstd * (double)g[i];
            if (bb) y += (double)bb[i];
            store_operand(a.out[k], r, i, (float)y);
        }
    }
    for (int k = 0; k < a.n_init; ++k) {
        const InitJob &job = a.init[k];
        float *dst = job.dst + (size_t)r * job.ld;
        for (int i = threadIdx.x; i < job.n; i += blockDim.x) dst[i] = job.bias ? job.bias[i] : 0.f;
    }
}

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752f)); }
__device__ __forceinline__ float silu(float v) { return v / (1.f + expf(-v)); }

// act[r, i] = GELU(t[r, i])  or  SiLU(t[r, i]) * t[r, F + i];  grid (ceil(F/256), R)
__global__ void act_kernel(const float *__restrict__ t, int ld_t, int F, int swiglu, Operand out, float *x, int d,
                           BiasJob bias) {
    const int r = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < F) {
        const float *tr = t + (size_t)r * ld_t;
        float v = swiglu ? silu(tr[i]) * tr[F + i] : gelu_erf(tr[i]);
        store_operand(out, r, i, v);
    }
    if (blockIdx.x == 0 && (bias.b0 || bias.b1)) {
        for (int k = threadIdx.x; k < d; k += blockDim.x) {
            float add = (bias.b0 ? bias.b0[k] : 0.f) + (bias.b1 ? bias.b1[k] : 0.f);
            x[(size_t)r * d + k] += add;
        }
    }
}

struct RopeArgs {
    const float *qkv;  // [R, 3d]
    float *q_out;      // [R, d] position-encoded queries
    void *cache;       // slab of this layer: [B][2][H][S][Dh]
    int d, H, Dh, S, rotary_dim;
    RowInfo ri;
};

// rotary on q and k (half-split pairing), then append k, v to the cache at the row's position
template <typename T>
__global__ void rope_append_kernel(RopeArgs a) {
    const int r = blockIdx.x;
    const int b = a.ri.seq[r], pos = a.ri.pos[r], valid = a.ri.valid[r];
    const int half = a.rotary_dim / 2;
    const float *row = a.qkv + (size_t)r * 3 * a.d;
    const float *cs = a.ri.rope_cos + (size_t)r * half, *sn = a.ri.rope_sin + (size_t)r * half;
    T *kc = (T *)a.cache + (size_t)b * 2 * a.H * a.S * a.Dh;
    T *vc = kc + (size_t)a.H * a.S * a.Dh;
    for (int idx = threadIdx.x; idx < a.d; idx += blockDim.x) {
        const int h = idx / a.Dh, e = idx % a.Dh;
        float q = row[idx], k = row[a.d + idx], v = row[2 * a.d + idx];
        if (e < a.rotary_dim) {
            const int j = e < half ? e : e - half;
            const float c = cs[j], s = sn[j];
            if (e < half) {
                q = q * c - row[idx + half] * s;
                k = k * c - row[a.d + idx + half] * s;
            } else {
                q = row[idx - half] * s + q * c;
                k = row[a.d + idx - half] * s + k * c;
            }
        }
        a.q_out[(size_t)r * a.d + idx] = q;
        if (valid) {
            const size_t off = ((size_t)h * a.S + pos) * a.Dh + e;
            kc[off] = from_f32<T>(k);
            vc[off] = from_f32<T>(v);
        }
    }
}

}  // namespace ssd

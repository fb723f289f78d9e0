// The whole decoder forward of a verification pass (or a draft step) as ONE persistent
// cooperative kernel, one CTA per SM.
//
// Why: a pass is a chain of ~8 small dependent steps per layer; as separate launches the HBM
// stream stops at every boundary (the paper's point in Section "Autoregressive vs Speculative
// Sampling" is that the pass is memory-bound, so idle HBM time is the cost).  Here the weight
// stream never stops: a producer thread per CTA walks the static schedule of every weight tile
// this CTA will need in the whole forward and keeps a deep shared-memory ring full with TMA
// copies, running ahead across phase boundaries; only the small activation tiles wait for the
// grid barrier of the phase that produces them.
//
// Roles in a CTA (288 threads):
//   warps 0-7   consumers: bf16 tensor-core MMAs on (weight tile, activation tile) stages,
//               fp32 reductions of partial tiles into the output (bias added by the unit that
//               holds k-chunk 0); between GEMM phases the same warps run the small phases
//               (row set-up, embedding, norm, activation, attention with rotary + KV append +
//               split merge), which leave every GEMM operand in global memory already split
//               into bf16 hi + lo, and the grid barriers
//   warp 8      producer: TMA issue for weight tiles (free-running) and operand tiles (gated
//               by the grid barrier of the phase that wrote them)
// Every wait (mbarrier, grid barrier) is bounded; on time-out SSD_E_TIMEOUT is recorded, the CTA
// stops taking work, waits (bounded) for its copies in flight and returns.
#pragma once
#include <cuda.h>

#include "attention.cuh"
#include "common.cuh"
#include "gemm.cuh"
#include "rowops.cuh"

namespace ssd {

constexpr int kConsumerWarps = 8;
constexpr int kWorkThreads = kConsumerWarps * 32;  // 256: everyone but the producer
constexpr int kPersistThreads = kWorkThreads + 32;
constexpr int kAttnThreadsP = 256;

struct alignas(64) LayerDesc {
    CUtensorMap tm[4];  // qkv, o, in, out
    const float *ln1_g, *ln1_b, *b_qkv, *b_o, *ln2_g, *ln2_b, *b_in, *b_out;
};
struct alignas(64) ModelDesc {
    CUtensorMap tm_lm;
    const float *lnf_g, *lnf_b;
    const void *pad[6];
    // LayerDesc layers[] follow
};
__device__ __forceinline__ const LayerDesc *layer_desc(const ModelDesc *md, int l) {
    return reinterpret_cast<const LayerDesc *>(md + 1) + l;
}

enum { OP_XN1 = 0, OP_XN2 = 1, OP_AO = 2, OP_ACT = 3 };

struct alignas(64) FwdParams {
    // GEMM operands in global memory, bf16 hi rows [0, rk) then lo rows [rk, 2 rk), row pitch = K:
    // normalised rows (two sets for parallel-residual blocks), attention output, MLP activation.
    CUtensorMap tm_op[4];  // box 64 x (2 rk), 128-byte swizzle
    __nv_bfloat16 *op[4];
    int op_ld[4];
    int rk;
    const ModelDesc *md;
    // architecture
    int n_layers, d, H, Dh, F, d_in, V, norm_kind, swiglu, parallel, rotary_dim, learned_pos, is_bf16_emb;
    float eps, rotary_base, attn_scale;
    // rows
    int B, M, R;
    const int32_t *tokens;
    int tok_stride;
    const int32_t *n_rows;
    const void *tok_emb, *pos_emb;
    int pos_limit;
    // cache
    uint8_t *cache;
    size_t layer_bytes;
    const int32_t *len;
    int S;
    int32_t *status;
    // workspace
    RowInfo ri;
    float *x, *qkv, *t_in, *logits;
    float *part_m, *part_l, *part_o;
    unsigned *tickets;  // [B*H]
    unsigned *gbar;     // grid barrier counter (zeroed before launch)
    int chunk, n_split;
    int want_logits;
    int stages, attn_smem_off;  // ring depth; byte offset of the attention scratch
    unsigned long long *trace;  // optional: CTA 0 stamps the global timer after every grid barrier
};

struct GemmDesc {
    const CUtensorMap *tmW, *tmX;
    int N, Kd, n_tiles, kchunks;
    int need;  // grid barriers that must have completed before its operand exists
    float *out;
    int ldo;
    const float *bias;
};

__device__ __forceinline__ int n_gemms(const FwdParams &p) { return 4 * p.n_layers + (p.want_logits ? 1 : 0); }
__device__ __forceinline__ int barriers_per_layer(const FwdParams &p) { return p.parallel ? 4 : 8; }

// GEMM number gi in execution order.  sequential: qkv, o, in, out; parallel: qkv, in, o, out.
// Barrier count before layer l: 2 (set-up; embedding + first norm) + barriers_per_layer * l.
//   sequential layer: qkv | attention | o | norm2 | in | act | out | next norm   (8 barriers)
//   parallel layer:   qkv, in | attention + act | o, out | next norms            (4 barriers)
__device__ __forceinline__ GemmDesc gemm_desc(const FwdParams &p, int gi) {
    GemmDesc g;
    const int l = gi >> 2, e = gi & 3;
    const int base = 2 + barriers_per_layer(p) * l;
    if (l >= p.n_layers) {  // LM head
        g.tmW = &p.md->tm_lm; g.tmX = &p.tm_op[OP_XN1];
        g.N = p.V; g.Kd = p.d; g.need = base; g.out = p.logits; g.ldo = p.V; g.bias = nullptr;
    } else {
        const LayerDesc *ld = layer_desc(p.md, l);
        int kind;  // 0 qkv, 1 o, 2 in, 3 out
        if (p.parallel) kind = (e == 0) ? 0 : (e == 1) ? 2 : (e == 2) ? 1 : 3;
        else kind = e;
        g.tmW = &ld->tm[kind];
        if (kind == 0) {
            g.tmX = &p.tm_op[OP_XN1]; g.N = 3 * p.d; g.Kd = p.d; g.need = base;
            g.out = p.qkv; g.ldo = 3 * p.d; g.bias = ld->b_qkv;
        } else if (kind == 1) {
            g.tmX = &p.tm_op[OP_AO]; g.N = p.d; g.Kd = p.d; g.need = base + 2;
            g.out = p.x; g.ldo = p.d; g.bias = ld->b_o;
        } else if (kind == 2) {
            g.tmX = &p.tm_op[p.parallel ? OP_XN2 : OP_XN1]; g.N = p.d_in; g.Kd = p.d; g.need = p.parallel ? base : base + 4;
            g.out = p.t_in; g.ldo = p.d_in; g.bias = ld->b_in;
        } else {
            g.tmX = &p.tm_op[OP_ACT]; g.N = p.d; g.Kd = p.F; g.need = p.parallel ? base + 2 : base + 6;
            g.out = p.x; g.ldo = p.d; g.bias = ld->b_out;
        }
    }
    g.n_tiles = (g.N + kTileN - 1) / kTileN;
    g.kchunks = (g.Kd + kTileK - 1) / kTileK;
    return g;
}

// This CTA's contiguous share of a GEMM's (tile, k-chunk) units.
__device__ __forceinline__ void unit_range(const GemmDesc &g, int &c0, int &c1) {
    const long long total = (long long)g.n_tiles * g.kchunks;
    c0 = (int)(total * blockIdx.x / gridDim.x);
    c1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
}

__device__ __forceinline__ void named_bar(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned *p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }

// operand element (r, i) of a hi/lo buffer
__device__ __forceinline__ void store_hilo(__nv_bfloat16 *buf, int rk, int ld, int r, int i, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    buf[(size_t)r * ld + i] = h;
    buf[(size_t)(rk + r) * ld + i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

struct alignas(16) Shared {
    volatile int released;  // grid barriers completed so far
    volatile int abort;     // some wait in this CTA gave up
    volatile int go;        // snapshot of !abort taken inside the grid barrier: uniform for all work threads
    int flag;
};

// Grid barrier for the 320 work threads of every CTA.  Returns false (the same value in every work
// thread of the CTA) once a wait has timed out anywhere in this CTA; the caller then stops.
__device__ __forceinline__ bool grid_sync(const FwdParams &p, Shared *sh, int &epoch) {
    fence_async_proxy();  // this thread's operand writes must be seen by other CTAs' TMA reads
    __threadfence();
    named_bar(1, kWorkThreads);
    ++epoch;
    if (threadIdx.x == 0) {
        bool ok = sh->abort == 0;
        if (ok) {
            red_release_add(p.gbar, 1u);
            const unsigned target = (unsigned)epoch * gridDim.x;
            if (ld_acquire(p.gbar) < target) {
                const long long t0 = clock64();
                while (ld_acquire(p.gbar) < target) {
                    if (clock64() - t0 > kWaitCycles) { ok = false; break; }
                }
            }
        }
        if (!ok) {
            set_status(p.status, kTimeoutCode);
            sh->abort = 1;
        }
        sh->go = ok ? 1 : 0;
        __threadfence();
        sh->released = epoch;
        if (p.trace && blockIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            p.trace[epoch] = t;
        }
    }
    named_bar(1, kWorkThreads);
    return sh->go != 0;
}

// ---- non-GEMM phases (256 work threads) -------------------------------------------------------

__device__ __forceinline__ float block_sum_work(float v, float *red) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    named_bar(2, kWorkThreads);
    if (lane == 0) red[w] = v;
    named_bar(2, kWorkThreads);
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < kConsumerWarps; ++i) t += red[i];
    return t;
}
__device__ __forceinline__ double block_sum_work(double v, double *red) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    named_bar(2, kWorkThreads);
    if (lane == 0) red[w] = v;
    named_bar(2, kWorkThreads);
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < kConsumerWarps; ++i) t += red[i];
    return t;
}

// zero a [R, n] fp32 buffer (row pitch ld), spread over the whole grid
__device__ __forceinline__ void grid_zero(float *dst, int R, int n, int ld) {
    const long long total = (long long)R * n;
    for (long long i = (long long)blockIdx.x * kWorkThreads + threadIdx.x; i < total;
         i += (long long)gridDim.x * kWorkThreads) {
        int r = (int)(i / n), c = (int)(i % n);
        dst[(size_t)r * ld + c] = 0.f;
    }
}

// Norm of every row of x into hi/lo operand buffers (one or two gain/bias sets from the same
// statistics); one CTA per row.
__device__ __forceinline__ void norm_phase(const FwdParams &p, const float *g1, const float *b1, int op1,
                                           const float *g2, const float *b2, int op2, double *red) {
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const float *x = p.x + (size_t)r * p.d;
        double s1 = 0.0, s2 = 0.0;
        for (int i = threadIdx.x; i < p.d; i += kWorkThreads) {
            const double v = __ldcg(x + i);
            s1 += v;
            s2 += v * v;
        }
        s1 = block_sum_work(s1, red);
        s2 = block_sum_work(s2, red);
        double mean = 0.0, var;
        if (p.norm_kind == 0) {
            mean = s1 / p.d;
            var = s2 / p.d - mean * mean;
            if (var < 0.0) var = 0.0;
        } else {
            var = s2 / p.d;
        }
        const float mu = (float)mean, rs = (float)rsqrt(var + (double)p.eps);
        for (int i = threadIdx.x; i < p.d; i += kWorkThreads) {
            const float c = (__ldcg(x + i) - mu) * rs;
            store_hilo(p.op[op1], p.rk, p.op_ld[op1], r, i, c * g1[i] + (b1 ? b1[i] : 0.f));
            if (g2) store_hilo(p.op[op2], p.rk, p.op_ld[op2], r, i, c * g2[i] + (b2 ? b2[i] : 0.f));
        }
    }
}

// MLP activation of t_in into the hi/lo operand of the down projection, spread over the grid
__device__ __forceinline__ void act_phase(const FwdParams &p) {
    const long long total = (long long)p.R * p.F;
    for (long long i = (long long)blockIdx.x * kWorkThreads + threadIdx.x; i < total;
         i += (long long)gridDim.x * kWorkThreads) {
        const int r = (int)(i / p.F), c = (int)(i % p.F);
        const float *t = p.t_in + (size_t)r * p.d_in;
        const float v = p.swiglu ? silu(__ldcg(t + c)) * __ldcg(t + p.F + c) : gelu_erf(__ldcg(t + c));
        store_hilo(p.op[OP_ACT], p.rk, p.op_ld[OP_ACT], r, c, v);
    }
}

__device__ __forceinline__ void setup_phase(const FwdParams &p) {
    const int half = p.rotary_dim / 2;
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const int b = r / p.M, j = r % p.M;
        int n = p.n_rows ? p.n_rows[b] : p.M;
        n = max(0, min(n, p.M));
        const int len = p.len[b];
        const bool fits = len + n <= p.S && (p.pos_limit == 0 || len + n <= p.pos_limit);
        if (!fits) {
            n = 0;
            if (threadIdx.x == 0) set_status(p.status, -3);
        }
        int pos = len + j, lim = p.S - 1;
        if (p.pos_limit && p.pos_limit - 1 < lim) lim = p.pos_limit - 1;
        if (pos > lim) pos = lim;
        if (threadIdx.x == 0) {
            p.ri.seq[r] = b;
            p.ri.pos[r] = pos;
            p.ri.valid[r] = j < n;
            if (j == 0) p.ri.n_eff[b] = n;
        }
        for (int i = threadIdx.x; i < half; i += kWorkThreads) {
            double theta = (double)pos * exp2(-2.0 * i / p.rotary_dim * log2((double)p.rotary_base));
            double s, c;
            sincos(theta, &s, &c);
            p.ri.rope_cos[(size_t)r * half + i] = (float)c;
            p.ri.rope_sin[(size_t)r * half + i] = (float)s;
        }
    }
}

__device__ __forceinline__ void embed_phase(const FwdParams &p) {
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const int b = r / p.M, j = r % p.M;
        int tok = __ldcg(p.ri.valid + r) ? p.tokens[(size_t)b * p.tok_stride + j] : 0;
        tok = max(0, min(tok, p.V - 1));
        const int pos = __ldcg(p.ri.pos + r);
        for (int i = threadIdx.x; i < p.d; i += kWorkThreads) {
            float v;
            if (p.is_bf16_emb) {
                v = __bfloat162float(((const __nv_bfloat16 *)p.tok_emb)[(size_t)tok * p.d + i]);
                if (p.learned_pos) v = v + __bfloat162float(((const __nv_bfloat16 *)p.pos_emb)[(size_t)pos * p.d + i]);
            } else {
                v = ((const float *)p.tok_emb)[(size_t)tok * p.d + i];
                if (p.learned_pos) v = v + ((const float *)p.pos_emb)[(size_t)pos * p.d + i];
            }
            p.x[(size_t)r * p.d + i] = v;
        }
    }
}

// Attention of one (sequence, head, split) item by 256 threads: rotary on q, the new rows' keys /
// values taken from qkv (rotary, cache rounding) and appended to the cache by the split that owns
// their positions, running softmax, P.V; the last split to finish merges all splits into ao.
template <int MR>
__device__ void attention_item(const FwdParams &p, int layer, int item, uint8_t *scratch, Shared *sh) {
    const int split = item % p.n_split, bh = item / p.n_split, b = bh / p.H, h = bh % p.H;
    const int Dh = p.Dh, pitch = Dh + 8, d = p.d;
    float *Qs = reinterpret_cast<float *>(scratch);
    float *Ps = Qs + MR * Dh;
    float *fac = Ps + MR * kAttnTile;
    float *run_m = fac + MR, *run_l = run_m + MR;
    __nv_bfloat16 *Ks = reinterpret_cast<__nv_bfloat16 *>(run_l + MR);
    __nv_bfloat16 *Vs = Ks + kAttnTile * pitch;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_rows = __ldcg(p.ri.n_eff + b);
    const int len = p.len[b];
    const int r0 = b * p.M;
    const int p_begin = split * p.chunk;
    const int p_end = min(p_begin + p.chunk, len + n_rows);
    const int half = p.rotary_dim / 2;
    constexpr int MH = (MR + 1) / 2;
    float o[MH];
#pragma unroll
    for (int m = 0; m < MH; ++m) o[m] = 0.f;
    const int e_col = tid & 127, m_par = tid >> 7;  // P.V: column e, rows of parity m_par

    if (tid < kAttnThreadsP) {
        if (tid < MR) { run_m[tid] = -INFINITY; run_l[tid] = 0.f; }
        if (p_begin < p_end) {
            for (int i = tid; i < n_rows * Dh; i += kAttnThreadsP) {
                const int m = i / Dh, e = i % Dh, r = r0 + m;
                const float *row = p.qkv + (size_t)r * 3 * d + h * Dh;
                float q = __ldcg(row + e);
                if (e < p.rotary_dim) {
                    const int j = e < half ? e : e - half;
                    const float c = __ldcg(p.ri.rope_cos + (size_t)r * half + j), s = __ldcg(p.ri.rope_sin + (size_t)r * half + j);
                    q = e < half ? q * c - __ldcg(row + e + half) * s : __ldcg(row + e - half) * s + q * c;
                }
                Qs[m * Dh + e] = q;
            }
            __nv_bfloat16 *kc = (__nv_bfloat16 *)(p.cache + (size_t)layer * p.layer_bytes) + ((size_t)(b * 2) * p.H + h) * p.S * Dh;
            __nv_bfloat16 *vc = kc + (size_t)p.H * p.S * Dh;
            const int vec_per_row = Dh / 8;
            for (int t0 = p_begin; t0 < p_end; t0 += kAttnTile) {
                const int np = min(kAttnTile, p_end - t0);
                named_bar(3, kAttnThreadsP);
                for (int i = tid; i < np * vec_per_row; i += kAttnThreadsP) {
                    const int pp = i / vec_per_row, v8 = i % vec_per_row, pos = t0 + pp;
                    uint4 kq, vq;
                    if (pos < len) {
                        const size_t g = (size_t)pos * Dh + v8 * 8;
                        kq = __ldcs(reinterpret_cast<const uint4 *>(kc + g));
                        vq = __ldcs(reinterpret_cast<const uint4 *>(vc + g));
                    } else {  // a row of this pass: from qkv, position-encoded and rounded as the cache stores it
                        const int r = r0 + (pos - len);
                        const float *krow = p.qkv + (size_t)r * 3 * d + d + h * Dh;
                        const float *vrow = krow + d;
                        __nv_bfloat16 kb[8], vb[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t) {
                            const int e = v8 * 8 + t;
                            float k = __ldcg(krow + e);
                            if (e < p.rotary_dim) {
                                const int j = e < half ? e : e - half;
                                const float c = __ldcg(p.ri.rope_cos + (size_t)r * half + j), s = __ldcg(p.ri.rope_sin + (size_t)r * half + j);
                                k = e < half ? k * c - __ldcg(krow + e + half) * s : __ldcg(krow + e - half) * s + k * c;
                            }
                            kb[t] = __float2bfloat16_rn(k);
                            vb[t] = __float2bfloat16_rn(__ldcg(vrow + e));
                        }
                        kq = *reinterpret_cast<uint4 *>(kb);
                        vq = *reinterpret_cast<uint4 *>(vb);
                        const size_t g = (size_t)pos * Dh + v8 * 8;  // append: exactly one split owns this position
                        *reinterpret_cast<uint4 *>(kc + g) = kq;
                        *reinterpret_cast<uint4 *>(vc + g) = vq;
                    }
                    *reinterpret_cast<uint4 *>(Ks + pp * pitch + v8 * 8) = kq;
                    *reinterpret_cast<uint4 *>(Vs + pp * pitch + v8 * 8) = vq;
                }
                named_bar(3, kAttnThreadsP);
                {   // scores: thread = (position, row group of 4)
                    const int pp = tid % kAttnTile, mg = tid / kAttnTile;
                    constexpr int MQ = (MR + 3) / 4;
                    float s[MQ];
#pragma unroll
                    for (int i = 0; i < MQ; ++i) s[i] = 0.f;
                    if (pp < np) {
                        for (int v8 = 0; v8 < vec_per_row; ++v8) {
                            float kv[8];
                            load8<__nv_bfloat16>(Ks + pp * pitch + v8 * 8, kv);
#pragma unroll
                            for (int i = 0; i < MQ; ++i) {
                                const int m = mg + 4 * i;
                                if (m < n_rows) {
                                    const float *qv = Qs + m * Dh + v8 * 8;
#pragma unroll
                                    for (int e = 0; e < 8; ++e) s[i] = fmaf(qv[e], kv[e], s[i]);
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int i = 0; i < MQ; ++i) {
                        const int m = mg + 4 * i;
                        if (m < MR && m < n_rows) {
                            const bool vis = pp < np && (t0 + pp) <= len + m;
                            Ps[m * kAttnTile + pp] = vis ? s[i] * p.attn_scale : -INFINITY;
                        }
                    }
                }
                named_bar(3, kAttnThreadsP);
                for (int m = warp; m < n_rows; m += kAttnThreadsP / 32) {
                    float s0 = Ps[m * kAttnTile + lane], s1 = Ps[m * kAttnTile + lane + 32];
                    float tmax = warp_max(fmaxf(s0, s1));
                    float m_old = run_m[m], m_new = fmaxf(m_old, tmax);
                    float f = 1.f, e0 = 0.f, e1 = 0.f;
                    if (m_new > -INFINITY) {
                        f = __expf(m_old - m_new);
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
                named_bar(3, kAttnThreadsP);
                if (e_col < Dh) {
#pragma unroll
                    for (int i = 0; i < MH; ++i) {
                        const int m = 2 * i + m_par;
                        if (m < n_rows) o[i] *= fac[m];
                    }
                    for (int pp = 0; pp < np; ++pp) {
                        const float v = __bfloat162float(Vs[pp * pitch + e_col]);
#pragma unroll
                        for (int i = 0; i < MH; ++i) {
                            const int m = 2 * i + m_par;
                            if (m < n_rows) o[i] = fmaf(Ps[m * kAttnTile + pp], v, o[i]);
                        }
                    }
                }
            }
        }
        named_bar(3, kAttnThreadsP);
        for (int m = 0; m < p.M; ++m) {
            const size_t slot = ((size_t)(r0 + m) * p.H + h) * p.n_split + split;
            const bool live = m < n_rows && m < MR;
            if (tid == 0) {
                p.part_m[slot] = live ? run_m[m] : -INFINITY;
                p.part_l[slot] = live ? run_l[m] : 0.f;
            }
            if (e_col < Dh && (m & 1) == m_par) {
                float val = 0.f;
#pragma unroll
                for (int i = 0; i < MH; ++i)
                    if (2 * i + m_par == m) val = o[i];
                p.part_o[slot * Dh + e_col] = live ? val : 0.f;
            }
        }
        // ticket: the split that finishes last for this (sequence, head) merges them
        __threadfence();
        named_bar(3, kAttnThreadsP);
        if (tid == 0) sh->flag = (atomicAdd(p.tickets + bh, 1u) == (unsigned)(p.n_split - 1));
        named_bar(3, kAttnThreadsP);
        if (sh->flag) {
            __threadfence();
            for (int idx = tid; idx < p.M * Dh; idx += kAttnThreadsP) {
                const int m = idx / Dh, e = idx % Dh;
                const size_t base = ((size_t)(r0 + m) * p.H + h) * p.n_split;
                float mx = -INFINITY;
                for (int s = 0; s < p.n_split; ++s) mx = fmaxf(mx, __ldcg(p.part_m + base + s));
                float L = 0.f, acc = 0.f;
                if (mx > -INFINITY) {
                    for (int s = 0; s < p.n_split; ++s) {
                        const float pm = __ldcg(p.part_m + base + s);
                        if (pm == -INFINITY) continue;
                        const float w = __expf(pm - mx);
                        L = fmaf(__ldcg(p.part_l + base + s), w, L);
                        acc = fmaf(__ldcg(p.part_o + (base + s) * Dh + e), w, acc);
                    }
                }
                store_hilo(p.op[OP_AO], p.rk, p.op_ld[OP_AO], r0 + m, h * Dh + e, L > 0.f ? acc / L : 0.f);
            }
            if (tid == 0) p.tickets[bh] = 0;  // ready for the next layer (a grid barrier lies between)
        }
        named_bar(3, kAttnThreadsP);
    }
}

template <int MR>
__device__ __forceinline__ void attention_phase(const FwdParams &p, int layer, uint8_t *scratch, Shared *sh) {
    const int items = p.B * p.H * p.n_split;
    for (int item = blockIdx.x; item < items; item += gridDim.x) attention_item<MR>(p, layer, item, scratch, sh);
}

// ---- the kernel -----------------------------------------------------------------------------
// NT = padded rows / 8;  MR = compile-time bound on rows per sequence for attention
template <int NT, int MR>
__global__ void __launch_bounds__(kPersistThreads, 1) forward_kernel(const __grid_constant__ FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int kRp = NT * 8;
    constexpr int kXBytes = 2 * kRp * kTileK * 2;  // hi tile followed by lo tile
    constexpr int kStageBytes = kWTileBytes + kXBytes;
    const int S = p.stages;
    uint8_t *ring = smem;
    uint8_t *attn_scratch = smem + p.attn_smem_off;
    uint64_t *fullW = (uint64_t *)(smem + (size_t)S * kStageBytes);
    uint64_t *fullX = fullW + S, *empty = fullX + S;
    Shared *sh = (Shared *)(((uintptr_t)(empty + S) + 15) & ~(uintptr_t)15);
    double *red = (double *)(sh + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&fullW[s], 1);
            mbar_init(&fullX[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        sh->released = 0;
        sh->abort = 0;
        sh->go = 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int NG = n_gemms(p);

    if (warp == kConsumerWarps) {
        // =============================== producer ===============================
        // Two cursors over the same unit sequence.  Weights never change, so their cursor runs as far
        // ahead as the ring allows, across grid barriers; an operand tile is fetched once the phase
        // that wrote it has been released.
        if (lane == 0) {
            int issuedW = 0, issuedX = 0;
            int gw = 0, cw = 0, cw1 = 0, tw = 0, kw = 0;
            int gx = 0, cx = 0, cx1 = 0, kx = 0;
            GemmDesc dw, dx;
            bool have_w = false, have_x = false;
            auto next_w = [&]() {
                for (; gw < NG; ++gw) {
                    dw = gemm_desc(p, gw);
                    unit_range(dw, cw, cw1);
                    if (cw < cw1) { tw = cw / dw.kchunks; kw = cw % dw.kchunks; have_w = true; return; }
                }
                have_w = false;
            };
            auto next_x = [&]() {
                for (; gx < NG; ++gx) {
                    dx = gemm_desc(p, gx);
                    unit_range(dx, cx, cx1);
                    if (cx < cx1) { kx = cx % dx.kchunks; have_x = true; return; }
                }
                have_x = false;
            };
            next_w();
            next_x();
            int seen_release = 0;
            long long idle_since = clock64();
            while ((have_w || have_x) && !sh->abort) {
                bool progressed = false;
                if (have_w) {
                    const int s = issuedW % S;
                    if (issuedW < S || mbar_test_wait(&empty[s], ((issuedW / S) - 1) & 1)) {
                        mbar_expect_tx(&fullW[s], kWTileBytes);
                        tma_load_2d(ring + (size_t)s * kStageBytes, dw.tmW, kw * kTileK, tw * kTileN, &fullW[s]);
                        ++issuedW;
                        progressed = true;
                        if (++kw == dw.kchunks) { kw = 0; ++tw; }
                        if (++cw == cw1) { ++gw; next_w(); }
                    }
                }
                if (have_x && issuedX < issuedW) {
                    if (dx.need > seen_release) {
                        seen_release = sh->released;
                        if (dx.need <= seen_release) fence_async_proxy();  // that phase's writes -> visible to TMA
                    }
                    if (dx.need <= seen_release) {
                        const int s = issuedX % S;
                        mbar_expect_tx(&fullX[s], kXBytes);
                        tma_load_2d(ring + (size_t)s * kStageBytes + kWTileBytes, dx.tmX, kx * kTileK, 0, &fullX[s]);
                        ++issuedX;
                        progressed = true;
                        if (++kx == dx.kchunks) kx = 0;
                        if (++cx == cx1) { ++gx; next_x(); }
                    }
                }
                if (progressed) {
                    idle_since = clock64();
                } else if (clock64() - idle_since > kWaitCycles) {
                    set_status(p.status, kTimeoutCode);
                    sh->abort = 1;
                }
            }
            // error path only: wait (bounded) for copies still in flight before the CTA may exit
            if (sh->abort) {
                for (int i = (issuedW > S ? issuedW - S : 0); i < issuedW; ++i) mbar_wait(&fullW[i % S], (i / S) & 1);
                for (int i = (issuedX > S ? issuedX - S : 0); i < issuedX; ++i) mbar_wait(&fullX[i % S], (i / S) & 1);
            }
        }
    } else {
        // =============================== work warps ===============================
        int epoch = 0, it = 0;  // grid barriers passed; ring stages consumed
        bool alive = true;      // per warp: false once one of its waits gave up
        float acc[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

        // run this CTA's units of GEMM gi
        auto run_gemm = [&](int gi) {
            const GemmDesc g = gemm_desc(p, gi);
            int c0, c1;
            unit_range(g, c0, c1);
            if (c0 >= c1) return;
            int tile = c0 / g.kchunks, kc = c0 % g.kchunks;
            auto flush = [&](int t, bool with_bias) {
                const int n = t * kTileN + warp * 16 + (lane >> 2);
                float b0 = 0.f, b1 = 0.f;
                if (with_bias && g.bias) {
                    if (n < g.N) b0 = __ldg(g.bias + n);
                    if (n + 8 < g.N) b1 = __ldg(g.bias + n + 8);
                }
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const int m0 = 8 * j + (lane & 3) * 2;
                    if (n < g.N) {
                        if (m0 < p.R) atomicAdd(g.out + (size_t)m0 * g.ldo + n, acc[j][0] + b0);
                        if (m0 + 1 < p.R) atomicAdd(g.out + (size_t)(m0 + 1) * g.ldo + n, acc[j][1] + b0);
                    }
                    if (n + 8 < g.N) {
                        if (m0 < p.R) atomicAdd(g.out + (size_t)m0 * g.ldo + n + 8, acc[j][2] + b1);
                        if (m0 + 1 < p.R) atomicAdd(g.out + (size_t)(m0 + 1) * g.ldo + n + 8, acc[j][3] + b1);
                    }
                    acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
                }
            };
            const int arow = lane & 15, achunk = lane >> 4, brow = lane & 7, bsel = lane >> 3;
            bool has_k0 = (kc == 0);  // does the running tile segment include k-chunk 0 (it adds the bias)
            for (int c = c0; c < c1 && alive; ++c, ++it) {
                const int s = it % S;
                if (!mbar_wait(&fullW[s], (it / S) & 1) || !mbar_wait(&fullX[s], (it / S) & 1)) {
                    set_status(p.status, kTimeoutCode);
                    sh->abort = 1;
                    alive = false;
                    break;
                }
                const uint32_t st = smem_u32(ring + (size_t)s * kStageBytes);
                const uint32_t wbase = st + (uint32_t)(warp * 16 + arow) * 128u;
                const uint32_t xbase = st + kWTileBytes + (bsel >= 2 ? kRp * 128 : 0) + (uint32_t)brow * 128u;
#pragma unroll
                for (int ks = 0; ks < kTileK / 16; ++ks) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(wbase + ((uint32_t)((2 * ks + achunk) ^ (arow & 7)) << 4), a0, a1, a2, a3);
#pragma unroll
                    for (int j = 0; j < NT; ++j) {
                        uint32_t h0, h1, l0, l1;
                        ldmatrix_x4(xbase + (uint32_t)j * 1024u + ((uint32_t)((2 * ks + (bsel & 1)) ^ brow) << 4), h0, h1, l0, l1);
                        mma_bf16(acc[j], a0, a1, a2, a3, h0, h1);
                        mma_bf16(acc[j], a0, a1, a2, a3, l0, l1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
                if (++kc == g.kchunks) {
                    flush(tile, has_k0);
                    kc = 0;
                    ++tile;
                    has_k0 = true;
                }
            }
            if (alive && kc != 0) flush(tile, has_k0);
        };

        if (p.trace && blockIdx.x == 0 && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            p.trace[0] = t;
        }
        // ---- phase program (the same structure gemm_desc() encodes) ----
        // `go` is uniform over the work threads (taken inside the grid barrier), so every named barrier
        // below is reached by all of them or by none.
        auto norm_for_layer = [&](int l) {  // operand(s) of layer l's first GEMM(s), or of the LM head
            if (l < p.n_layers) {
                const LayerDesc *ld = layer_desc(p.md, l);
                if (p.parallel) norm_phase(p, ld->ln1_g, ld->ln1_b, OP_XN1, ld->ln2_g, ld->ln2_b, OP_XN2, red);
                else norm_phase(p, ld->ln1_g, ld->ln1_b, OP_XN1, nullptr, nullptr, 0, red);
                grid_zero(p.qkv, p.R, 3 * p.d, 3 * p.d);
                if (p.parallel) grid_zero(p.t_in, p.R, p.d_in, p.d_in);
            } else if (p.want_logits) {
                norm_phase(p, p.md->lnf_g, p.md->lnf_b, OP_XN1, nullptr, nullptr, 0, red);
                grid_zero(p.logits, p.R, p.V, p.V);
            }
        };
        setup_phase(p);
        bool go = grid_sync(p, sh, epoch);
        if (go) {
            embed_phase(p);
            named_bar(2, kWorkThreads);  // the embedding rows are read back by the CTA that wrote them
            norm_for_layer(0);
            go = grid_sync(p, sh, epoch);
        }
        for (int l = 0; l < p.n_layers && go; ++l) {
            run_gemm(4 * l + 0);                       // qkv
            if (p.parallel) run_gemm(4 * l + 1);       // MLP in (same block input)
            if (!(go = grid_sync(p, sh, epoch))) break;
            attention_phase<MR>(p, l, attn_scratch, sh);
            if (p.parallel) act_phase(p);
            if (!(go = grid_sync(p, sh, epoch))) break;
            if (p.parallel) {
                run_gemm(4 * l + 2);                   // out-proj -> x
                run_gemm(4 * l + 3);                   // MLP out  -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
            } else {
                run_gemm(4 * l + 1);                   // out-proj -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
                const LayerDesc *ld = layer_desc(p.md, l);
                norm_phase(p, ld->ln2_g, ld->ln2_b, OP_XN1, nullptr, nullptr, 0, red);
                grid_zero(p.t_in, p.R, p.d_in, p.d_in);
                if (!(go = grid_sync(p, sh, epoch))) break;
                run_gemm(4 * l + 2);                   // MLP in
                if (!(go = grid_sync(p, sh, epoch))) break;
                act_phase(p);
                if (!(go = grid_sync(p, sh, epoch))) break;
                run_gemm(4 * l + 3);                   // MLP out -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
            }
            norm_for_layer(l + 1);
            if (!(go = grid_sync(p, sh, epoch))) break;
        }
        if (go && p.want_logits) run_gemm(4 * p.n_layers);
        if (p.trace && blockIdx.x == 0 && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            p.trace[epoch + 1] = t;
            p.trace[epoch + 2] = 0;
        }
    }
    __syncthreads();
}

}  // namespace ssd

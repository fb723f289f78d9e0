// The whole decoder forward of a verification pass (or a draft step) as ONE persistent
// cooperative kernel, one CTA per SM.
//
// Why: a pass is a chain of ~7 small dependent steps per layer; as separate launches the HBM
// stream stops at every boundary (the paper's point in Section "Autoregressive vs Speculative
// Sampling" is that the pass is memory-bound, so idle HBM time is the cost).  Here the weight
// stream never stops: a producer thread per CTA walks the static schedule of every weight tile
// this CTA will need in the whole forward and keeps a deep shared-memory ring full with TMA
// copies, running ahead across phase boundaries; only the small activation tiles wait for the
// grid barrier of the phase that produces them.
//
// Roles in a CTA (384 threads):
//   warps 0-7   consumers: bf16 tensor-core MMAs on (weight tile, activation tile) stages,
//               fp32 reductions of partial tiles into the output (bias added by the unit that
//               holds k-chunk 0)
//   warps 8-10  transform: fetch the fp32 activation slice of a stage from L2 (cp.async, a few
//               stages ahead) and turn it, in place in shared memory, into the bf16 hi/lo pair
//               the MMAs read -- applying LayerNorm/RMSNorm (row statistics from the previous
//               phase), GELU / SwiGLU, or nothing
//   warp 11     producer: TMA issue for the weight tiles, free-running across phases
// Warps 0-10 also execute the non-GEMM phases (row set-up, embedding, row statistics,
// attention with rotary + KV append + split merge) and the grid barriers.
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
constexpr int kTransformWarps = 3;  // 8 + 3 + 1 = 12 warps: three per SM partition, 168 registers each
constexpr int kXThreads = kTransformWarps * 32;
constexpr int kXAheadMax = 8;  // activation slices in flight per CTA (bounded by the ring depth)
constexpr int kWorkThreads = (kConsumerWarps + kTransformWarps) * 32;  // 352: everyone but the producer
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

enum { XF_IDENT = 0, XF_NORM = 1, XF_GELU = 2, XF_SWIGLU = 3 };

struct alignas(64) FwdParams {
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
    float *x, *qkv, *t_in, *ao, *logits;
    float2 *stats;  // [slot][R] (mean, rstd)
    float *part_m, *part_l, *part_o;
    unsigned *tickets;  // [B*H]
    unsigned *gbar;     // grid barrier counter (zeroed before launch)
    int chunk, n_split;
    int want_logits;
    int stages, attn_smem_off;  // ring depth; byte offset of the attention scratch
    unsigned long long *trace;  // optional: CTA 0 stamps the global timer after every grid barrier
};

struct GemmDesc {
    const CUtensorMap *tmW;
    const float *srcA;  // fp32 activations [R, lda]; SwiGLU reads a second slice at column colB
    int lda, colB;
    int N, Kd, n_tiles, kchunks;
    int xf, need;    // transform kind; grid barriers that must have completed before its activations exist
    float *out;
    int ldo;
    const float *bias, *g, *b;
    int stat_slot;
};

__device__ __forceinline__ int n_gemms(const FwdParams &p) { return 4 * p.n_layers + (p.want_logits ? 1 : 0); }
__device__ __forceinline__ int barriers_per_layer(const FwdParams &p) { return p.parallel ? 4 : 7; }

// GEMM number gi in execution order.  sequential: qkv, o, in, out; parallel: qkv, in, o, out.
__device__ __forceinline__ GemmDesc gemm_desc(const FwdParams &p, int gi) {
    GemmDesc g;
    const int l = gi >> 2, e = gi & 3;
    const int base = 2 + barriers_per_layer(p) * l;
    if (l >= p.n_layers) {  // LM head
        g.tmW = &p.md->tm_lm; g.srcA = p.x; g.lda = p.d; g.colB = 0;
        g.N = p.V; g.Kd = p.d; g.xf = XF_NORM; g.need = base; g.out = p.logits; g.ldo = p.V;
        g.bias = nullptr; g.g = p.md->lnf_g; g.b = p.md->lnf_b; g.stat_slot = 2 * p.n_layers;
    } else {
        const LayerDesc *ld = layer_desc(p.md, l);
        int kind;  // 0 qkv, 1 o, 2 in, 3 out
        if (p.parallel) kind = (e == 0) ? 0 : (e == 1) ? 2 : (e == 2) ? 1 : 3;
        else kind = e;
        g.tmW = &ld->tm[kind]; g.colB = 0; g.g = nullptr; g.b = nullptr; g.stat_slot = 0;
        if (kind == 0) {
            g.srcA = p.x; g.lda = p.d; g.N = 3 * p.d; g.Kd = p.d; g.xf = XF_NORM; g.need = base;
            g.out = p.qkv; g.ldo = 3 * p.d; g.bias = ld->b_qkv; g.g = ld->ln1_g; g.b = ld->ln1_b; g.stat_slot = 2 * l;
        } else if (kind == 1) {
            g.srcA = p.ao; g.lda = p.d; g.N = p.d; g.Kd = p.d; g.xf = XF_IDENT; g.need = base + 2;
            g.out = p.x; g.ldo = p.d; g.bias = ld->b_o;
        } else if (kind == 2) {
            g.srcA = p.x; g.lda = p.d; g.N = p.d_in; g.Kd = p.d; g.xf = XF_NORM; g.need = p.parallel ? base : base + 4;
            g.out = p.t_in; g.ldo = p.d_in; g.bias = ld->b_in; g.g = ld->ln2_g; g.b = ld->ln2_b;
            g.stat_slot = p.parallel ? 2 * l : 2 * l + 1;
        } else {
            g.srcA = p.t_in; g.lda = p.d_in; g.N = p.d; g.Kd = p.F; g.xf = p.swiglu ? XF_SWIGLU : XF_GELU; g.colB = p.F;
            g.need = p.parallel ? base + 2 : base + 5;
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
__device__ __forceinline__ void cp_async16(void *dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// wait until at most n (0..8) of this thread's most recent cp.async groups are pending
__device__ __forceinline__ void cp_async_wait_dyn(int n) {
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        case 6: cp_async_wait<6>(); break;
        case 7: cp_async_wait<7>(); break;
        default: cp_async_wait<8>(); break;
    }
}

struct alignas(16) Shared {
    volatile int released;  // grid barriers completed so far
    volatile int abort;     // some wait in this CTA gave up
    volatile int go;        // snapshot of !abort taken inside the grid barrier: uniform for all work threads
    volatile int abort_x;   // set by a transform warp only, read by both after their own barrier
    float mean[kMaxRows], rstd[kMaxRows];
    int flag;
    int pad[3];
};

// Grid barrier for the 320 work threads of every CTA.  Returns false (the same value in every work
// thread of the CTA) once a wait has timed out anywhere in this CTA; the caller then stops.
__device__ __forceinline__ bool grid_sync(const FwdParams &p, Shared *sh, int &epoch) {
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

// ---- non-GEMM phases (320 work threads) -------------------------------------------------------

__device__ __forceinline__ float block_sum_work(float v, float *red) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    named_bar(2, kWorkThreads);
    if (lane == 0) red[w] = v;
    named_bar(2, kWorkThreads);
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < kConsumerWarps + kTransformWarps; ++i) t += red[i];
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
    for (int i = 0; i < kConsumerWarps + kTransformWarps; ++i) t += red[i];
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

// (mean, rstd) of row r of x -> stats[slot][r]; one CTA per row
__device__ __forceinline__ void row_stats_phase(const FwdParams &p, int slot, double *red) {
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
        if (threadIdx.x == 0) p.stats[(size_t)slot * p.R + r] = make_float2((float)mean, (float)rsqrt(var + (double)p.eps));
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
                p.ao[(size_t)(r0 + m) * d + h * Dh + e] = L > 0.f ? acc / L : 0.f;
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
    constexpr int kRawBytes = kRp * kTileK * 4;  // one fp32 activation slice == one hi/lo bf16 pair
    const int kStageBytes = kWTileBytes + (p.swiglu ? 2 : 1) * kRawBytes;
    const int S = p.stages;
    uint8_t *ring = smem;
    uint8_t *attn_scratch = smem + p.attn_smem_off;
    uint64_t *fullW = (uint64_t *)(smem + (size_t)S * kStageBytes);
    uint64_t *xrdy = fullW + S, *empty = xrdy + S;
    Shared *sh = (Shared *)(((uintptr_t)(empty + S) + 15) & ~(uintptr_t)15);
    double *red = (double *)(sh + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&fullW[s], 1);
            mbar_init(&xrdy[s], kTransformWarps);
            mbar_init(&empty[s], kConsumerWarps);
        }
        sh->released = 0;
        sh->abort = 0;
        sh->go = 1;
        sh->abort_x = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int NG = n_gemms(p);

    if (warp == kConsumerWarps + kTransformWarps) {
        // =============================== producer: weight tiles only ===============================
        // Weights never change, so this stream does not wait for any phase: it runs as far ahead
        // of the consumers as the ring allows, across grid barriers.
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int gi = 0; gi < NG && ok; ++gi) {
                const GemmDesc g = gemm_desc(p, gi);
                int c0, c1;
                unit_range(g, c0, c1);
                int tile = c0 / g.kchunks, kc = c0 % g.kchunks;
                for (int c = c0; c < c1; ++c, ++issued) {
                    const int s = issued % S;
                    if (sh->abort || (issued >= S && !mbar_wait(&empty[s], ((issued / S) - 1) & 1))) {
                        set_status(p.status, kTimeoutCode);
                        sh->abort = 1;
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(&fullW[s], kWTileBytes);
                    tma_load_2d(ring + (size_t)s * kStageBytes, g.tmW, kc * kTileK, tile * kTileN, &fullW[s]);
                    if (++kc == g.kchunks) { kc = 0; ++tile; }
                }
            }
            // error path only: wait (bounded) for copies still in flight before the CTA may exit
            if (!ok)
                for (int i = (issued > S ? issued - S : 0); i < issued; ++i) mbar_wait(&fullW[i % S], (i / S) & 1);
        }
    } else {
        // =============================== work warps ===============================
        int epoch = 0, it = 0;  // grid barriers passed; ring stages consumed
        bool alive = true;
        float acc[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

        // run this CTA's units of GEMM gi (consumers: MMA; transform warps: operand preparation)
        auto run_gemm = [&](int gi) {
            const GemmDesc g = gemm_desc(p, gi);
            int c0, c1;
            unit_range(g, c0, c1);
            if (c0 >= c1) return;
            const int n_units = c1 - c0;
            if (warp >= kConsumerWarps) {
                // ---------------- transform warps ----------------
                const int tt = threadIdx.x - kConsumerWarps * 32;  // 0..95
                const int kp = tt & 31, rw = tt >> 5;              // k pair; row = kTransformWarps * i + rw
                constexpr int kRowsPer = (kRp + kTransformWarps - 1) / kTransformWarps;
                constexpr int kChunksPer = (kRp * 16 + kXThreads - 1) / kXThreads;
                const bool two = g.xf == XF_SWIGLU;
                if (g.xf == XF_NORM) {
                    for (int r = tt; r < p.R; r += kXThreads) {
                        const float2 st = __ldcg(p.stats + (size_t)g.stat_slot * p.R + r);
                        sh->mean[r] = st.x;
                        sh->rstd[r] = st.y;
                    }
                }
                // fetch of unit j's activation slice(s) into its ring slot (16-byte cp.async chunks)
                const int it0 = it;  // ring stage of this GEMM's first unit
                auto issue = [&](int j) {
                    const int its = it0 + j, s = its % S;
                    if (its >= S && !mbar_wait(&empty[s], ((its / S) - 1) & 1)) {
                        set_status(p.status, kTimeoutCode);
                        sh->abort = 1;
                        sh->abort_x = 1;
                    } else {
                        uint8_t *xa = ring + (size_t)s * kStageBytes + kWTileBytes;
                        const int k0 = ((c0 + j) % g.kchunks) * kTileK;
#pragma unroll
                        for (int q = 0; q < kChunksPer; ++q) {
                            const int ch = tt + kXThreads * q, r = ch >> 4, c16 = ch & 15, k = k0 + c16 * 4;
                            if (r < p.R && k < g.Kd) {
                                const float *src = g.srcA + (size_t)r * g.lda + k;
                                cp_async16(xa + r * 256 + c16 * 16, src);
                                if (two) cp_async16(xa + kRawBytes + r * 256 + c16 * 16, src + g.colB);
                            }
                        }
                    }
                    cp_async_commit();
                };
                // exactly `ahead` groups are committed before the loop and one per iteration, so that
                // "at most `ahead` groups pending" means "slice j has landed" whatever n_units is
                const int ahead = min(kXAheadMax, S - 2);
                for (int j = 0; j < ahead; ++j) {
                    if (j < n_units) issue(j); else cp_async_commit();
                }
                int kc = c0 % g.kchunks;
                for (int j = 0; j < n_units; ++j, ++it) {
                    if (j + ahead < n_units) issue(j + ahead); else cp_async_commit();
                    cp_async_wait_dyn(ahead);
                    named_bar(4, kXThreads);  // every thread's chunks of slice j have landed
                    if (sh->abort_x) { alive = false; break; }  // the same value in all transform warps here
                    const int s = it % S;
                    uint8_t *xa = ring + (size_t)s * kStageBytes + kWTileBytes;
                    const float *ra = reinterpret_cast<const float *>(xa);
                    const float *rb = reinterpret_cast<const float *>(xa + kRawBytes);
                    float2 v[kRowsPer];
                    const int k = kc * kTileK + 2 * kp;
                    float2 gg = make_float2(1.f, 1.f), bb = make_float2(0.f, 0.f);
                    if (g.xf == XF_NORM && k < g.Kd) {
                        gg = __ldg(reinterpret_cast<const float2 *>(g.g + k));
                        if (g.b) bb = __ldg(reinterpret_cast<const float2 *>(g.b + k));
                    }
#pragma unroll
                    for (int i = 0; i < kRowsPer; ++i) {
                        const int r = kTransformWarps * i + rw;
                        float2 a = make_float2(0.f, 0.f);
                        if (r < p.R && k < g.Kd) {  // rows / columns beyond the data were not fetched
                            a = *reinterpret_cast<const float2 *>(ra + r * kTileK + 2 * kp);
                            if (g.xf == XF_NORM) {
                                const float mu = sh->mean[r], rs = sh->rstd[r];
                                a.x = (a.x - mu) * rs * gg.x + bb.x;
                                a.y = (a.y - mu) * rs * gg.y + bb.y;
                            } else if (g.xf == XF_GELU) {
                                a.x = gelu_erf(a.x);
                                a.y = gelu_erf(a.y);
                            } else if (g.xf == XF_SWIGLU) {
                                const float2 u = *reinterpret_cast<const float2 *>(rb + r * kTileK + 2 * kp);
                                a.x = silu(a.x) * u.x;
                                a.y = silu(a.y) * u.y;
                            }
                        }
                        v[i] = a;
                    }
                    named_bar(4, kXThreads);  // all raw values are in registers: overwrite in place
#pragma unroll
                    for (int i = 0; i < kRowsPer; ++i) {
                        const int r = kTransformWarps * i + rw;
                        if (r >= kRp) break;
                        const __nv_bfloat162 hi = __floats2bfloat162_rn(v[i].x, v[i].y);
                        const __nv_bfloat162 lo = __floats2bfloat162_rn(v[i].x - __low2float(hi), v[i].y - __high2float(hi));
                        const uint32_t off = (uint32_t)r * 128u + ((uint32_t)((kp >> 2) ^ (r & 7)) << 4) + (uint32_t)(kp & 3) * 4u;
                        *reinterpret_cast<__nv_bfloat162 *>(xa + off) = hi;
                        *reinterpret_cast<__nv_bfloat162 *>(xa + kRp * 128 + off) = lo;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&xrdy[s]);
                    if (++kc == g.kchunks) kc = 0;
                }
                cp_async_wait<0>();
            } else {
                // ---------------- consumers ----------------
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
                    if (!mbar_wait(&fullW[s], (it / S) & 1) || !mbar_wait(&xrdy[s], (it / S) & 1)) {
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
            }
        };

        if (p.trace && blockIdx.x == 0 && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            p.trace[0] = t;
        }
        // ---- phase program (the same structure gemm_desc() encodes) ----
        // `go` is uniform over the work threads (taken inside the grid barrier), so every named barrier
        // below is reached by all of them or by none.
        setup_phase(p);
        bool go = grid_sync(p, sh, epoch);
        if (go) {
            embed_phase(p);
            grid_zero(p.qkv, p.R, 3 * p.d, 3 * p.d);
            if (p.parallel) grid_zero(p.t_in, p.R, p.d_in, p.d_in);
            named_bar(2, kWorkThreads);  // the embedding rows are read back by the CTA that wrote them
            row_stats_phase(p, 0, red);
            go = grid_sync(p, sh, epoch);
        }
        for (int l = 0; l < p.n_layers && go; ++l) {
            run_gemm(4 * l + 0);                       // qkv
            if (p.parallel) run_gemm(4 * l + 1);       // MLP in (same input)
            if (!(go = grid_sync(p, sh, epoch))) break;
            attention_phase<MR>(p, l, attn_scratch, sh);
            if (!(go = grid_sync(p, sh, epoch))) break;
            if (p.parallel) {
                run_gemm(4 * l + 2);                   // out-proj -> x
                run_gemm(4 * l + 3);                   // MLP out  -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
            } else {
                run_gemm(4 * l + 1);                   // out-proj -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
                row_stats_phase(p, 2 * l + 1, red);
                grid_zero(p.t_in, p.R, p.d_in, p.d_in);
                if (!(go = grid_sync(p, sh, epoch))) break;
                run_gemm(4 * l + 2);                   // MLP in
                if (!(go = grid_sync(p, sh, epoch))) break;
                run_gemm(4 * l + 3);                   // MLP out -> x
                if (!(go = grid_sync(p, sh, epoch))) break;
            }
            row_stats_phase(p, 2 * (l + 1), red);
            if (l + 1 < p.n_layers) grid_zero(p.qkv, p.R, 3 * p.d, 3 * p.d);
            if (l + 1 < p.n_layers && p.parallel) grid_zero(p.t_in, p.R, p.d_in, p.d_in);
            if (l + 1 == p.n_layers && p.want_logits) grid_zero(p.logits, p.R, p.V, p.V);
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

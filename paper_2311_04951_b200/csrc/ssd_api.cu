// C ABI of the verification path (declared in include/ssd.h): argument checks, workspace
// carving and the launch sequences.  All arithmetic runs in the kernels of gemm.cuh,
// rowops.cuh, attention.cuh and tail.cuh; there is no CPU or library fallback.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/ssd.h"
#include "attention.cuh"
#include "common.cuh"
#include "gemm.cuh"
#include "persistent.cuh"
#include "rowops.cuh"
#include "tail.cuh"
#include "prefill.cuh"

using namespace ssd;

namespace {

std::atomic<uint64_t> g_launches{0};
int g_num_sms = 0;
int g_l2_window = 0;  // bytes of L2 that may hold persisting lines (0: the device has none / the limit could not be set)
bool g_attr_done = false;
std::mutex g_mu;

// ---- optional per-launch timing of the kernel that streams the weights (forward_kernel for bf16
//      models in single-kernel mode, otherwise every gemm launch) ----
bool g_persistent = true;  // bf16 models: whole forward in one cooperative kernel
int g_attn_mode = 0;       // 0: choose per pass; 1: warp-MMA attention items; 2: tensor-core items wherever they apply
bool g_trace = false;       // stamp the global timer after every grid barrier of the forward kernel
int g_top_k = 0;           // restriction of both models' distributions before sampling / verification (0: none)
float g_top_p = 1.0f;      // (1: none)
int g_prefill_mode = 0;    // 0: many-row prompt pass where it pays; 1: never; 2: wherever the model allows it
long long g_wait_cycles = 0;  // 0: the kernels' default bound (about two seconds) on every wait that takes work
bool g_prof = false;
std::vector<cudaEvent_t> g_prof_events;  // pairs
size_t g_prof_used = 0;

// start/stop events around a launch when profiling is on (0 = ok)
int prof_begin(cudaStream_t st, cudaEvent_t *stop) {
    *stop = nullptr;
    if (!g_prof) return 0;
    if (g_prof_used + 2 > g_prof_events.size()) {
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return -1;
            g_prof_events.push_back(e);
        }
    }
    cudaEvent_t e0 = g_prof_events[g_prof_used];
    *stop = g_prof_events[g_prof_used + 1];
    g_prof_used += 2;
    return cudaEventRecord(e0, st) == cudaSuccess ? 0 : -1;
}
int prof_end(cudaStream_t st, cudaEvent_t stop) {
    if (!stop) return 0;
    return cudaEventRecord(stop, st) == cudaSuccess ? 0 : -1;
}

#define CUDA_OK(expr)                        \
    do {                                     \
        cudaError_t e__ = (expr);            \
        if (e__ != cudaSuccess) return SSD_E_CUDA; \
    } while (0)

#define LAUNCH(kernel, grid, block, smem, stream, ...)                 \
    do {                                                                \
        kernel<<<grid, block, smem, stream>>>(__VA_ARGS__);             \
        g_launches.fetch_add(1, std::memory_order_relaxed);             \
        if (cudaPeekAtLastError() != cudaSuccess) return SSD_E_CUDA;    \
    } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 matrix [rows, cols] row-major -> tensor map with a (box_rows x 64) box, 128-byte swizzle
int make_map(CUtensorMap *map, const void *ptr, int rows, int cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_E_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_E_CUDA;
}

template <int NT>
constexpr int gemm_stage_bytes() { return kWTileBytes + 2 * NT * 8 * kTileK * 2; }
constexpr int kSmemBudget = 227 * 1024;

template <int NT>
int gemm_stages() {
    int s = (kSmemBudget - 1024 - 512) / gemm_stage_bytes<NT>();
    return s > 12 ? 12 : s;
}
template <int NT>
size_t gemm_smem() { return 1024 + (size_t)gemm_stages<NT>() * gemm_stage_bytes<NT>() + 16 * gemm_stages<NT>() + 16; }

template <typename K>
int set_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess ? 0 : -1;
}

template <typename T, int MR>
size_t attn_smem(int Dh) {
    return (size_t)MR * (Dh + kAttnTile + 3) * 4 + 2 * (size_t)kAttnTile * (Dh + 16 / sizeof(T)) * sizeof(T);
}

int init_device_once() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_attr_done) return SSD_OK;
    int dev = 0;
    CUDA_OK(cudaGetDevice(&dev));
    CUDA_OK(cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev));
    {   // room in L2 for persisting lines (a limit of this process's context, gone with it)
        int max_persist = 0, max_window = 0;
        cudaDeviceGetAttribute(&max_persist, cudaDevAttrMaxPersistingL2CacheSize, dev);
        cudaDeviceGetAttribute(&max_window, cudaDevAttrMaxAccessPolicyWindowSize, dev);
        size_t want = 32u << 20;
        if ((size_t)max_persist < want) want = (size_t)max_persist;
        if (want > 0 && cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) == cudaSuccess)
            g_l2_window = (int)(want < (size_t)max_window ? want : (size_t)max_window);
        (void)cudaGetLastError();
    }
    int rc = 0;
    rc |= set_smem(gemm_bf16_kernel<1>, gemm_smem<1>());
    rc |= set_smem(gemm_bf16_kernel<2>, gemm_smem<2>());
    rc |= set_smem(gemm_bf16_kernel<3>, gemm_smem<3>());
    rc |= set_smem(gemm_bf16_kernel<4>, gemm_smem<4>());
    rc |= set_smem(gemm_bf16_kernel<5>, gemm_smem<5>());
    rc |= set_smem(gemm_bf16_kernel<6>, gemm_smem<6>());
    rc |= set_smem(gemm_bf16_kernel<7>, gemm_smem<7>());
    rc |= set_smem(gemm_bf16_kernel<8>, gemm_smem<8>());
    rc |= set_smem(attn_partial_kernel<float, 8>, attn_smem<float, 8>(128));
    rc |= set_smem(attn_partial_kernel<float, 16>, attn_smem<float, 16>(128));
    rc |= set_smem(attn_partial_kernel<float, 32>, attn_smem<float, 32>(128));
    rc |= set_smem(attn_partial_kernel<__nv_bfloat16, 8>, attn_smem<__nv_bfloat16, 8>(128));
    rc |= set_smem(attn_partial_kernel<__nv_bfloat16, 16>, attn_smem<__nv_bfloat16, 16>(128));
    rc |= set_smem(attn_partial_kernel<__nv_bfloat16, 32>, attn_smem<__nv_bfloat16, 32>(128));
    rc |= set_smem(prefill_gemm_kernel, kPfSmem);
    rc |= set_smem(prefill_attn_kernel, prefill_attn_smem(128));
    rc |= set_smem(prefill_attn_tc_kernel, kPtSmem);
    if (rc) return SSD_E_CUDA;
    g_attr_done = true;
    return SSD_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------
struct ssd_model {
    ssd_arch a;
    std::vector<const void *> w;  // 2 + 12 L + 3 tensors
    std::vector<CUtensorMap> tm;  // bf16 models: per layer {qkv, o, in, out}, then lm head
    std::vector<CUtensorMap> tm256;  // the same four per layer with 256-row boxes (many-row prompt pass)
    int d_in;
    const ModelDesc *dev_desc;    // bf16 models: the same maps + vector pointers in device memory (caller-owned)
};

struct ssd_kv {
    ssd_arch a;
    int B, S;
    uint8_t *buf;
    int32_t *status, *len, *keep;
    uint8_t *cache;
    size_t layer_bytes, esize;
    CUtensorMap tm_rows;  // bf16 caches of head dim 128: every (layer, sequence, K|V, head, position) row, box 64 x 128
    bool tm_rows_ok;
    int len_ub;   // host-side upper bound of the committed lengths
    int last_rows;  // rows the last forward left uncommitted (upper bound bookkeeping)
    // The bound follows the device without a synchronisation: every kernel that changes the lengths writes
    // (operation number << 32 | largest length) into this word of mapped host memory; the host adds what the
    // operations queued behind that number can add at most (growth_at[n & 255] = total growth bound after op n).
    unsigned long long *mailbox, *mailbox_dev;
    unsigned op_seq;
    long long growth_total;
    long long growth_at[256];
};

namespace {

// A length-changing operation is about to be queued: it may add up to `growth` positions to a sequence.
unsigned kv_note_op(ssd_kv *kv, int growth) {
    ++kv->op_seq;
    kv->growth_total += growth;
    kv->growth_at[kv->op_seq & 255] = kv->growth_total;
    kv->len_ub += growth;
    if (kv->len_ub > kv->S) kv->len_ub = kv->S;
    return kv->op_seq;
}
// Upper bound of the committed lengths once everything queued so far has run.
int kv_bound(ssd_kv *kv) {
    if (kv->mailbox) {
        const unsigned long long v = *reinterpret_cast<volatile unsigned long long *>(kv->mailbox);
        const unsigned seq = (unsigned)(v >> 32);
        if (seq != 0 && kv->op_seq - seq < 256u) {
            const long long ub = (long long)(unsigned)(v & 0xffffffffu) + kv->growth_total - kv->growth_at[seq & 255];
            kv->len_ub = ub > kv->S ? kv->S : (int)ub;
        }
    }
    return kv->len_ub;
}

enum { T_TOK = 0, T_POS = 1, T_L0 = 2, PER_LAYER = 12 };
enum { L_LN1G, L_LN1B, L_WQKV, L_BQKV, L_WO, L_BO, L_LN2G, L_LN2B, L_WIN, L_BIN, L_WOUT, L_BOUT };

const void *lw(const ssd_model *m, int layer, int which) { return m->w[T_L0 + PER_LAYER * layer + which]; }
const void *fw(const ssd_model *m, int which) { return m->w[T_L0 + PER_LAYER * m->a.n_layers + which]; }
const void *lm_matrix(const ssd_model *m) { return m->a.tie_lm_head ? m->w[T_TOK] : fw(m, 2); }

int build_maps(ssd_model *m) {
    if (m->a.dtype != 1) return SSD_OK;
    const ssd_arch &a = m->a;
    m->tm.resize((size_t)4 * a.n_layers + 1);
    m->tm256.resize((size_t)4 * a.n_layers);
    for (int l = 0; l < a.n_layers; ++l) {
        int rc = 0;
        rc |= make_map(&m->tm256[4 * l + 0], lw(m, l, L_WQKV), 3 * a.d_model, a.d_model, kPfTileN);
        rc |= make_map(&m->tm256[4 * l + 1], lw(m, l, L_WO), a.d_model, a.d_model, kPfTileN);
        rc |= make_map(&m->tm256[4 * l + 2], lw(m, l, L_WIN), m->d_in, a.d_model, kPfTileN);
        rc |= make_map(&m->tm256[4 * l + 3], lw(m, l, L_WOUT), a.d_model, a.d_ff, kPfTileN);
        rc |= make_map(&m->tm[4 * l + 0], lw(m, l, L_WQKV), 3 * a.d_model, a.d_model, kTileN);
        rc |= make_map(&m->tm[4 * l + 1], lw(m, l, L_WO), a.d_model, a.d_model, kTileN);
        rc |= make_map(&m->tm[4 * l + 2], lw(m, l, L_WIN), m->d_in, a.d_model, kTileN);
        rc |= make_map(&m->tm[4 * l + 3], lw(m, l, L_WOUT), a.d_model, a.d_ff, kTileN);
        if (rc) return SSD_E_CUDA;
    }
    return make_map(&m->tm[(size_t)4 * a.n_layers], lm_matrix(m), a.vocab, a.d_model, kTileN);
}

int check_arch(const ssd_arch &a) {
    if (a.n_layers <= 0 || a.d_model <= 0 || a.n_heads <= 0 || a.head_dim <= 0 || a.d_ff <= 0 || a.vocab <= 0)
        return SSD_E_ARG;
    if (a.n_heads * a.head_dim != a.d_model) return SSD_E_SHAPE;
    if (a.head_dim > 128 || a.head_dim % 8) return SSD_E_SHAPE;
    if (a.norm < 0 || a.norm > 1 || a.act < 0 || a.act > 1 || a.pos < 0 || a.pos > 1 || a.dtype < 0 || a.dtype > 1)
        return SSD_E_ARG;
    if (a.pos == 1 && (a.rotary_dim <= 0 || a.rotary_dim % 2 || a.rotary_dim > a.head_dim)) return SSD_E_SHAPE;
    if (a.pos == 0 && a.max_pos <= 0) return SSD_E_ARG;
    if (a.dtype == 1) {
        if (a.d_model < 128 || a.d_model % 8 || a.d_ff < 128 || a.d_ff % 8 || a.vocab < 128) return SSD_E_SHAPE;
    }
    return SSD_OK;
}

// ---- workspace ----
struct Workspace {
    RowInfo ri;
    int32_t *n_rows_tmp;
    float *x, *qkv, *qrot, *t_in, *logits;
    RowStat *stats;
    RowFilter *filt;
    // in-kernel tail of a draft loop: per (sequence, CTA) partials and the draws' meeting places
    float *tp_m, *tp_s;
    int32_t *tp_a, *tail_hit;
    double *tp_mass;
    Operand xn1, xn2, ao, act;
    float *part_m, *part_l, *part_o;
    int max_split;
    // persistent kernel
    unsigned *sync;  // [0] grid barrier counter, [16..] attention tickets
    size_t sync_bytes;
    unsigned long long *trace;  // [kTraceSlots] phase time stamps (debug)
    int rows_k;      // rows the persistent kernel's tiles span (padded)
    size_t bytes;
};

constexpr int kMaxSplit = 32;
constexpr int kMaxCtas = 256;  // upper bound of the forward kernel's grid (one CTA per SM)

// A draft loop: n_steps forwards in one launch, each ended inside the kernel (q, draw, commit).
struct DraftLoop {
    int n_steps;
    float inv_t;
    const float *u;
    int u_stride;
    int32_t *tok_out;
    int tok_out_stride;
    float *q_out;
    size_t q_stride;
    unsigned mb_seq;
};
constexpr int kTraceSlots = 1024;

// Carve (or just size, base == nullptr) the workspace for B sequences x M rows.
Workspace carve(const ssd_model *m, int B, int M, uint8_t *base) {
    const ssd_arch &a = m->a;
    const int R = B * M, Rp = (R + 7) / 8 * 8, d = a.d_model, F = a.d_ff;
    const int Rk = Rp <= 40 ? Rp : 64;  // kernel instantiations exist for 8..40 and 64 rows
    size_t off = 0;
    auto take = [&](size_t bytes) -> uint8_t * {
        uint8_t *p = base ? base + off : nullptr;
        off += align_up(bytes, 1024);
        return p;
    };
    Workspace w;
    memset(&w, 0, sizeof(w));
    const int half = a.pos == 1 ? a.rotary_dim / 2 : 0;
    w.ri.seq = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.pos = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.valid = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.n_eff = (int32_t *)take(sizeof(int32_t) * B);
    w.ri.rope_cos = (float *)take(sizeof(float) * (size_t)R * (half ? half : 1));
    w.ri.rope_sin = (float *)take(sizeof(float) * (size_t)R * (half ? half : 1));
    w.n_rows_tmp = (int32_t *)take(sizeof(int32_t) * B);
    w.rows_k = Rk;
    w.x = (float *)take(sizeof(float) * (size_t)R * d);
    w.qkv = (float *)take(sizeof(float) * (size_t)R * 3 * d);
    w.qrot = (float *)take(sizeof(float) * (size_t)R * d);
    w.t_in = (float *)take(sizeof(float) * (size_t)R * m->d_in);
    w.sync_bytes = sizeof(unsigned) * (16 + (size_t)B * a.n_heads);
    w.sync = (unsigned *)take(w.sync_bytes);
    w.trace = (unsigned long long *)take(sizeof(unsigned long long) * kTraceSlots);
    w.logits = (float *)take(sizeof(float) * (size_t)R * a.vocab);
    w.stats = (RowStat *)take(sizeof(RowStat) * R);
    w.filt = (RowFilter *)take(sizeof(RowFilter) * R);
    w.tp_m = (float *)take(sizeof(float) * (size_t)B * kMaxCtas);
    w.tp_s = (float *)take(sizeof(float) * (size_t)B * kMaxCtas);
    w.tp_a = (int32_t *)take(sizeof(int32_t) * (size_t)B * kMaxCtas);
    w.tp_mass = (double *)take(sizeof(double) * (size_t)B * kMaxCtas);
    w.tail_hit = (int32_t *)take(sizeof(int32_t) * (size_t)kMaxRowsPerSeq * B * 2);
    // GEMM operands: hi rows [0, rows) then lo rows [rows, 2 rows) in one buffer; the stepwise path
    // pads rows to Rp, the single-kernel path to Rk (one allocation of 2 * Rk rows serves both)
    auto operand = [&](int ld, bool needed) {
        Operand o;
        o.f32 = nullptr; o.hi = nullptr; o.lo = nullptr; o.ld = ld;
        if (!needed) return o;
        if (a.dtype == 0) {
            o.f32 = (float *)take(sizeof(float) * (size_t)Rp * ld);
        } else {
            o.hi = (__nv_bfloat16 *)take(2 * (size_t)2 * Rk * align_up((size_t)ld, 64));  // whole 64-wide k tiles
            o.lo = o.hi + (size_t)Rk * ld;
        }
        return o;
    };
    w.xn1 = operand(d, true);
    w.xn2 = operand(d, a.parallel_residual != 0);
    w.ao = operand(d, true);
    w.act = operand(F, true);
    w.max_split = kMaxSplit;
    size_t slots = (size_t)R * a.n_heads * kMaxSplit;
    w.part_m = (float *)take(sizeof(float) * slots);
    w.part_l = (float *)take(sizeof(float) * slots);
    w.part_o = (float *)take(sizeof(float) * slots * a.head_dim);
    w.bytes = off;
    return w;
}

struct GemmCall {
    const ssd_model *m;
    cudaStream_t st;
    int R, Rp;
};

template <int NT>
int launch_gemm_nt(cudaStream_t st, const CUtensorMap &tw, const CUtensorMap &th, const CUtensorMap &tl, GemmArgs g,
                   int grid) {
    g.stages = gemm_stages<NT>();
    LAUNCH(gemm_bf16_kernel<NT>, grid, kGemmThreads, gemm_smem<NT>(), st, tw, th, tl, g);
    return SSD_OK;
}

// out[R, ldo] += X[R, Kd] * W[N, Kd]^T
int gemm(const GemmCall &c, const void *W, const CUtensorMap *tw, const Operand &X, int Kd, int N, float *out, int ldo,
         int32_t *status) {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (g_prof) {
        if (g_prof_used + 2 > g_prof_events.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                CUDA_OK(cudaEventCreate(&e));
                g_prof_events.push_back(e);
            }
        }
        e0 = g_prof_events[g_prof_used];
        e1 = g_prof_events[g_prof_used + 1];
        g_prof_used += 2;
        CUDA_OK(cudaEventRecord(e0, c.st));
    }
    int rc = SSD_OK;
    if (c.m->a.dtype == 0) {
        const int warps = 8;
        LAUNCH(gemm_f32_kernel, ceil_div(N, warps), warps * 32, 0, c.st, (const float *)W, X.f32, X.ld, out, ldo, N,
               Kd, c.R);
    } else {
        CUtensorMap th, tl;
        if (make_map(&th, X.hi, c.Rp, Kd, c.Rp) || make_map(&tl, X.lo, c.Rp, Kd, c.Rp)) return SSD_E_CUDA;
        GemmArgs g;
        g.out = out; g.ldo = ldo; g.N = N; g.Kd = Kd; g.R = c.R;
        g.n_tiles = ceil_div(N, kTileN);
        g.kchunks = ceil_div(Kd, kTileK);
        g.stages = 0;
        g.status = status;
        long long total = (long long)g.n_tiles * g.kchunks;
        int grid = (int)(total < g_num_sms ? total : g_num_sms);
        switch (c.Rp / 8) {
            case 1: rc = launch_gemm_nt<1>(c.st, *tw, th, tl, g, grid); break;
            case 2: rc = launch_gemm_nt<2>(c.st, *tw, th, tl, g, grid); break;
            case 3: rc = launch_gemm_nt<3>(c.st, *tw, th, tl, g, grid); break;
            case 4: rc = launch_gemm_nt<4>(c.st, *tw, th, tl, g, grid); break;
            case 5: rc = launch_gemm_nt<5>(c.st, *tw, th, tl, g, grid); break;
            case 6: rc = launch_gemm_nt<6>(c.st, *tw, th, tl, g, grid); break;
            case 7: rc = launch_gemm_nt<7>(c.st, *tw, th, tl, g, grid); break;
            case 8: rc = launch_gemm_nt<8>(c.st, *tw, th, tl, g, grid); break;
            default: return SSD_E_CAPACITY;
        }
    }
    if (rc) return rc;
    if (e1) CUDA_OK(cudaEventRecord(e1, c.st));
    return SSD_OK;
}

// Split of the position axis for a context of up to `ctx` positions, `groups` = independent
// (sequence, head, row-tile) streams.  Every item pays a few microseconds of fixed latency, so the
// aim is one round of items over the SMs: as many splits as keep groups * splits <= #SMs.
void plan_split(int groups, int ctx, int *chunk, int *n_split, int tile = kAttnTile) {
    if (ctx < 1) ctx = 1;
    const int sms = g_num_sms > 0 ? g_num_sms : 148;
    int ns = ctx <= 256 ? 1 : sms / (groups > 0 ? groups : 1);
    int max_by_len = ceil_div(ctx, 2 * kAttnTile);  // at least 128 positions per split
    if (ns > max_by_len) ns = max_by_len;
    if (ns > kMaxSplit) ns = kMaxSplit;
    if (ns < 1) ns = 1;
    int ch = ceil_div(ceil_div(ctx, ns), tile) * tile;
    *chunk = ch;
    *n_split = ceil_div(ctx, ch);
}

template <typename T>
int launch_attn(cudaStream_t st, const AttnArgs &a, int B, int M) {
    dim3 grid(a.n_split, B * a.H);
    auto k8 = attn_partial_kernel<T, 8>;
    auto k16 = attn_partial_kernel<T, 16>;
    auto k32 = attn_partial_kernel<T, 32>;
    if (M <= 8) {
        LAUNCH(k8, grid, kAttnThreads, (attn_smem<T, 8>(a.Dh)), st, a);
    } else if (M <= 16) {
        LAUNCH(k16, grid, kAttnThreads, (attn_smem<T, 16>(a.Dh)), st, a);
    } else {
        LAUNCH(k32, grid, kAttnThreads, (attn_smem<T, 32>(a.Dh)), st, a);
    }
    return SSD_OK;
}

int run_setup(const ssd_model *m, ssd_kv *kv, int M, const int32_t *n_rows, const Workspace &w, cudaStream_t st) {
    SetupArgs s;
    s.B = kv->B; s.M = M; s.n_rows = n_rows; s.len = kv->len; s.s_max = kv->S;
    s.pos_limit = m->a.pos == 0 ? m->a.max_pos : 0;
    s.rotary_dim = m->a.pos == 1 ? m->a.rotary_dim : 0;
    s.rotary_base = m->a.rotary_base;
    s.ri = w.ri;
    s.status = kv->status;
    LAUNCH(setup_rows_kernel, kv->B * M, 64, 0, st, s);
    return SSD_OK;
}

int run_attention(const ssd_model *m, ssd_kv *kv, int layer, const float *q, int M, const Workspace &w,
                  const CombineArgs &comb_in, cudaStream_t st) {
    const ssd_arch &a = m->a;
    AttnArgs at;
    at.q = q;
    at.cache = kv->cache + (size_t)layer * kv->layer_bytes;
    at.len = kv->len;
    at.M = M; at.H = a.n_heads; at.Dh = a.head_dim; at.S = kv->S; at.d = a.d_model;
    int ctx = kv_bound(kv) + M;
    if (ctx > kv->S) ctx = kv->S;
    plan_split(kv->B * a.n_heads, ctx, &at.chunk, &at.n_split);
    at.scale = 1.0f / sqrtf((float)a.head_dim);
    at.ri = w.ri;
    at.part_m = w.part_m; at.part_l = w.part_l; at.part_o = w.part_o;
    int rc = a.dtype ? launch_attn<__nv_bfloat16>(st, at, kv->B, M) : launch_attn<float>(st, at, kv->B, M);
    if (rc) return rc;
    CombineArgs cb = comb_in;
    cb.part_m = w.part_m; cb.part_l = w.part_l; cb.part_o = w.part_o;
    cb.H = a.n_heads; cb.Dh = a.head_dim; cb.n_split = at.n_split; cb.d = a.d_model;
    LAUNCH(attn_combine_kernel, dim3(a.n_heads, kv->B * M), 128, 0, st, cb);
    return SSD_OK;
}

inline int barriers_needed(const ssd_arch &a) { return (a.parallel_residual ? 5 : 8) * a.n_layers; }  // upper bound

template <int NT>
int launch_forward_nt(FwdParams p, const void *ws_base, size_t ws_bytes, cudaStream_t st) {
    constexpr size_t stage = kWTileBytesP + 2 * NT * 8 * kTileK * 2;
    size_t attn = align_up(attn_scratch_bytes(p.Dh), 128);
    if (p.attn_tc == 1 && attn < (size_t)kTcScratchBytes) attn = kTcScratchBytes;
    if (p.attn_tc == 2) attn = m8_scratch_bytes(p.Dh);
    const size_t tail = 24 * 32 + 64 + 16 + sizeof(Shared) + 16 * sizeof(double) + kEpiBytes + 256;  // barriers, small state, epilogue tile
    const size_t total = (size_t)kSmemBudget - 1024 - tail;
    // upper slots share their bytes with the attention scratch; two slots never do where they fit
    // (one with the 48 KB stages of 64 rows, which only the prompt pass uses)
    size_t S2 = (attn + stage - 1) / stage;
    size_t region2 = S2 * stage;
    if (region2 + 2 * stage > total) {
        S2 = attn / stage;
        region2 = attn;
    }
    if (region2 + stage > total) return SSD_E_CAPACITY;
    size_t S1 = (total - region2) / stage;
    if (S1 + S2 > 32) S1 = 32 - S2;  // one parity bit per slot
    p.stages = (int)(S1 + S2);
    p.stages_lo = (int)S1;
    p.attn_smem_off = (int)(S1 * stage);
    p.bar_off = (int)align_up(S1 * stage + region2, 128);
    const size_t smem = 1024 + (size_t)p.bar_off + tail;
    static bool attr[64] = {false};  // the attribute belongs to the device's copy of the kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SSD_E_CUDA;
    if (!attr[dev]) {
        if (cudaFuncSetAttribute(forward_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) !=
            cudaSuccess)
            return SSD_E_CUDA;
        attr[dev] = true;
    }
    void *args[] = {&p};
    // The workspace (residual stream, GEMM outputs and operands: a few MB that every phase re-reads and that the
    // GEMMs reduce into) is marked persisting in L2 for this launch, so that the weight stream does not push it
    // out between the phase that writes a buffer and the phase that reads it.
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(g_num_sms);
    cfg.blockDim = dim3(kPersistThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    int na = 0;
    attrs[na].id = cudaLaunchAttributeCooperative;
    attrs[na].val.cooperative = 1;
    ++na;
    if (g_l2_window > 0 && ws_base && ws_bytes > 0) {
        attrs[na].id = cudaLaunchAttributeAccessPolicyWindow;
        attrs[na].val.accessPolicyWindow.base_ptr = const_cast<void *>(ws_base);
        attrs[na].val.accessPolicyWindow.num_bytes = ws_bytes < (size_t)g_l2_window ? ws_bytes : (size_t)g_l2_window;
        attrs[na].val.accessPolicyWindow.hitRatio = 1.0f;
        attrs[na].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        attrs[na].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    if (cudaLaunchKernelExC(&cfg, (const void *)forward_kernel<NT>, args) != cudaSuccess) return SSD_E_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return SSD_OK;
}

int launch_forward_rows(const FwdParams &p, int rows_k, const void *ws_base, size_t ws_bytes, cudaStream_t st) {
    switch (rows_k / 8) {
        case 1: return launch_forward_nt<1>(p, ws_base, ws_bytes, st);
        case 2: return launch_forward_nt<2>(p, ws_base, ws_bytes, st);
        case 3: return launch_forward_nt<3>(p, ws_base, ws_bytes, st);
        case 4: return launch_forward_nt<4>(p, ws_base, ws_bytes, st);
        case 5: return launch_forward_nt<5>(p, ws_base, ws_bytes, st);
        case 8: return launch_forward_nt<8>(p, ws_base, ws_bytes, st);
        default: break;
    }
    return SSD_E_CAPACITY;
}

// The whole forward as one cooperative launch (bf16 models).
int forward_persistent(ssd_model *m, ssd_kv *kv, const int32_t *tokens, int tok_stride, int M, const int32_t *n_rows,
                       bool want_logits, const Workspace &w, cudaStream_t st, const DraftLoop *dl = nullptr) {
    const ssd_arch &a = m->a;
    FwdParams p;
    memset(&p, 0, sizeof(p));
    const int R = kv->B * M, Rk = w.rows_k;
    const Operand *ops[4] = {&w.xn1, &w.xn2, &w.ao, &w.act};
    for (int i = 0; i < 4; ++i) {
        p.op[i] = ops[i]->hi;
        p.op_ld[i] = ops[i]->ld;
    }
    p.rk = Rk;
    p.md = m->dev_desc;
    p.n_layers = a.n_layers; p.d = a.d_model; p.H = a.n_heads; p.Dh = a.head_dim; p.F = a.d_ff; p.d_in = m->d_in;
    p.V = a.vocab; p.norm_kind = a.norm; p.swiglu = a.act == 1; p.parallel = a.parallel_residual;
    p.rotary_dim = a.pos == 1 ? a.rotary_dim : 0; p.learned_pos = a.pos == 0; p.is_bf16_emb = 1;
    p.inv_d = 1.0 / (double)a.d_model;
    p.eps = a.norm_eps; p.rotary_base = a.rotary_base; p.attn_scale = 1.0f / sqrtf((float)a.head_dim);
    p.B = kv->B; p.M = M; p.R = R;
    p.tokens = tokens; p.tok_stride = tok_stride; p.n_rows = n_rows;
    p.tok_emb = m->w[T_TOK]; p.pos_emb = m->w[T_POS];
    p.pos_limit = a.pos == 0 ? a.max_pos : 0;
    p.cache = kv->cache; p.layer_bytes = kv->layer_bytes; p.len = kv->len; p.S = kv->S; p.status = kv->status;
    p.ri = w.ri;
    p.x = w.x; p.qkv = w.qkv; p.t_in = w.t_in; p.logits = w.logits;
    p.part_m = w.part_m; p.part_l = w.part_l; p.part_o = w.part_o;
    p.gbar = w.sync; p.tickets = w.sync + 16;
    int ctx = kv_bound(kv) + M;
    if (ctx > kv->S) ctx = kv->S;
    // Tensor-core attention items stream 128 positions per ~2 us but cost ~8 us more to start than the
    // warp-MMA items (64 positions per ~2 us): they pay off from about a thousand positions per split.
    const int groups = kv->B * a.n_heads * ((M + 15) / 16);
    p.attn_tc = 0;
    p.kv_rows_per_layer = kv->B * 2 * a.n_heads * kv->S;
    // Passes of at most eight rows per sequence (draft steps, decode steps, verification with K <= 7): the warp-MMA
    // items that carry hi and lo in one tile.
    const bool packed_form = M <= kM8Rows && (a.head_dim == 64 || a.head_dim == 128) && (g_attn_mode == 0 || g_attn_mode == 3);
    if (packed_form) {
        plan_split(groups, ctx, &p.chunk, &p.n_split, kAttnTile);
        p.attn_tc = 2;
    } else if (a.head_dim == 128 && kv->tm_rows_ok && g_attn_mode != 1 && g_attn_mode != 3) {
        plan_split(groups, ctx, &p.chunk, &p.n_split, kTcChunk);
        if (p.chunk >= 1024 || g_attn_mode == 2) {
            p.attn_tc = 1;
            p.tm_kv = kv->tm_rows;
        }
    }
    if (!p.attn_tc) plan_split(groups, ctx, &p.chunk, &p.n_split, kAttnTile);
    {
        const int items = groups * p.n_split, sms = g_num_sms > 0 ? g_num_sms : 148;
        p.attn_ctas = items < sms ? items : sms;
        p.overlap_out = (a.parallel_residual && 2 * p.attn_ctas <= sms) ? 1 : 0;
    }
    p.want_logits = want_logits ? 1 : 0;
    p.wait_cycles = g_wait_cycles;
    p.n_steps = 1;
    if (dl) {
        if (g_num_sms > kMaxCtas) return SSD_E_CAPACITY;
        p.n_steps = dl->n_steps; p.tail = 1; p.inv_t = dl->inv_t;
        p.u = dl->u; p.u_stride = dl->u_stride;
        p.tok_out = dl->tok_out; p.tok_out_stride = dl->tok_out_stride;
        p.q_out = dl->q_out; p.q_stride = dl->q_stride;
        p.len_rw = kv->len;
        p.tp_m = w.tp_m; p.tp_s = w.tp_s; p.tp_a = w.tp_a; p.tp_mass = w.tp_mass; p.tail_hit = w.tail_hit;
        p.mailbox = kv->mailbox_dev; p.mb_seq = dl->mb_seq;
    }
    p.trace = (g_trace && 2 + p.n_steps * (barriers_needed(a) + 6) + 3 < kTraceSlots) ? w.trace : nullptr;
    CUDA_OK(cudaMemsetAsync(w.sync, 0, w.sync_bytes, st));
    cudaEvent_t prof_stop;
    if (prof_begin(st, &prof_stop)) return SSD_E_CUDA;
    int rc = launch_forward_rows(p, Rk, w.ri.seq, w.bytes, st);
    if (!rc && prof_end(st, prof_stop)) return SSD_E_CUDA;
    if (rc) return rc;
    kv->last_rows = M;
    return SSD_OK;
}

// One decoder forward over B x M rows against the cache.  Appends (does not commit) the rows'
// keys/values; leaves logits in w.logits when want_logits.
bool single_kernel_path(const ssd_model *m) {
    const ssd_arch &a = m->a;
    return a.dtype == 1 && g_persistent && m->dev_desc && a.head_dim % 16 == 0 &&
           (a.pos == 0 || a.rotary_dim % 16 == 0);  // the MMA attention tiles heads by 16 and rotary halves by 8
}

int forward(ssd_model *m, ssd_kv *kv, const int32_t *tokens, int tok_stride, int M, const int32_t *n_rows,
            bool want_logits, const Workspace &w, cudaStream_t st) {
    const ssd_arch &a = m->a;
    if (single_kernel_path(m)) return forward_persistent(m, kv, tokens, tok_stride, M, n_rows, want_logits, w, st);
    const int B = kv->B, R = B * M, d = a.d_model, F = a.d_ff;
    GemmCall gc{m, st, R, (R + 7) / 8 * 8};
    int rc = run_setup(m, kv, M, n_rows, w, st);
    if (rc) return rc;
    if (a.dtype) {
        LAUNCH(embed_kernel<__nv_bfloat16>, R, 256, 0, st, (const __nv_bfloat16 *)m->w[T_TOK],
               (const __nv_bfloat16 *)m->w[T_POS], tokens, tok_stride, M, a.vocab, d, w.ri, w.x);
    } else {
        LAUNCH(embed_kernel<float>, R, 256, 0, st, (const float *)m->w[T_TOK], (const float *)m->w[T_POS], tokens,
               tok_stride, M, a.vocab, d, w.ri, w.x);
    }
    auto norm_args = [&](const float *g1, const float *b1, Operand o1) {
        NormArgs n;
        memset(&n, 0, sizeof(n));
        n.x = w.x; n.d = d; n.kind = a.norm; n.eps = a.norm_eps;
        n.n_norms = 1; n.g[0] = g1; n.b[0] = b1; n.out[0] = o1;
        return n;
    };
    for (int l = 0; l < a.n_layers; ++l) {
        const CUtensorMap *tm = a.dtype ? &m->tm[4 * l] : nullptr;
        const float *b_qkv = (const float *)lw(m, l, L_BQKV), *b_o = (const float *)lw(m, l, L_BO);
        const float *b_in = (const float *)lw(m, l, L_BIN), *b_out = (const float *)lw(m, l, L_BOUT);
        // ---- norm(s) + pre-load of the GEMM outputs ----
        NormArgs n1 = norm_args((const float *)lw(m, l, L_LN1G), (const float *)lw(m, l, L_LN1B), w.xn1);
        n1.init[n1.n_init++] = InitJob{w.qkv, b_qkv, 3 * d, 3 * d};
        if (a.parallel_residual) {
            n1.n_norms = 2;
            n1.g[1] = (const float *)lw(m, l, L_LN2G);
            n1.b[1] = (const float *)lw(m, l, L_LN2B);
            n1.out[1] = w.xn2;
            n1.init[n1.n_init++] = InitJob{w.t_in, b_in, m->d_in, m->d_in};
        }
        LAUNCH(norm_kernel, R, 256, 0, st, n1);
        if ((rc = gemm(gc, lw(m, l, L_WQKV), tm ? tm + 0 : nullptr, w.xn1, d, 3 * d, w.qkv, 3 * d, kv->status))) return rc;
        if (a.parallel_residual)
            if ((rc = gemm(gc, lw(m, l, L_WIN), tm ? tm + 2 : nullptr, w.xn2, d, m->d_in, w.t_in, m->d_in, kv->status)))
                return rc;
        // ---- rotary + append, attention ----
        RopeArgs ra;
        ra.qkv = w.qkv; ra.q_out = w.qrot;
        ra.cache = kv->cache + (size_t)l * kv->layer_bytes;
        ra.d = d; ra.H = a.n_heads; ra.Dh = a.head_dim; ra.S = kv->S;
        ra.rotary_dim = a.pos == 1 ? a.rotary_dim : 0;
        ra.ri = w.ri;
        if (a.dtype) {
            LAUNCH(rope_append_kernel<__nv_bfloat16>, R, 256, 0, st, ra);
        } else {
            LAUNCH(rope_append_kernel<float>, R, 256, 0, st, ra);
        }
        CombineArgs cb;
        memset(&cb, 0, sizeof(cb));
        cb.out = w.ao;
        cb.x = w.x;
        cb.bias.b0 = b_o;
        cb.bias.b1 = a.parallel_residual ? b_out : nullptr;
        if ((rc = run_attention(m, kv, l, w.qrot, M, w, cb, st))) return rc;
        BiasJob no_bias{nullptr, nullptr};
        if (a.parallel_residual) {
            LAUNCH(act_kernel, dim3(ceil_div(F, 256), R), 256, 0, st, w.t_in, m->d_in, F, a.act == 1, w.act, w.x, d,
                   no_bias);
            if ((rc = gemm(gc, lw(m, l, L_WO), tm ? tm + 1 : nullptr, w.ao, d, d, w.x, d, kv->status))) return rc;
            if ((rc = gemm(gc, lw(m, l, L_WOUT), tm ? tm + 3 : nullptr, w.act, F, d, w.x, d, kv->status))) return rc;
        } else {
            if ((rc = gemm(gc, lw(m, l, L_WO), tm ? tm + 1 : nullptr, w.ao, d, d, w.x, d, kv->status))) return rc;
            NormArgs n2 = norm_args((const float *)lw(m, l, L_LN2G), (const float *)lw(m, l, L_LN2B), w.xn1);
            n2.init[n2.n_init++] = InitJob{w.t_in, b_in, m->d_in, m->d_in};
            LAUNCH(norm_kernel, R, 256, 0, st, n2);
            if ((rc = gemm(gc, lw(m, l, L_WIN), tm ? tm + 2 : nullptr, w.xn1, d, m->d_in, w.t_in, m->d_in, kv->status)))
                return rc;
            BiasJob bj{b_out, nullptr};
            LAUNCH(act_kernel, dim3(ceil_div(F, 256), R), 256, 0, st, w.t_in, m->d_in, F, a.act == 1, w.act, w.x, d, bj);
            if ((rc = gemm(gc, lw(m, l, L_WOUT), tm ? tm + 3 : nullptr, w.act, F, d, w.x, d, kv->status))) return rc;
        }
    }
    if (want_logits) {
        NormArgs nf = norm_args((const float *)fw(m, 0), (const float *)fw(m, 1), w.xn1);
        nf.init[nf.n_init++] = InitJob{w.logits, nullptr, a.vocab, a.vocab};
        LAUNCH(norm_kernel, R, 256, 0, st, nf);
        if ((rc = gemm(gc, lm_matrix(m), a.dtype ? &m->tm[(size_t)4 * a.n_layers] : nullptr, w.xn1, d, a.vocab, w.logits,
                       a.vocab, kv->status)))
            return rc;
    }
    kv->last_rows = M;
    return SSD_OK;
}


// ---- prompt pass over many rows (bf16 models) --------------------------------------------------
constexpr int kWideMaxRows = 8192;  // rows of one many-row pass (sequences x rows per sequence)
constexpr int kWideMinRows = 256;   // below this the few-row kernel's passes are as fast

struct WideWs {
    RowInfo ri;
    int32_t *n_rows_tmp;
    float *x, *qkv, *qrot, *t_in;
    Operand xn1, xn2, ao, act;
    int rows_pad;
    size_t bytes;
};

WideWs carve_wide(const ssd_model *m, int B, int C, uint8_t *base) {
    const ssd_arch &a = m->a;
    const size_t R = (size_t)B * C, Rp = align_up(R, kPfTileM), d = a.d_model, F = a.d_ff;
    size_t off = 0;
    auto take = [&](size_t bytes) -> uint8_t * {
        uint8_t *p = base ? base + off : nullptr;
        off += align_up(bytes, 1024);
        return p;
    };
    WideWs w;
    memset(&w, 0, sizeof(w));
    const size_t half = a.pos == 1 ? a.rotary_dim / 2 : 0;
    w.ri.seq = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.pos = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.valid = (int32_t *)take(sizeof(int32_t) * R);
    w.ri.n_eff = (int32_t *)take(sizeof(int32_t) * B);
    w.ri.rope_cos = (float *)take(sizeof(float) * R * (half ? half : 1));
    w.ri.rope_sin = (float *)take(sizeof(float) * R * (half ? half : 1));
    w.n_rows_tmp = (int32_t *)take(sizeof(int32_t) * B);
    w.x = (float *)take(sizeof(float) * R * d);
    w.qkv = (float *)take(sizeof(float) * R * 3 * d);
    w.qrot = (float *)take(sizeof(float) * R * d);
    w.t_in = (float *)take(sizeof(float) * R * m->d_in);
    auto operand = [&](size_t ld, bool needed) {  // rows padded to whole 128-row tiles; hi and lo apart
        Operand o;
        o.f32 = nullptr; o.hi = nullptr; o.lo = nullptr; o.ld = (int)ld;
        if (!needed) return o;
        o.hi = (__nv_bfloat16 *)take(2 * Rp * ld);
        o.lo = (__nv_bfloat16 *)take(2 * Rp * ld);
        return o;
    };
    w.xn1 = operand(d, true);
    w.xn2 = operand(d, a.parallel_residual != 0);
    w.ao = operand(d, true);
    w.act = operand(F, true);
    w.rows_pad = (int)Rp;
    w.bytes = off;
    return w;
}

bool wide_path_ok(const ssd_model *m) {
    const ssd_arch &a = m->a;
    return a.dtype == 1 && g_prefill_mode != 1 && a.head_dim % 16 == 0 && a.d_model % 8 == 0 && a.d_ff % 8 == 0 && m->d_in % 4 == 0 &&
           !m->tm256.empty();
}

// out[R, ldo] (+)= X[R, Kd] W[N, Kd]^T + bias over 128 x 256 output tiles
int gemm_wide(cudaStream_t st, const CUtensorMap *tw, const Operand &X, int rows_pad, int R, int Kd, int N, float *out,
              int ldo, const float *bias, bool accumulate, int32_t *status) {
    CUtensorMap th, tl;
    if (make_map(&th, X.hi, rows_pad, Kd, kPfTileM) || make_map(&tl, X.lo, rows_pad, Kd, kPfTileM)) return SSD_E_CUDA;
    PfGemmArgs g;
    g.out = out; g.bias = bias; g.accumulate = accumulate ? 1 : 0;
    g.ldo = ldo; g.N = N; g.Kd = Kd; g.R = R; g.status = status;
    g.wait_cycles = g_wait_cycles > 0 ? g_wait_cycles : kWaitCycles;
    const int n_tiles = ceil_div(N, kPfTileN) * ceil_div(R, kPfTileM), sms = g_num_sms > 0 ? g_num_sms : 148;
    LAUNCH(prefill_gemm_kernel, n_tiles < sms ? n_tiles : sms, kPfThreads, kPfSmem, st, *tw, th, tl, g);
    return SSD_OK;
}

// One decoder forward over B x C prompt rows: fills the cache (no logits).  The steps of the stepwise forward with
// many-row kernels: the projections write (q, k, v and the MLP input) or add to (the residual stream) their output
// together with the bias, so nothing is pre-loaded.
int forward_wide(ssd_model *m, ssd_kv *kv, const int32_t *tokens, int tok_stride, int C, const int32_t *n_rows,
                 const WideWs &w, cudaStream_t st) {
    const ssd_arch &a = m->a;
    const int B = kv->B, R = B * C, d = a.d_model, F = a.d_ff, Rp = w.rows_pad;
    SetupArgs s;
    s.B = B; s.M = C; s.n_rows = n_rows; s.len = kv->len; s.s_max = kv->S;
    s.pos_limit = a.pos == 0 ? a.max_pos : 0;
    s.rotary_dim = a.pos == 1 ? a.rotary_dim : 0;
    s.rotary_base = a.rotary_base;
    s.ri = w.ri;
    s.status = kv->status;
    LAUNCH(setup_rows_kernel, R, 64, 0, st, s);
    LAUNCH(embed_kernel<__nv_bfloat16>, R, 256, 0, st, (const __nv_bfloat16 *)m->w[T_TOK],
           (const __nv_bfloat16 *)m->w[T_POS], tokens, tok_stride, C, a.vocab, d, w.ri, w.x);
    auto norm_args = [&](const float *g1, const float *b1, const Operand &o1) {
        PfNormArgs n;
        memset(&n, 0, sizeof(n));
        n.x = w.x; n.d = d; n.kind = a.norm; n.eps = a.norm_eps;
        n.n_norms = 1; n.g[0] = g1; n.b[0] = b1; n.hi[0] = o1.hi; n.lo[0] = o1.lo;
        return n;
    };
    int rc;
    for (int l = 0; l < a.n_layers; ++l) {
        const CUtensorMap *tm = &m->tm256[4 * l];
        const float *b_qkv = (const float *)lw(m, l, L_BQKV), *b_o = (const float *)lw(m, l, L_BO);
        const float *b_in = (const float *)lw(m, l, L_BIN), *b_out = (const float *)lw(m, l, L_BOUT);
        PfNormArgs n1 = norm_args((const float *)lw(m, l, L_LN1G), (const float *)lw(m, l, L_LN1B), w.xn1);
        if (a.parallel_residual) {
            n1.n_norms = 2;
            n1.g[1] = (const float *)lw(m, l, L_LN2G);
            n1.b[1] = (const float *)lw(m, l, L_LN2B);
            n1.hi[1] = w.xn2.hi; n1.lo[1] = w.xn2.lo;
        }
        LAUNCH(prefill_norm_kernel, R, 256, 0, st, n1);
        if ((rc = gemm_wide(st, tm + 0, w.xn1, Rp, R, d, 3 * d, w.qkv, 3 * d, b_qkv, false, kv->status))) return rc;
        if (a.parallel_residual)
            if ((rc = gemm_wide(st, tm + 2, w.xn2, Rp, R, d, m->d_in, w.t_in, m->d_in, b_in, false, kv->status))) return rc;
        RopeArgs ra;
        ra.qkv = w.qkv; ra.q_out = w.qrot;
        ra.cache = kv->cache + (size_t)l * kv->layer_bytes;
        ra.d = d; ra.H = a.n_heads; ra.Dh = a.head_dim; ra.S = kv->S;
        ra.rotary_dim = a.pos == 1 ? a.rotary_dim : 0;
        ra.ri = w.ri;
        LAUNCH(rope_append_kernel<__nv_bfloat16>, R, 256, 0, st, ra);
        PfAttnArgs at;
        at.q = w.qrot;
        at.cache = (const __nv_bfloat16 *)(kv->cache + (size_t)l * kv->layer_bytes);
        at.len = kv->len; at.n_eff = w.ri.n_eff;
        at.out_hi = w.ao.hi; at.out_lo = w.ao.lo;
        at.M = C; at.H = a.n_heads; at.Dh = a.head_dim; at.S = kv->S; at.d = d;
        at.scale = 1.0f / sqrtf((float)a.head_dim);
        if (a.head_dim == 128 && kv->tm_rows_ok && g_prefill_mode != 3) {  // tensor-core form
            PtAttnArgs pt;
            pt.q = w.qrot; pt.len = kv->len; pt.n_eff = w.ri.n_eff;
            pt.out_hi = w.ao.hi; pt.out_lo = w.ao.lo;
            pt.M = C; pt.H = a.n_heads; pt.S = kv->S; pt.d = d;
            pt.kv_row0 = l * (kv->B * 2 * a.n_heads * kv->S);
            pt.scale = at.scale;
            pt.wait_cycles = g_wait_cycles > 0 ? g_wait_cycles : kWaitCycles;
            pt.status = kv->status;
            LAUNCH(prefill_attn_tc_kernel, dim3(ceil_div(C, kPtRows), a.n_heads, B), kPtThreads, kPtSmem, st, kv->tm_rows, pt);
        } else {
            LAUNCH(prefill_attn_kernel, dim3(ceil_div(C, kPaRows), a.n_heads, B), kPaThreads, prefill_attn_smem(a.head_dim), st,
                   at);
        }
        if ((rc = gemm_wide(st, tm + 1, w.ao, Rp, R, d, d, w.x, d, b_o, true, kv->status))) return rc;
        if (!a.parallel_residual) {
            PfNormArgs n2 = norm_args((const float *)lw(m, l, L_LN2G), (const float *)lw(m, l, L_LN2B), w.xn1);
            LAUNCH(prefill_norm_kernel, R, 256, 0, st, n2);
            if ((rc = gemm_wide(st, tm + 2, w.xn1, Rp, R, d, m->d_in, w.t_in, m->d_in, b_in, false, kv->status))) return rc;
        }
        LAUNCH(prefill_act_kernel, dim3(ceil_div(F, 1024), R), 256, 0, st, w.t_in, m->d_in, F, a.act == 1, w.act.hi, w.act.lo);
        if ((rc = gemm_wide(st, tm + 3, w.act, Rp, R, F, d, w.x, d, b_out, true, kv->status))) return rc;
    }
    kv->last_rows = C;
    return SSD_OK;
}

int check_ws(const ssd_model *m, int B, int M, void *ws, size_t ws_bytes, Workspace *out) {
    if (!ws) return SSD_E_ARG;
    if (B * M > kMaxRows || M > kMaxRowsPerSeq || M < 1) return SSD_E_CAPACITY;
    if (((uintptr_t)ws & 255) != 0) return SSD_E_ARG;
    *out = carve(m, B, M, (uint8_t *)ws);
    if (out->bytes > ws_bytes) return SSD_E_CAPACITY;
    return SSD_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------
extern "C" {

size_t ssd_model_desc_bytes(const ssd_arch *arch) {
    if (!arch || arch->n_layers < 1 || arch->dtype != 1) return 0;
    return sizeof(ModelDesc) + sizeof(LayerDesc) * (size_t)arch->n_layers;
}

int ssd_model_create(const ssd_arch *arch, const void *const *dev_weights, int n_tensors, void *dev_desc,
                     size_t desc_bytes, ssd_model **out) {
    if (!arch || !dev_weights || !out) return SSD_E_ARG;
    if (arch->dtype == 1 && (!dev_desc || desc_bytes < ssd_model_desc_bytes(arch) || ((uintptr_t)dev_desc & 255)))
        return SSD_E_ARG;
    int rc = check_arch(*arch);
    if (rc) return rc;
    if (n_tensors != 2 + PER_LAYER * arch->n_layers + 3) return SSD_E_ARG;
    // required tensors
    auto need = [&](int i) { return dev_weights[i] != nullptr; };
    if (!need(T_TOK) || (arch->pos == 0 && !need(T_POS))) return SSD_E_ARG;
    for (int l = 0; l < arch->n_layers; ++l) {
        const int b = T_L0 + PER_LAYER * l;
        if (!need(b + L_LN1G) || !need(b + L_WQKV) || !need(b + L_WO) || !need(b + L_LN2G) || !need(b + L_WIN) ||
            !need(b + L_WOUT))
            return SSD_E_ARG;
    }
    const int fb = T_L0 + PER_LAYER * arch->n_layers;
    if (!need(fb) || (!arch->tie_lm_head && !need(fb + 2))) return SSD_E_ARG;
    if ((rc = init_device_once())) return rc;
    ssd_model *m = new (std::nothrow) ssd_model();
    if (!m) return SSD_E_ARG;
    m->a = *arch;
    m->w.assign(dev_weights, dev_weights + n_tensors);
    m->d_in = arch->act == 1 ? 2 * arch->d_ff : arch->d_ff;
    if ((rc = build_maps(m))) {
        delete m;
        return rc;
    }
    m->dev_desc = nullptr;
    if (arch->dtype == 1) {
        // the tensor maps and vector pointers the persistent kernel walks, copied once to the caller's block
        std::vector<uint8_t> host(ssd_model_desc_bytes(arch), 0);
        ModelDesc *md = reinterpret_cast<ModelDesc *>(host.data());
        // (its own maps: 256-row boxes, one MMA's worth of weight rows)
        int mrc = make_map(&md->tm_lm, lm_matrix(m), arch->vocab, arch->d_model, kTileNP);
        md->lnf_g = (const float *)fw(m, 0);
        md->lnf_b = (const float *)fw(m, 1);
        LayerDesc *ld = reinterpret_cast<LayerDesc *>(md + 1);
        for (int l = 0; l < arch->n_layers; ++l) {
            mrc |= make_map(&ld[l].tm[0], lw(m, l, L_WQKV), 3 * arch->d_model, arch->d_model, kTileNP);
            mrc |= make_map(&ld[l].tm[1], lw(m, l, L_WO), arch->d_model, arch->d_model, kTileNP);
            mrc |= make_map(&ld[l].tm[2], lw(m, l, L_WIN), m->d_in, arch->d_model, kTileNP);
            mrc |= make_map(&ld[l].tm[3], lw(m, l, L_WOUT), arch->d_model, arch->d_ff, kTileNP);
            ld[l].ln1_g = (const float *)lw(m, l, L_LN1G); ld[l].ln1_b = (const float *)lw(m, l, L_LN1B);
            ld[l].b_qkv = (const float *)lw(m, l, L_BQKV); ld[l].b_o = (const float *)lw(m, l, L_BO);
            ld[l].ln2_g = (const float *)lw(m, l, L_LN2G); ld[l].ln2_b = (const float *)lw(m, l, L_LN2B);
            ld[l].b_in = (const float *)lw(m, l, L_BIN); ld[l].b_out = (const float *)lw(m, l, L_BOUT);
        }
        if (mrc || cudaMemcpy(dev_desc, host.data(), host.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
            delete m;
            return SSD_E_CUDA;
        }
        m->dev_desc = reinterpret_cast<const ModelDesc *>(dev_desc);
    }
    *out = m;
    return SSD_OK;
}

int ssd_set_attention_mode(int mode) {
    if (mode < 0 || mode > 3) return SSD_E_ARG;
    g_attn_mode = mode;
    return SSD_OK;
}

int ssd_set_prefill_mode(int mode) {
    if (mode < 0 || mode > 3) return SSD_E_ARG;
    g_prefill_mode = mode;
    return SSD_OK;
}

size_t ssd_prefill_workspace_bytes(const ssd_model *m, int batch, int rows_per_seq) {
    if (!m || batch < 1 || rows_per_seq < 1 || !wide_path_ok(m)) return 0;
    if ((long long)batch * rows_per_seq > kWideMaxRows) rows_per_seq = kWideMaxRows / batch;
    if (rows_per_seq < 1) return 0;
    return carve_wide(m, batch, rows_per_seq, nullptr).bytes;
}

int ssd_set_persistent(int enable) {
    g_persistent = enable != 0;
    return SSD_OK;
}

int ssd_model_share_prefix(const ssd_model *target, int n_layers, ssd_model **draft_out) {
    if (!target || !draft_out || n_layers < 1 || n_layers > target->a.n_layers) return SSD_E_ARG;
    ssd_model *m = new (std::nothrow) ssd_model();
    if (!m) return SSD_E_ARG;
    m->a = target->a;
    m->a.n_layers = n_layers;
    m->d_in = target->d_in;
    m->dev_desc = target->dev_desc;  // LM head first, then the layers: a prefix of the layers is a prefix of the block
    m->w.assign(target->w.begin(), target->w.begin() + T_L0 + PER_LAYER * n_layers);
    m->w.insert(m->w.end(), target->w.end() - 3, target->w.end());
    if (!target->tm.empty()) {
        m->tm.assign(target->tm.begin(), target->tm.begin() + 4 * n_layers);
        m->tm.push_back(target->tm.back());
    }
    *draft_out = m;
    return SSD_OK;
}

void ssd_model_destroy(ssd_model *m) { delete m; }

static size_t kv_header_bytes(int batch) { return align_up(sizeof(int32_t) * (kHeaderInts + 2 * (size_t)batch), 1024); }

size_t ssd_kv_bytes(const ssd_model *m, int batch, int max_len) {
    if (!m || batch < 1 || max_len < 1) return 0;
    size_t es = m->a.dtype ? 2 : 4;
    return kv_header_bytes(batch) + (size_t)m->a.n_layers * batch * 2 * m->a.d_model * max_len * es;
}

size_t ssd_workspace_bytes(const ssd_model *m, int batch, int rows_per_seq, int max_len) {
    (void)max_len;
    if (!m || batch < 1 || rows_per_seq < 1 || batch * rows_per_seq > kMaxRows || rows_per_seq > kMaxRowsPerSeq) return 0;
    return carve(m, batch, rows_per_seq, nullptr).bytes;
}

int kv_init(const ssd_model *m, int batch, int max_len, void *dev_buf, size_t bytes, void *stream, ssd_kv **out) {
    if (!m || !dev_buf || !out || batch < 1 || max_len < 1) return SSD_E_ARG;
    if (batch > kMaxRows) return SSD_E_CAPACITY;
    if (((uintptr_t)dev_buf & 255) != 0) return SSD_E_ARG;
    if (bytes < ssd_kv_bytes(m, batch, max_len)) return SSD_E_CAPACITY;
    ssd_kv *kv = new (std::nothrow) ssd_kv();
    if (!kv) return SSD_E_ARG;
    kv->a = m->a;
    kv->B = batch;
    kv->S = max_len;
    kv->buf = (uint8_t *)dev_buf;
    kv->status = (int32_t *)dev_buf;
    kv->len = kv->status + kHeaderInts;
    kv->keep = kv->len + batch;
    kv->cache = kv->buf + kv_header_bytes(batch);
    kv->esize = m->a.dtype ? 2 : 4;
    kv->layer_bytes = (size_t)batch * 2 * m->a.d_model * max_len * kv->esize;
    kv->len_ub = 0;
    kv->last_rows = 0;
    kv->op_seq = 0;
    kv->growth_total = 0;
    memset(kv->growth_at, 0, sizeof(kv->growth_at));
    kv->mailbox = kv->mailbox_dev = nullptr;
    {   // eight bytes of mapped host memory (not device memory); without it the bound is only advanced
        void *h = nullptr, *d = nullptr;
        if (cudaHostAlloc(&h, sizeof(unsigned long long), cudaHostAllocMapped) == cudaSuccess) {
            *reinterpret_cast<unsigned long long *>(h) = 0;
            if (cudaHostGetDevicePointer(&d, h, 0) == cudaSuccess) {
                kv->mailbox = (unsigned long long *)h;
                kv->mailbox_dev = (unsigned long long *)d;
            } else {
                cudaFreeHost(h);
            }
        }
        (void)cudaGetLastError();
    }
    // Rows beyond a sequence's length are read (masked) by the chunked attention: they must hold finite numbers.
    if (cudaMemsetAsync(kv->cache, 0, kv->layer_bytes * m->a.n_layers, (cudaStream_t)stream) != cudaSuccess) {
        kv_destroy(kv);
        return SSD_E_CUDA;
    }
    kv->tm_rows_ok = false;
    {
        const long long rows = (long long)m->a.n_layers * batch * 2 * m->a.n_heads * max_len;
        if (m->a.dtype == 1 && m->a.head_dim == 128 && rows < (1ll << 31))
            kv->tm_rows_ok = make_map(&kv->tm_rows, kv->cache, (int)rows, 128, kTcChunk) == SSD_OK;
    }
    if (cudaMemsetAsync(dev_buf, 0, kv_header_bytes(batch), (cudaStream_t)stream) != cudaSuccess) {
        kv_destroy(kv);
        return SSD_E_CUDA;
    }
    *out = kv;
    return SSD_OK;
}

void kv_destroy(ssd_kv *kv) {
    if (kv && kv->mailbox) {
        // the word may still be written by queued kernels: wait for the device before it goes away
        cudaDeviceSynchronize();
        cudaFreeHost(kv->mailbox);
    }
    delete kv;
}

static bool same_cache_shape(const ssd_model *m, const ssd_kv *kv) {
    return m->a.n_layers == kv->a.n_layers && m->a.d_model == kv->a.d_model && m->a.n_heads == kv->a.n_heads &&
           m->a.dtype == kv->a.dtype;
}

int kv_prefill(ssd_model *m, ssd_kv *kv, const int32_t *dev_tokens, const int32_t *dev_n_tokens, int max_tokens,
               void *dev_ws, size_t ws_bytes, void *stream) {
    if (!m || !kv || !dev_tokens || !dev_n_tokens || max_tokens < 0) return SSD_E_ARG;
    if (!same_cache_shape(m, kv)) return SSD_E_ARG;
    if (kv_bound(kv) + max_tokens > kv->S) return SSD_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    if (max_tokens == 0) return SSD_OK;
    if (wide_path_ok(m) && dev_ws && ((uintptr_t)dev_ws & 255) == 0) {
        // many rows per pass: the largest share of the prompt (in equal passes) whose buffers fit the workspace
        int cap = kWideMaxRows / kv->B;
        while (cap >= 1 && carve_wide(m, kv->B, cap < max_tokens ? cap : max_tokens, nullptr).bytes > ws_bytes) cap /= 2;
        if (cap >= 1) {
            const int passes = ceil_div(max_tokens, cap);
            int Cw = ceil_div(ceil_div(max_tokens, passes), 16) * 16;
            if (Cw > max_tokens) Cw = max_tokens;
            if (Cw > cap) Cw = cap;
            if (g_prefill_mode >= 2 || kv->B * Cw >= kWideMinRows) {
                const WideWs ww = carve_wide(m, kv->B, Cw, (uint8_t *)dev_ws);
                const int chunks = ceil_div(max_tokens, Cw);
                for (int c = 0; c < chunks; ++c) {
                    LAUNCH(prefill_rows_kernel, ceil_div(kv->B, 64), 64, 0, st, dev_n_tokens, c, Cw, ww.n_rows_tmp, kv->B);
                    int rcw = forward_wide(m, kv, dev_tokens + (size_t)c * Cw, max_tokens, Cw, ww.n_rows_tmp, ww, st);
                    if (rcw) return rcw;
                    const unsigned seq = kv_note_op(kv, Cw);
                    LAUNCH(kv_commit_rows_kernel, 1, 64, 0, st, kv->len, ww.ri.n_eff, kv->B, kv->mailbox_dev, seq);
                }
                return SSD_OK;
            }
        }
    }
    // rows per sequence and pass: as many as the row limits and the caller's workspace allow (every pass streams
    // all weights once, whatever its rows)
    int C = kMaxRows / kv->B;
    if (C > kMaxRowsPerSeq) C = kMaxRowsPerSeq;
    if (C < 1) return SSD_E_CAPACITY;
    Workspace w;
    int rc = check_ws(m, kv->B, C, dev_ws, ws_bytes, &w);
    while (rc == SSD_E_CAPACITY && C > 1) {
        C = C > 8 ? C / 2 : C - 1;
        rc = check_ws(m, kv->B, C, dev_ws, ws_bytes, &w);
    }
    if (rc) return rc;
    const int chunks = ceil_div(max_tokens, C);
    for (int c = 0; c < chunks; ++c) {
        LAUNCH(prefill_rows_kernel, ceil_div(kv->B, 64), 64, 0, st, dev_n_tokens, c, C, w.n_rows_tmp, kv->B);
        if ((rc = forward(m, kv, dev_tokens + (size_t)c * C, max_tokens, C, w.n_rows_tmp, false, w, st))) return rc;
        const unsigned seq = kv_note_op(kv, C);
        LAUNCH(kv_commit_rows_kernel, 1, 64, 0, st, kv->len, w.ri.n_eff, kv->B, kv->mailbox_dev, seq);
    }
    return SSD_OK;
}

int draft_step(ssd_model *draft, ssd_kv *dkv, const int32_t *dev_tokens_in, int tokens_stride, int rows_in,
               const int32_t *dev_n_in, float temperature, const float *dev_u, int u_stride, int32_t *dev_token_out,
               int token_out_stride, float *dev_q_out, size_t q_stride, void *dev_ws, size_t ws_bytes, void *stream) {
    if (!draft || !dkv || !dev_tokens_in || !dev_u || !dev_token_out || !dev_q_out) return SSD_E_ARG;
    if (rows_in < 1 || rows_in > 2 || tokens_stride < rows_in || temperature < 0.f) return SSD_E_ARG;
    if (!same_cache_shape(draft, dkv)) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w;
    int rc = check_ws(draft, dkv->B, rows_in, dev_ws, ws_bytes, &w);
    if (rc) return rc;
    if ((rc = forward(draft, dkv, dev_tokens_in, tokens_stride, rows_in, dev_n_in, true, w, st))) return rc;
    DraftTailArgs t;
    t.logits = w.logits; t.M = rows_in; t.V = draft->a.vocab; t.n_eff = w.ri.n_eff;
    t.inv_t = temperature > 0.f ? 1.0f / temperature : 0.f;
    t.u = dev_u; t.u_stride = u_stride;
    t.token_out = dev_token_out; t.token_stride = token_out_stride;
    t.q_out = dev_q_out; t.q_stride = q_stride;
    t.top_k = g_top_k; t.top_p = g_top_p;
    LAUNCH(draft_tail_kernel, dkv->B * kTailCluster, kTailThreads, 0, st, t);
    const unsigned seq = kv_note_op(dkv, rows_in);
    LAUNCH(kv_commit_rows_kernel, 1, 64, 0, st, dkv->len, w.ri.n_eff, dkv->B, dkv->mailbox_dev, seq);
    return SSD_OK;
}

int draft_steps(ssd_model *draft, ssd_kv *dkv, int n_steps, const int32_t *dev_tokens_in, int tokens_stride, int rows_in,
                const int32_t *dev_n_in, float temperature, const float *dev_u, int u_stride, int32_t *dev_tokens_out,
                int token_out_stride, float *dev_q_out, size_t q_stride, void *dev_ws, size_t ws_bytes, void *stream) {
    if (!draft || !dkv || !dev_tokens_in || !dev_u || !dev_tokens_out || !dev_q_out) return SSD_E_ARG;
    if (n_steps < 1 || n_steps > kMaxRowsPerSeq || rows_in < 1 || rows_in > 2 || tokens_stride < rows_in ||
        temperature < 0.f || token_out_stride < n_steps || u_stride < n_steps ||
        q_stride < (size_t)n_steps * (size_t)draft->a.vocab)
        return SSD_E_ARG;
    if (!same_cache_shape(draft, dkv)) return SSD_E_ARG;
    const bool restricted = g_top_k > 0 || (g_top_p > 0.f && g_top_p < 1.f);
    if (!single_kernel_path(draft) || restricted) {
        // the same steps, one call each (fp32 models, head dimensions the single kernel does not cover, or a
        // sampling restriction, whose threshold search lives in the stand-alone tail kernel)
        for (int s = 0; s < n_steps; ++s) {
            const int rc = s == 0 ? draft_step(draft, dkv, dev_tokens_in, tokens_stride, rows_in, dev_n_in, temperature, dev_u,
                                               u_stride, dev_tokens_out, token_out_stride, dev_q_out, q_stride, dev_ws,
                                               ws_bytes, stream)
                                  : draft_step(draft, dkv, dev_tokens_out + (s - 1), token_out_stride, 1, nullptr, temperature,
                                               dev_u + s, u_stride, dev_tokens_out + s, token_out_stride,
                                               dev_q_out + (size_t)s * draft->a.vocab, q_stride, dev_ws, ws_bytes, stream);
            if (rc) return rc;
        }
        return SSD_OK;
    }
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w;
    int rc = check_ws(draft, dkv->B, rows_in, dev_ws, ws_bytes, &w);
    if (rc) return rc;
    DraftLoop dl;
    dl.n_steps = n_steps;
    dl.inv_t = temperature > 0.f ? 1.0f / temperature : 0.f;
    dl.u = dev_u; dl.u_stride = u_stride;
    dl.tok_out = dev_tokens_out; dl.tok_out_stride = token_out_stride;
    dl.q_out = dev_q_out; dl.q_stride = q_stride;
    dl.mb_seq = kv_note_op(dkv, rows_in + n_steps - 1);
    return forward_persistent(draft, dkv, dev_tokens_in, tokens_stride, rows_in, dev_n_in, true, w, st, &dl);
}

size_t verify_scratch_bytes(int batch, int K) {
    if (batch < 1 || K < 0) return 0;
    return align_up(sizeof(RowStat) * (size_t)batch * (K + 1), 256) + align_up(sizeof(RowFilter) * (size_t)batch * (K + 1), 256);
}

static int run_verify_tail(const float *logits, int B, int K, int V, const int32_t *rows, const float *q,
                           const float *u, float temperature, int32_t *n_acc, int32_t *next, int next_stride,
                           float *p_debug, int32_t *keep, RowStat *stats, RowFilter *filt, cudaStream_t st) {
    VerifyArgs v;
    v.logits = logits; v.K = K; v.V = V; v.rows = rows; v.q = q; v.u = u;
    v.inv_t = temperature > 0.f ? 1.0f / temperature : 0.f;
    v.n_accepted = n_acc; v.next_token = next; v.next_stride = next_stride;
    v.p_debug = p_debug; v.keep = keep; v.stats = stats;
    v.filt = filt; v.top_k = filt ? g_top_k : 0; v.top_p = filt ? g_top_p : 1.0f;
    LAUNCH(row_stats_kernel, dim3((K + 1) * kTailCluster, B), kTailThreads, 0, st, v);
    LAUNCH(verify_kernel, B * kTailCluster, kTailThreads, 0, st, v);
    return SSD_OK;
}

int verify_from_logits(const float *dev_logits, int batch, int K, int vocab, const int32_t *dev_rows,
                       const float *dev_q, const float *dev_u, float temperature, int32_t *dev_n_accepted,
                       int32_t *dev_next_token, int next_token_stride, float *dev_p_debug, void *dev_scratch,
                       size_t scratch_bytes, void *stream) {
    if (!dev_logits || !dev_rows || !dev_u || !dev_n_accepted || !dev_next_token || !dev_scratch) return SSD_E_ARG;
    if (batch < 1 || K < 0 || K + 1 > kMaxRowsPerSeq || vocab < 1 || temperature < 0.f || next_token_stride < 1)
        return SSD_E_ARG;
    if (K > 0 && !dev_q) return SSD_E_ARG;
    if (scratch_bytes < verify_scratch_bytes(batch, K)) return SSD_E_CAPACITY;
    return run_verify_tail(dev_logits, batch, K, vocab, dev_rows, dev_q, dev_u, temperature, dev_n_accepted,
                           dev_next_token, next_token_stride, dev_p_debug, nullptr, (RowStat *)dev_scratch,
                           (RowFilter *)((uint8_t *)dev_scratch + align_up(sizeof(RowStat) * (size_t)batch * (K + 1), 256)),
                           (cudaStream_t)stream);
}

int target_verify(ssd_model *target, ssd_kv *tkv, const int32_t *dev_rows, int K, const float *dev_q,
                  const float *dev_u, float temperature, int32_t *dev_n_accepted, int32_t *dev_next_token,
                  int next_token_stride, float *dev_p_debug, void *dev_ws, size_t ws_bytes, void *stream) {
    if (!target || !tkv || !dev_rows || !dev_u || !dev_n_accepted || !dev_next_token) return SSD_E_ARG;
    if (K < 0 || K + 1 > kMaxRowsPerSeq || temperature < 0.f || next_token_stride < 1) return SSD_E_ARG;
    if (K > 0 && !dev_q) return SSD_E_ARG;
    if (!same_cache_shape(target, tkv)) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w;
    int rc = check_ws(target, tkv->B, K + 1, dev_ws, ws_bytes, &w);
    if (rc) return rc;
    if ((rc = forward(target, tkv, dev_rows, K + 1, K + 1, nullptr, true, w, st))) return rc;
    return run_verify_tail(w.logits, tkv->B, K, target->a.vocab, dev_rows, dev_q, dev_u, temperature, dev_n_accepted,
                           dev_next_token, next_token_stride, dev_p_debug, tkv->keep, w.stats, w.filt, st);
}

int kv_commit(ssd_kv *kv, const int32_t *dev_n_keep, void *stream) {
    if (!kv) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const unsigned seq = kv_note_op(kv, kv->last_rows > 0 ? kv->last_rows : 1);
    LAUNCH(kv_commit_kernel, 1, 64, 0, st, kv->len, dev_n_keep ? dev_n_keep : kv->keep, kv->B, kv->S, kv->status,
           kv->mailbox_dev, seq);
    return SSD_OK;
}

int kv_rollback(ssd_kv *kv, const int32_t *dev_new_len, void *stream) {
    if (!kv || !dev_new_len) return SSD_E_ARG;
    const unsigned seq = kv_note_op(kv, 0);
    LAUNCH(kv_rollback_kernel, 1, 64, 0, (cudaStream_t)stream, kv->len, dev_new_len, kv->B, kv->mailbox_dev, seq);
    return SSD_OK;
}

int spec_advance(ssd_kv *tkv, ssd_kv *dkv, int32_t *dev_rows, int K, const int32_t *dev_n_accepted,
                 const int32_t *dev_next_token, int next_token_stride, int32_t *dev_out_tokens, int out_cap,
                 int32_t *dev_out_count, int32_t *dev_draft_in, int32_t *dev_draft_n_in, void *stream) {
    if (!tkv || !dev_rows || !dev_n_accepted || !dev_next_token || K < 0 || next_token_stride < 1) return SSD_E_ARG;
    if (dkv && dkv->B != tkv->B) return SSD_E_ARG;
    AdvanceArgs a;
    a.tlen = tkv->len; a.dlen = dkv ? dkv->len : nullptr;
    a.rows = dev_rows; a.K = K; a.B = tkv->B;
    a.n_accepted = dev_n_accepted; a.next_token = dev_next_token; a.next_stride = next_token_stride;
    a.out_tokens = dev_out_tokens; a.out_cap = out_cap; a.out_count = dev_out_count;
    a.draft_in = dev_draft_in; a.draft_n_in = dev_draft_n_in;
    a.t_mailbox = tkv->mailbox_dev;
    a.t_seq = kv_note_op(tkv, K + 1);
    a.d_mailbox = dkv ? dkv->mailbox_dev : nullptr;
    a.d_seq = dkv ? kv_note_op(dkv, 0) : 0u;  // the draft cache is only cut back here
    LAUNCH(spec_advance_kernel, 1, 64, 0, (cudaStream_t)stream, a);
    return SSD_OK;
}

int kv_lengths(ssd_kv *kv, int32_t *host_out, void *stream) {
    if (!kv || !host_out) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(host_out, kv->len, sizeof(int32_t) * kv->B, cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    int mx = 0;
    for (int b = 0; b < kv->B; ++b) mx = host_out[b] > mx ? host_out[b] : mx;
    kv->len_ub = mx;  // the bound is exact again
    return SSD_OK;
}

int ssd_device_status(ssd_kv *kv, int32_t *host_out, void *stream) {
    if (!kv || !host_out) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_OK(cudaMemcpyAsync(host_out, kv->status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CUDA_OK(cudaStreamSynchronize(st));
    return SSD_OK;
}

int attention_rows(ssd_model *m, ssd_kv *kv, int layer, const float *dev_q, int rows, float *dev_out, void *dev_ws,
                   size_t ws_bytes, void *stream) {
    if (!m || !kv || !dev_q || !dev_out || layer < 0 || layer >= m->a.n_layers) return SSD_E_ARG;
    if (!same_cache_shape(m, kv)) return SSD_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace w;
    int rc = check_ws(m, kv->B, rows, dev_ws, ws_bytes, &w);
    if (rc) return rc;
    // the probe rows are not appended: row j attends whatever the cache holds at 0 .. len + j
    if ((rc = run_setup(m, kv, rows, nullptr, w, st))) return rc;
    CombineArgs cb;
    memset(&cb, 0, sizeof(cb));
    cb.out_f32 = dev_out;
    return run_attention(m, kv, layer, dev_q, rows, w, cb, st);
}

int ssd_last_logits(const ssd_model *m, int batch, int rows_per_seq, const void *dev_ws, size_t ws_bytes,
                    float *dev_out, void *stream) {
    if (!m || !dev_out) return SSD_E_ARG;
    Workspace w;
    int rc = check_ws(m, batch, rows_per_seq, const_cast<void *>(dev_ws), ws_bytes, &w);
    if (rc) return rc;
    CUDA_OK(cudaMemcpyAsync(dev_out, w.logits, sizeof(float) * (size_t)batch * rows_per_seq * m->a.vocab,
                            cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return SSD_OK;
}

// ---------------------------------------------------------------------------------------------
// verify_from_logits for callers that cannot allocate device memory.
//
// The row statistics (max, normaliser, argmax of every logits row) that the two tail kernels hand
// to each other live in a fixed array inside the library image instead of a caller buffer.  The
// array is part of every context that loads the library (64 KB per GPU, held until exit).
static __device__ __align__(256) RowStat g_noalloc_stats[SSD_NOALLOC_MAX_ROWS];

namespace {
constexpr int kMaxDevices = 64;
RowStat *g_noalloc_ptr[kMaxDevices] = {nullptr};
std::mutex g_noalloc_mu;

// In host code `g_noalloc_stats` is only a handle for the runtime, not a device address: the real
// address differs per device and has to be asked for with that device current.
int noalloc_scratch(RowStat **out) {
    int dev = -1;
    CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SSD_E_CAPACITY;
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_stats) != cudaSuccess || !p) return SSD_E_CUDA;
        g_noalloc_ptr[dev] = (RowStat *)p;
    }
    *out = g_noalloc_ptr[dev];
    return SSD_OK;
}
}  // namespace

int verify_from_logits_noalloc(const float *dev_logits, int batch, int K, int vocab, const int32_t *dev_rows,
                               const float *dev_q, const float *dev_u, float temperature,
                               int32_t *dev_n_accepted, int32_t *dev_next_token, int next_token_stride,
                               float *dev_p_debug, void *stream) {
    if (!dev_logits || !dev_rows || !dev_u || !dev_n_accepted || !dev_next_token) return SSD_E_ARG;
    if (batch < 1 || K < 0 || K + 1 > kMaxRowsPerSeq || vocab < 1 || temperature < 0.f || next_token_stride < 1)
        return SSD_E_ARG;
    if (K > 0 && !dev_q) return SSD_E_ARG;
    if ((long long)batch * (K + 1) > SSD_NOALLOC_MAX_ROWS) return SSD_E_CAPACITY;
    if (g_top_k > 0 || (g_top_p > 0.f && g_top_p < 1.f)) return SSD_E_UNIMPL;  // its fixed array has no room for the restriction
    RowStat *stats = nullptr;
    int rc = noalloc_scratch(&stats);
    if (rc) return rc;
    // every entry a call reads is written earlier in the same call (row_stats_kernel fills
    // stats[0 .. batch*(K+1)) before verify_kernel looks at them): nothing has to start at zero
    return run_verify_tail(dev_logits, batch, K, vocab, dev_rows, dev_q, dev_u, temperature, dev_n_accepted,
                           dev_next_token, next_token_stride, dev_p_debug, nullptr, stats, nullptr, (cudaStream_t)stream);
}

uint64_t ssd_launch_count(void) { return g_launches.load(); }

int ssd_set_sampling(int top_k, float top_p) {
    if (top_k < 0 || !(top_p > 0.f) || top_p > 1.f) return SSD_E_ARG;
    g_top_k = top_k;
    g_top_p = top_p;
    return SSD_OK;
}

int ssd_set_wait_limit(long long cycles) {
    if (cycles < 0) return SSD_E_ARG;
    g_wait_cycles = cycles;
    return SSD_OK;
}

// One thread waits, through the same bounded-wait helper the other kernels use, on a barrier that nobody
// arrives at; the wait runs out and the kernel records the time-out and returns.
__global__ void wait_probe_kernel(int32_t *status, long long limit) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_limit(&bar, 0, limit)) set_status(status, kTimeoutCode);
    }
}

int ssd_wait_probe(ssd_kv *kv, void *stream) {
    if (!kv) return SSD_E_ARG;
    LAUNCH(wait_probe_kernel, 1, 32, 0, (cudaStream_t)stream, kv->status, g_wait_cycles > 0 ? g_wait_cycles : kWaitCycles);
    return SSD_OK;
}

int ssd_set_trace(int enable) {
    g_trace = enable != 0;
    return SSD_OK;
}

int ssd_read_trace(const ssd_model *m, int batch, int rows_per_seq, const void *dev_ws, size_t ws_bytes,
                   uint64_t *host_out, int max_entries, int *n_out, void *stream) {
    if (!m || !host_out || !n_out || max_entries < 1) return SSD_E_ARG;
    Workspace w;
    int rc = check_ws(m, batch, rows_per_seq, const_cast<void *>(dev_ws), ws_bytes, &w);
    if (rc) return rc;
    std::vector<unsigned long long> tmp(kTraceSlots);
    CUDA_OK(cudaMemcpyAsync(tmp.data(), w.trace, sizeof(unsigned long long) * kTraceSlots, cudaMemcpyDeviceToHost,
                            (cudaStream_t)stream));
    CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    int n = 0;
    while (n < kTraceSlots && n < max_entries && tmp[n] != 0) { host_out[n] = tmp[n]; ++n; }
    *n_out = n;
    return SSD_OK;
}

int ssd_gemm_profile(int enable) {
    g_prof = enable != 0;
    g_prof_used = 0;
    return SSD_OK;
}

int ssd_gemm_profile_read(uint64_t *launches, double *total_ms, int reset) {
    if (!launches || !total_ms) return SSD_E_ARG;
    CUDA_OK(cudaDeviceSynchronize());
    double ms = 0.0;
    for (size_t i = 0; i + 1 < g_prof_used; i += 2) {
        float t = 0.f;
        CUDA_OK(cudaEventElapsedTime(&t, g_prof_events[i], g_prof_events[i + 1]));
        ms += t;
    }
    *launches = g_prof_used / 2;
    *total_ms = ms;
    if (reset) g_prof_used = 0;
    return SSD_OK;
}

const char *ssd_strerror(int status) {
    switch (status) {
        case SSD_OK: return "ok";
        case SSD_E_ARG: return "bad argument";
        case SSD_E_SHAPE: return "architecture not covered by the kernels";
        case SSD_E_CAPACITY: return "rows do not fit (cache, workspace or position table)";
        case SSD_E_CUDA: return "CUDA call failed";
        case SSD_E_TIMEOUT: return "a bounded device-side wait gave up";
        case SSD_E_UNIMPL: return "not implemented";
        default: return "unknown status";
    }
}

}  // extern "C"

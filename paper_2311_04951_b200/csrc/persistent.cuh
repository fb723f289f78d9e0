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
//   warp 8      producer: TMA issue for weight tiles, free-running across phase boundaries
//   warp 5      (one lane) during a GEMM phase: bulk copies of that GEMM's operand tiles, which
//               exist only once the grid barrier of the phase that wrote them has been passed
//   warp 4      (one lane) issues the GEMM: per ring stage four tcgen05.mma, each (activation
//               rows, hi and lo, as the M = 64 or 128 operand) x (256 weight rows as the N
//               operand) x 16 k, accumulating in tensor memory.  A K = 16 MMA step costs about
//               120 cycles whatever M and N are, so the weights sit on the side that lets one
//               step consume the most of them (8 KB).  tcgen05.commit hands the stage back to
//               the producer and, at the end of a tile segment, the accumulator to the
//               epilogue; two accumulator buffers overlap that epilogue with the next MMAs
//   warps 0-3   epilogue: tensor memory -> registers with the 16-lane x 256-bit load, which
//               puts a row's hi and lo products in one thread; hi + lo goes through a small
//               shared-memory tile so that all four warps add it (+ bias from the segment that
//               holds k-chunk 0) to the output with 16-byte vector reductions: a reduction
//               costs its warp a memory latency, so there must be few of them per thread
//   warps 0-7   between GEMM phases: the small phases (row set-up, embedding, norm, activation,
//               attention with rotary + KV append + split merge - on warp-level MMAs, or for head
//               dim 128 and long splits on tcgen05 with its own roles, see attention_item_tc),
//               which leave every GEMM operand in global memory already split into bf16 hi + lo,
//               and the grid barriers
// Every phase is a function of its own (not inlined) that reads a shared-memory copy of the kernel
// parameters and keeps what must survive between calls in shared memory: the phase loop holds nothing
// across calls, because a spilled value or a read through the parameter bank would be a trip to L2 at
// the head of every one of the pass's ~130-260 phases (227 KB of shared memory leave next to no L1).
// Every wait (mbarrier, grid barrier) is bounded; on time-out SSD_E_TIMEOUT is recorded, the CTA
// stops taking work, waits (bounded) for its copies in flight, drains the tensor core, frees its
// tensor memory and returns.  A parity wait is used only where the waiter follows every phase of its
// barrier in order and the barrier cannot pass it by two phases.
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
constexpr int kMaxStagedLayers = 64;  // layers whose gain / bias pointers are staged in shared memory
constexpr int kTileNP = 256;                        // weight rows per tile: the N of one MMA
constexpr int kWTileBytesP = kTileNP * kTileK * 2;  // 32 KB

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
    // GEMM operands in global memory (normalised rows - two sets for parallel-residual blocks -,
    // attention output, MLP activation), stored the way a ring stage wants them: one contiguous
    // tile per 64-wide k-chunk, 2 rk rows of 128 bytes (per block of 8 rows: their 8 bf16 hi rows, then
    // their 8 lo rows), 16-byte chunks already in 128-byte-swizzle order, so one linear bulk copy
    // fetches a tile.
    // (A strided 2-D tensor copy of the same tile costs a sixth of the weight stream's bandwidth.)
    __nv_bfloat16 *op[4];
    int op_ld[4];  // K of each operand
    int rk;
    const ModelDesc *md;
    // architecture
    int n_layers, d, H, Dh, F, d_in, V, norm_kind, swiglu, parallel, rotary_dim, learned_pos, is_bf16_emb;
    float eps, rotary_base, attn_scale;
    double inv_d;  // 1 / d (the norms' statistics are taken in fp64; a division there is a long routine)
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
    // Shared-memory ring: slots [0, stages_lo) hold weights at any time; slots [stages_lo, stages) share
    // their bytes with the attention scratch (at attn_smem_off = stages_lo * stage bytes) and are used
    // only between attention phases.  bar_off: byte offset of the barriers behind both.
    int stages, stages_lo, attn_smem_off, bar_off;
    unsigned long long *trace;  // optional: CTA 0 stamps the global timer after every grid barrier
    // tensor-core attention (head dim 128): the whole cache as rows of Dh bf16, box 64 x 128 rows
    CUtensorMap tm_kv;
    const CUtensorMap *tm_kv_ptr;  // where the copy engine can read tm_kv (set by the kernel: see params copy)
    int attn_tc;             // 0: attention_item (warp MMAs, 16-row tiles); 1: attention_item_tc; 2: attention_item_mma8 (up to eight rows, hi and lo in one MMA tile)
    int kv_rows_per_layer;   // B * 2 * H * S
    int attn_ctas;           // min(attention items, CTAs): set by the host together with the split plan
    int overlap_out;         // parallel-residual block and at most half of the CTAs on attention
    long long wait_cycles;   // bound of every wait that takes work (see Shared::wait_limit)
    // Several draft steps in one launch (n_steps >= 1; the draft loop of a speculative iteration).  With tail == 1
    // every step ends inside the kernel: the logits of each sequence's last fed row become q = softmax(logits / T),
    // a token is drawn from q with the step's uniform, both are written out, the fed rows are committed, and the
    // next step feeds that token (one row per sequence).  cur_step is kept by the kernel in its copy of this block.
    int n_steps, tail, cur_step;
    float inv_t;                                   // 1 / T; 0 = greedy
    const float *u;     int u_stride;              // uniform of sequence b at step s: u[b * u_stride + s]
    int32_t *tok_out;   int tok_out_stride;        // token of step s: tok_out[b * tok_out_stride + s]
    float *q_out;       size_t q_stride;           // q row of step s: q_out + b * q_stride + s * V
    int32_t *len_rw;                               // the committed lengths, advanced after every step
    float *tp_m, *tp_s; int32_t *tp_a;             // per (sequence, CTA): max, sum of exp relative to it, argmax of the CTA's slice
    double *tp_mass;                               // per (sequence, CTA): mass of q in the CTA's slice
    int32_t *tail_hit;                             // [n_steps][B][2]: smallest index past u S (INT_MAX: none) / largest index with q > 0
    unsigned long long *mailbox; unsigned mb_seq;  // the largest length, reported to the host at the end
};

struct GemmDesc {
    const CUtensorMap *tmW;
    const __nv_bfloat16 *xop;  // tiled operand
    int N, Kd, n_tiles, kchunks;
    int need;  // grid barriers that must have completed before its operand exists
    int need_hi;  // ... before its tiles may use the ring slots shared with the attention scratch
    int kind;     // 0 qkv, 1 o, 2 in, 3 out, 4 LM head
    unsigned wait_attn;  // attention CTAs that must have signalled before its operand exists (0: a grid barrier covers it)
    float *out;
    int ldo;
    const float *bias;
};

__device__ __forceinline__ int n_gemms(const FwdParams &p) { return 4 * p.n_layers + (p.want_logits ? 1 : 0); }
// CTAs that run an attention item in a phase (each at most one when this is below the grid size).
__device__ __forceinline__ int attention_ctas(const FwdParams &p) { return p.attn_ctas; }
// Parallel-residual blocks with at most half of the CTAs on attention: the MLP-out GEMM depends on the
// activation, not on attention, so the CTAs without an attention item run it during the attention phase.
__device__ __forceinline__ bool overlap_mlp_out(const FwdParams &p) { return p.overlap_out != 0; }
__device__ __forceinline__ int barriers_per_layer(const FwdParams &p) { return p.parallel ? 4 : 8; }
__device__ __forceinline__ int attention_end(const FwdParams &p) { return overlap_mlp_out(p) ? 3 : 2; }  // barriers into the layer

// GEMM number gi in execution order.  sequential: qkv, o, in, out; parallel: qkv, in, o, out.
// Barrier count before layer l: 1 (set-up, embedding and first norm) + barriers_per_layer * l.
//   sequential layer: qkv | attention | o | norm2 | in | act | out | next norm   (8 barriers)
//   parallel layer:   qkv, in | attention + act | o, out | next norms            (4 barriers)
//   ... with few attention items: qkv, in | act | attention (some CTAs); out, then - once every attention CTA has
//       signalled - o (the others) | next norms   (4)
// Grid barriers of one step of a launch: the head, the layers', and five around the phases of the in-kernel tail.
__device__ __forceinline__ int step_barriers(const FwdParams &p) { return 1 + barriers_per_layer(p) * p.n_layers + (p.tail ? 5 : 0); }
constexpr int kStepShift = 12;  // a GEMM is named (step << kStepShift) | number within the forward

__device__ __forceinline__ GemmDesc gemm_desc(const FwdParams &p, int gi_step, const float *const *ltab = nullptr) {
    GemmDesc g;
    g.wait_attn = 0;
    const int step = gi_step >> kStepShift, gi = gi_step & ((1 << kStepShift) - 1);
    const int sb = step * step_barriers(p);  // barriers before this step
    const int l = gi >> 2, e = gi & 3;
    const int base = sb + 1 + barriers_per_layer(p) * l;
    if (l >= p.n_layers) {  // LM head
        g.tmW = &p.md->tm_lm; g.xop = p.op[OP_XN1];
        g.N = p.V; g.Kd = p.d; g.need = base; g.out = p.logits; g.ldo = p.V; g.bias = nullptr;
        g.kind = 4; g.need_hi = base - barriers_per_layer(p) + attention_end(p);  // end of the last attention phase
    } else {
        const LayerDesc *ld = layer_desc(p.md, l);
        int kind;  // 0 qkv, 1 o, 2 in, 3 out
        if (p.parallel && overlap_mlp_out(p)) kind = (e == 0) ? 0 : (e == 1) ? 2 : (e == 2) ? 3 : 1;  // out before o
        else if (p.parallel) kind = (e == 0) ? 0 : (e == 1) ? 2 : (e == 2) ? 1 : 3;
        else kind = e;
        g.tmW = &ld->tm[kind];
        g.kind = kind;
        // the attention phase of layer l ends at barrier base + 2; qkv precedes it (previous layer's counts)
        // (so does the MLP input GEMM of a parallel-residual block)
        g.need_hi = (kind == 0 || (kind == 2 && p.parallel)) ? (l == 0 ? sb : base - barriers_per_layer(p) + attention_end(p))
                                                             : base + attention_end(p);
        if (kind == 0) {
            g.xop = p.op[OP_XN1]; g.N = 3 * p.d; g.Kd = p.d; g.need = base;
            g.out = p.qkv; g.ldo = 3 * p.d; g.bias = ltab ? ltab[8 * l + 2] : ld->b_qkv;
        } else if (kind == 1) {
            g.xop = p.op[OP_AO]; g.N = p.d; g.Kd = p.d; g.need = base + 2;
            if (overlap_mlp_out(p)) g.wait_attn = (unsigned)(step * p.n_layers + l + 1) * (unsigned)attention_ctas(p);
            g.out = p.x; g.ldo = p.d; g.bias = ltab ? ltab[8 * l + 3] : ld->b_o;
        } else if (kind == 2) {
            g.xop = p.op[p.parallel ? OP_XN2 : OP_XN1]; g.N = p.d_in; g.Kd = p.d; g.need = p.parallel ? base : base + 4;
            g.out = p.t_in; g.ldo = p.d_in; g.bias = ltab ? ltab[8 * l + 6] : ld->b_in;
        } else {
            g.xop = p.op[OP_ACT]; g.N = p.d; g.Kd = p.F; g.need = p.parallel ? base + 2 : base + 6;
            g.out = p.x; g.ldo = p.d; g.bias = ltab ? ltab[8 * l + 7] : ld->b_out;
        }
    }
    g.n_tiles = (g.N + kTileNP - 1) / kTileNP;
    g.kchunks = (g.Kd + kTileK - 1) / kTileK;
    return g;
}

// This CTA's contiguous share of a GEMM's (tile, k-chunk) units.  Equal shares, except in the GEMM that
// follows the attention phase (MLP-out of a parallel-residual block, out-projection otherwise) when
// at most half of the CTAs ran an attention item: those enter the phase with only the lower ring
// slots filled ahead, the others with the whole ring, so they get that many units fewer.
__device__ __forceinline__ void unit_range(const FwdParams &p, const GemmDesc &g, int &c0, int &c1) {
    const long long total = (long long)g.n_tiles * g.kchunks;
    const int N = (int)gridDim.x, i = (int)blockIdx.x;
    const int A = attention_ctas(p), bonus = p.stages - p.stages_lo;
    if (overlap_mlp_out(p)) {  // MLP-out runs beside attention on the CTAs without an item; everything else in equal shares
        if (g.kind == 3 || g.kind == 1) {  // (the out-projection follows on the same CTAs: see attn_done)
            c0 = i < A ? 0 : (int)(total * (i - A) / (N - A));
            c1 = i < A ? 0 : (int)(total * (i - A + 1) / (N - A));
            return;
        }
        c0 = (int)(total * i / N);
        c1 = (int)(total * (i + 1) / N);
        return;
    }
    const bool after_attention = p.parallel ? g.kind == 3 : g.kind == 1;
    if (after_attention && 2 * A <= N && bonus > 0) {  // (with most CTAs on attention the few others would become the stragglers)
        long long xa = (total + (long long)A * bonus) / N - bonus;  // an attention CTA's share
        if (xa < 0) xa = 0;
        const long long rest = total - xa * A;                      // over the N - A others
        if (i < A) {
            c0 = (int)(xa * i);
            c1 = (int)(xa * (i + 1));
        } else {
            c0 = (int)(xa * A + rest * (i - A) / (N - A));
            c1 = (int)(xa * A + rest * (i - A + 1) / (N - A));
        }
        return;
    }
    c0 = (int)(total * i / N);
    c1 = (int)(total * (i + 1) / N);
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

// Tile row of the hi part of row r (the lo part is 8 further): rows come in blocks of 8, each block
// as 8 hi rows followed by 8 lo rows, so that an accumulator load hands both to one thread.
__device__ __forceinline__ int op_row(int r) { return 16 * (r >> 3) + (r & 7); }
// Element offset of (tile row, column i) in a tiled operand: tile row in [0, 2 rk).
__device__ __forceinline__ size_t op_off(int rk, int row, int i) {
    const int kc = i >> 6, w = i & 63;
    return (size_t)kc * (size_t)(2 * rk * kTileK) + (size_t)(row * kTileK + ((((w >> 3) ^ (row & 7)) << 3) | (w & 7)));
}
// operand element (r, i) as hi + lo
__device__ __forceinline__ void store_hilo(__nv_bfloat16 *buf, int rk, int r, int i, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    buf[op_off(rk, op_row(r), i)] = h;
    buf[op_off(rk, op_row(r) + 8, i)] = __float2bfloat16_rn(v - __bfloat162float(h));
}
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---- tcgen05 (5th-generation tensor core) helpers ---------------------------------------------
constexpr int kTmemCols = 512;  // two accumulator buffers of 256 fp32 columns each
constexpr int kAccStride = 256;
constexpr int kEpiWarps = 4;    // warps 0-3: one tensor-memory lane quadrant each
constexpr int kMmaWarp = 4;
constexpr int kEpiPitch = kTileNP + 8;             // floats per row of the epilogue tile (bank spread)
constexpr int kEpiBytes = 8 * kEpiPitch * 4 + 16 + 16 * 8 + 16 * 4 + 16 + 2 * 16 + 8 * 4 + 1024 + 512 + (8 * kMaxStagedLayers + 2) * 8;  // ... + parameter copy, staged tables  // 8 rows, the four warps' wait results, attention barriers
constexpr int kXWarp = 5;      // issues the operand copies of a GEMM phase

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// mbarrier arrive once every MMA issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (what the TMA copies write): start address / 16, leading byte offset unused (1),
// stride between 8-row groups 1024 bytes, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, A and B bf16, both K-major, M = m, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 lanes x 32 columns of the accumulator (the 16-lane x 256-bit shape, four times along the columns).
// Thread (g = lane / 4, t = lane % 4) receives, for column block k = 0..3: v[4k], v[4k+1] = lane g,
// columns 8k + 2t, 8k + 2t + 1 and v[4k+2], v[4k+3] = lane g + 8, the same columns.  The wait is part
// of the same statement so that no use of the results can be scheduled before it.
__device__ __forceinline__ void tc_ld_16x32(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// the same shape eight times along the columns: 16 lanes x 64 columns in one round trip
__device__ __forceinline__ void tc_ld_16x64(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void red_add_v4(float *dst, float4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}

// Slot schedule of the ring, identical in every role that walks it (weight producer, operand issuer,
// MMA issuer).  Unit j of this CTA's share of a GEMM takes the next slot of the full cycle, except
// the first stages_lo units of an out-projection - the ones fetched while the attention phase still
// owns the upper slots - which cycle through the lower slots only.  One parity bit per slot.
struct RingPos {
    int pos_all = 0, pos_lo = 0;
    uint32_t par = 0, used = 0;
};
__device__ __forceinline__ int ring_next(RingPos &r, bool lo_only, int S, int S1, uint32_t &parity) {
    int s;
    if (lo_only) { s = r.pos_lo; if (++r.pos_lo == S1) r.pos_lo = 0; }
    else { s = r.pos_all; if (++r.pos_all == S) r.pos_all = 0; }
    parity = (r.par >> s) & 1u;
    r.par ^= 1u << s;
    r.used |= 1u << s;
    return s;
}
__device__ __forceinline__ bool ring_lo_only(const GemmDesc &g, int j, int S1) { return g.kind == 1 && j < S1; }

struct alignas(16) Shared {
    volatile int released;  // grid barriers completed so far
    volatile int abort;     // some wait in this CTA gave up
    volatile int go;        // snapshot of !abort taken inside the grid barrier: uniform for all work threads
    int flag;
    long long wait_limit;   // cycles after which a wait that takes work gives up (the drain waits of the error path keep kWaitCycles)
    // for the tensor-core attention items (kept here so that they take no more arguments than the others):
    uint32_t tmem_base;     // base address of this CTA's tensor memory
    uint32_t attn_bar_off;  // byte offset from this block to the attention barriers, followed by their counts
    // small tables staged in shared memory (byte offsets from this block), so that the head of a phase does
    // not start with a trip to global memory:
    uint32_t seq_off;       // int len[64], then int rows[64]: committed length and rows of this pass, per sequence
    uint32_t ltab_off;      // const float *[8 n_layers + 2]: the layers' gain / bias pointers, then the final norm's; 0 = not staged
};
__device__ __forceinline__ const int *staged_len(const Shared *sh) {
    return reinterpret_cast<const int *>(reinterpret_cast<const uint8_t *>(sh) + sh->seq_off);
}
__device__ __forceinline__ const float *const *staged_ltab(const Shared *sh) {
    return sh->ltab_off ? reinterpret_cast<const float *const *>(reinterpret_cast<const uint8_t *>(sh) + sh->ltab_off) : nullptr;
}

// Bounded wait that also gives up as soon as another thread of the CTA has.
__device__ __forceinline__ bool mbar_wait_or_abort(uint64_t *bar, uint32_t parity, const Shared *sh) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (sh->abort || clock64() - t0 > sh->wait_limit) return false;
    }
    return true;
}

// The same as a pure poll (a suspended waiter wakes up late; used where a hand-off is on the critical path).
__device__ __forceinline__ bool mbar_spin_or_abort(uint64_t *bar, uint32_t parity, const Shared *sh) {
    if (mbar_test_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_test_wait(bar, parity)) {
        if (sh->abort || clock64() - t0 > sh->wait_limit) return false;
    }
    return true;
}

// Grid barrier for the 256 work threads of every CTA.  Returns false (the same value in every work
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
                    if (clock64() - t0 > sh->wait_limit) { ok = false; break; }
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

// Arrival at the next grid barrier without waiting for it (for a CTA whose next work does not depend on
// what the others publish there).  Its own writes are published like at a full barrier.
__device__ __forceinline__ void grid_arrive(const FwdParams &p, Shared *sh, int &epoch) {
    fence_async_proxy();
    __threadfence();
    named_bar(1, kWorkThreads);
    ++epoch;
    if (threadIdx.x == 0 && sh->abort == 0) red_release_add(p.gbar, 1u);
    if (p.trace && blockIdx.x == 0 && threadIdx.x == 0) {  // (the stamp of a barrier this CTA does not wait at: its arrival)
        unsigned long long t;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        p.trace[epoch] = t;
    }
}

// Count of attention CTAs that have finished their items, over the layers of this pass (zeroed with the
// barrier counter before the launch).  With few attention items in a parallel-residual block the CTAs
// without an item run the MLP-out GEMM beside the attention and go straight on to the out-projection:
// its operand issuer waits for this count instead of a grid barrier.
__device__ __forceinline__ unsigned *attn_done(const FwdParams &p) { return p.gbar + 8; }
__device__ __forceinline__ void attn_signal(const FwdParams &p, Shared *sh) {
    fence_async_proxy();  // the attention output is read by other CTAs' bulk copies
    __threadfence();
    named_bar(1, kWorkThreads);
    if (threadIdx.x == 0 && sh->abort == 0) red_release_add(attn_done(p), 1u);
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

// two sums in one exchange
__device__ __forceinline__ void block_sum2_work(double &a, double &b, double *red) {
    a = warp_sum(a);
    b = warp_sum(b);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    named_bar(2, kWorkThreads);
    if (lane == 0) { red[w] = a; red[kConsumerWarps + w] = b; }
    named_bar(2, kWorkThreads);
    double ta = 0.0, tb = 0.0;
#pragma unroll
    for (int i = 0; i < kConsumerWarps; ++i) { ta += red[i]; tb += red[kConsumerWarps + i]; }
    a = ta;
    b = tb;
}
__device__ __forceinline__ void prefetch_l1(const void *ptr) { asm volatile("prefetch.global.L1 [%0];" ::"l"(ptr)); }

// zero a [R, n] fp32 buffer (row pitch ld), spread over the whole grid
__device__ __forceinline__ void grid_zero(float *dst, int R, int n, int ld) {
    if (n == ld && ((R * (long long)n) & 3) == 0) {  // contiguous: 16-byte stores
        const long long total4 = (long long)R * n / 4;
        float4 *d4 = reinterpret_cast<float4 *>(dst);
        for (long long i = (long long)blockIdx.x * kWorkThreads + threadIdx.x; i < total4;
             i += (long long)gridDim.x * kWorkThreads)
            d4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const long long total = (long long)R * n;
    for (long long i = (long long)blockIdx.x * kWorkThreads + threadIdx.x; i < total;
         i += (long long)gridDim.x * kWorkThreads) {
        int r = (int)(i / n), c = (int)(i % n);
        dst[(size_t)r * ld + c] = 0.f;
    }
}

// Norm of every row of x into hi/lo operand buffers (one or two gain/bias sets from the same
// statistics); one CTA per row.  The row (Q float4 per thread) stays in registers between the
// statistics and the write pass, and all loads of a pass are issued before the first use, so the
// phase costs about two L2 round trips instead of one per element.  Q is a template parameter so
// that a call executes only the code its row width needs: the instructions of a phase are not in
// the instruction cache when it starts (the kernel is far larger than that cache), and every KB of
// straight-line code costs a fraction of a microsecond to fetch.
__device__ __forceinline__ void norm_emit(const FwdParams &p, int r, int i, const float4 v, float mu, float rs,
                                          const float *g, const float *b, int op) {
    const float4 gg = __ldg(reinterpret_cast<const float4 *>(g) + i);
    float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
    if (b) bb = __ldg(reinterpret_cast<const float4 *>(b) + i);
    const float y0 = (v.x - mu) * rs * gg.x + bb.x, y1 = (v.y - mu) * rs * gg.y + bb.y;
    const float y2 = (v.z - mu) * rs * gg.z + bb.z, y3 = (v.w - mu) * rs * gg.w + bb.w;
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(y0, y1), h23 = __floats2bfloat162_rn(y2, y3);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(y0 - __low2float(h01), y1 - __high2float(h01));
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(y2 - __low2float(h23), y3 - __high2float(h23));
    __nv_bfloat16 *hi = p.op[op] + op_off(p.rk, op_row(r), 4 * i);
    __nv_bfloat16 *lo = p.op[op] + op_off(p.rk, op_row(r) + 8, 4 * i);
    uint2 hv, lv;
    hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
    lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
    *reinterpret_cast<uint2 *>(hi) = hv;
    *reinterpret_cast<uint2 *>(lo) = lv;
}

template <int Q>  // float4 per thread held in registers: rows up to Q * 1024 wide; wider rows are re-read
__device__ __noinline__ void norm_rows(const FwdParams &p, const float *g1, const float *b1, int op1,
                                          const float *g2, const float *b2, int op2, double *red) {
    const int n4 = p.d >> 2;  // d is a multiple of 8
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const float4 *x4 = reinterpret_cast<const float4 *>(p.x + (size_t)r * p.d);
        float4 xv[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int i = threadIdx.x + q * kWorkThreads;
            xv[q] = i < n4 ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // the gain / bias vectors were last read a whole pass of weights ago: fetch them now, under the
        // statistics, instead of as a second trip to DRAM after them
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int i = threadIdx.x + q * kWorkThreads;
            if (i < n4) {
                prefetch_l1(reinterpret_cast<const float4 *>(g1) + i);
                if (b1) prefetch_l1(reinterpret_cast<const float4 *>(b1) + i);
                if (g2) prefetch_l1(reinterpret_cast<const float4 *>(g2) + i);
                if (b2) prefetch_l1(reinterpret_cast<const float4 *>(b2) + i);
            }
        }
        double s1 = 0.0, s2 = 0.0;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            s1 += (double)xv[q].x + (double)xv[q].y + (double)xv[q].z + (double)xv[q].w;
            s2 += (double)xv[q].x * xv[q].x + (double)xv[q].y * xv[q].y + (double)xv[q].z * xv[q].z + (double)xv[q].w * xv[q].w;
        }
#pragma unroll 1
        for (int i = threadIdx.x + Q * kWorkThreads; i < n4; i += kWorkThreads) {
            const float4 v = __ldcg(x4 + i);
            s1 += (double)v.x + (double)v.y + (double)v.z + (double)v.w;
            s2 += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
        }
        block_sum2_work(s1, s2, red);
        double mean = 0.0, var;
        if (p.norm_kind == 0) {
            mean = s1 * p.inv_d;
            var = s2 * p.inv_d - mean * mean;
            if (var < 0.0) var = 0.0;
        } else {
            var = s2 * p.inv_d;
        }
        const float mu = (float)mean, rs = (float)rsqrt(var + (double)p.eps);
#pragma unroll 1
        for (int e = 0; e < (g2 ? 2 : 1); ++e) {  // (rolled: the second gain set reuses the first one's code)
            const float *g = e ? g2 : g1, *b = e ? b2 : b1;
            const int op = e ? op2 : op1;
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const int i = threadIdx.x + q * kWorkThreads;
                if (i < n4) norm_emit(p, r, i, xv[q], mu, rs, g, b, op);
            }
#pragma unroll 1
            for (int i = threadIdx.x + Q * kWorkThreads; i < n4; i += kWorkThreads)
                norm_emit(p, r, i, __ldcg(x4 + i), mu, rs, g, b, op);
        }
    }
}

__device__ __noinline__ void norm_phase(const FwdParams &p, const float *g1, const float *b1, int op1,
                                           const float *g2, const float *b2, int op2, double *red) {
    const int n4 = p.d >> 2;
    if (n4 <= kWorkThreads) norm_rows<1>(p, g1, b1, op1, g2, b2, op2, red);
    else if (n4 <= 2 * kWorkThreads) norm_rows<2>(p, g1, b1, op1, g2, b2, op2, red);
    else if (n4 <= 4 * kWorkThreads) norm_rows<4>(p, g1, b1, op1, g2, b2, op2, red);
    else norm_rows<8>(p, g1, b1, op1, g2, b2, op2, red);
}

// MLP activation of t_in into the hi/lo operand of the down projection, spread over the grid
__device__ __noinline__ void act_phase(const FwdParams &p) {
    const int f4 = p.F >> 2;
    const long long total = (long long)p.R * f4;
    for (long long i = (long long)blockIdx.x * kWorkThreads + threadIdx.x; i < total;
         i += (long long)gridDim.x * kWorkThreads) {
        const int r = (int)(i / f4), c = (int)(i % f4);
        const float4 *t = reinterpret_cast<const float4 *>(p.t_in + (size_t)r * p.d_in);
        const float4 a = __ldcg(t + c);
        float y0, y1, y2, y3;
        if (p.swiglu) {
            const float4 u = __ldcg(t + f4 + c);
            y0 = silu(a.x) * u.x; y1 = silu(a.y) * u.y; y2 = silu(a.z) * u.z; y3 = silu(a.w) * u.w;
        } else {
            y0 = gelu_erf(a.x); y1 = gelu_erf(a.y); y2 = gelu_erf(a.z); y3 = gelu_erf(a.w);
        }
        const __nv_bfloat162 h01 = __floats2bfloat162_rn(y0, y1), h23 = __floats2bfloat162_rn(y2, y3);
        const __nv_bfloat162 l01 = __floats2bfloat162_rn(y0 - __low2float(h01), y1 - __high2float(h01));
        const __nv_bfloat162 l23 = __floats2bfloat162_rn(y2 - __low2float(h23), y3 - __high2float(h23));
        uint2 hv, lv;
        hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
        lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
        __nv_bfloat16 *base = p.op[OP_ACT];
        *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r), 4 * c)) = hv;
        *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r) + 8, 4 * c)) = lv;
    }
}

__device__ __noinline__ void setup_phase(const FwdParams &p) {
    // K not a multiple of 64: the last tile's unused columns must be finite (the weight copy zero-fills its own)
    for (int o = 0; o < 4; ++o) {
        const int K = p.op_ld[o], pad = (-K) & (kTileK - 1);
        if (!p.op[o] || !pad) continue;
        for (int e = blockIdx.x * kWorkThreads + threadIdx.x; e < 2 * p.rk * pad; e += gridDim.x * kWorkThreads)
            p.op[o][op_off(p.rk, e / pad, K + e % pad)] = __float2bfloat16_rn(0.f);
    }
    const int half = p.rotary_dim / 2;
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const int b = r / p.M, j = r % p.M;
        int n = p.cur_step > 0 ? 1 : (p.n_rows ? p.n_rows[b] : p.M);
        n = max(0, min(n, p.M));
        const int len = __ldcg(p.len + b);  // (advanced between the steps of a draft loop)
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

__device__ __noinline__ void embed_phase(const FwdParams &p) {
    for (int r = blockIdx.x; r < p.R; r += gridDim.x) {
        const int b = r / p.M, j = r % p.M;
        int tok = 0;
        if (__ldcg(p.ri.valid + r))
            tok = p.cur_step > 0 ? __ldcg(p.tok_out + (size_t)b * p.tok_out_stride + p.cur_step - 1) : p.tokens[(size_t)b * p.tok_stride + j];
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

// ---- attention ---------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void *dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t &r0, uint32_t &r1) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

// Columns e0 .. e0+7 of one head's q or k row (fp32, `row` points at the head's first column) with
// the rotary turn of row r applied; rotary_dim and its half are multiples of 8, so the eight
// columns fall on one side of the split.  All loads are issued before the first use.
__device__ __forceinline__ void rope_vec8(const FwdParams &p, const float *row, int r, int e0, float (&out)[8]) {
    const float4 a0 = __ldcg(reinterpret_cast<const float4 *>(row + e0)), a1 = __ldcg(reinterpret_cast<const float4 *>(row + e0 + 4));
    out[0] = a0.x; out[1] = a0.y; out[2] = a0.z; out[3] = a0.w; out[4] = a1.x; out[5] = a1.y; out[6] = a1.z; out[7] = a1.w;
    if (e0 < p.rotary_dim) {
        const int half = p.rotary_dim >> 1;
        const bool low = e0 < half;
        const int j0 = low ? e0 : e0 - half;
        const float *pr_ = row + (low ? e0 + half : e0 - half);
        const float4 b0 = __ldcg(reinterpret_cast<const float4 *>(pr_)), b1 = __ldcg(reinterpret_cast<const float4 *>(pr_ + 4));
        const float *cp = p.ri.rope_cos + (size_t)r * half + j0, *sp = p.ri.rope_sin + (size_t)r * half + j0;
        const float4 c0 = __ldcg(reinterpret_cast<const float4 *>(cp)), c1 = __ldcg(reinterpret_cast<const float4 *>(cp + 4));
        const float4 s0 = __ldcg(reinterpret_cast<const float4 *>(sp)), s1 = __ldcg(reinterpret_cast<const float4 *>(sp + 4));
        const float pb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        const float cc[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        const float ss[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
        for (int u = 0; u < 8; ++u) out[u] = low ? out[u] * cc[u] - pb[u] * ss[u] : pb[u] * ss[u] + out[u] * cc[u];
    }
}

// four output columns of one row of the out-projection operand, as bf16 hi + lo
__device__ __forceinline__ void store_ao4(const FwdParams &p, int r, int col, float4 y) {
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(y.x, y.y), h23 = __floats2bfloat162_rn(y.z, y.w);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(y.x - __low2float(h01), y.y - __high2float(h01));
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(y.z - __low2float(h23), y.w - __high2float(h23));
    uint2 hv, lv;
    hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
    lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
    __nv_bfloat16 *base = p.op[OP_AO];
    *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r), col)) = hv;
    *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r) + 8, col)) = lv;
}

// The item that finishes last for a (sequence, head) merges the splits' partials (m, l, o) of all its
// rows into the out-projection operand; 256 threads.
__device__ __forceinline__ void merge_splits(const FwdParams &p, int r0, int h, int Dh) {
    const int tid = threadIdx.x, q4 = Dh >> 2;
    auto store_ao4 = [&](int r, int col, float4 y) { ssd::store_ao4(p, r, col, y); };
            // one work item = four columns of one row; the loads of up to eight splits are issued together
            for (int idx = tid; idx < p.M * q4; idx += kAttnThreadsP) {
                const int m = idx / q4, e = (idx % q4) * 4;
                const size_t base = ((size_t)(r0 + m) * p.H + h) * p.n_split;
                float mx = -INFINITY, L = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int s0 = 0; s0 < p.n_split; s0 += 8) {
                    float pm[8], pl[8];
                    float4 po[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const bool in = s0 + u < p.n_split;
                        pm[u] = in ? __ldcg(p.part_m + base + s0 + u) : -INFINITY;
                        pl[u] = in ? __ldcg(p.part_l + base + s0 + u) : 0.f;
                        po[u] = in ? __ldcg(reinterpret_cast<const float4 *>(p.part_o + (base + s0 + u) * Dh + e))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    float bm = mx;
#pragma unroll
                    for (int u = 0; u < 8; ++u) bm = fmaxf(bm, pm[u]);
                    if (bm == -INFINITY) continue;
                    const float f = exp2f(mx - bm);  // 0 while nothing has been accumulated
                    L *= f; acc.x *= f; acc.y *= f; acc.z *= f; acc.w *= f;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (pm[u] == -INFINITY) continue;
                        const float w = exp2f(pm[u] - bm);
                        L = fmaf(pl[u], w, L);
                        acc.x = fmaf(po[u].x, w, acc.x); acc.y = fmaf(po[u].y, w, acc.y);
                        acc.z = fmaf(po[u].z, w, acc.z); acc.w = fmaf(po[u].w, w, acc.w);
                    }
                    mx = bm;
                }
                const float inv = L > 0.f ? 1.f / L : 0.f;
                store_ao4(r0 + m, h * Dh + e, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
            }
}

// Positions per split of a sequence that holds `total` positions after this pass: equal shares of whole
// tiles, taken on the device from the sequence's own length.  The host fixes only the number of splits
// (from an upper bound of the lengths), so ragged sequences are each cut evenly and a loose bound costs
// nothing but an empty split.
__device__ __forceinline__ int split_chunk(const FwdParams &p, int total, int tile) {
    const int c = (max(total, 1) + p.n_split - 1) / p.n_split;
    return (c + tile - 1) / tile * tile;
}

constexpr int kAttnRows = 16;  // query rows per item (one MMA row tile)
constexpr int kAttnBufs = 3;   // K/V chunk buffers: two chunks (64 KB at head 128) in flight per SM
__host__ __device__ inline size_t attn_scratch_bytes(int Dh) {
    // Q hi/lo [16][Dh+8] bf16, kAttnBufs K/V chunk buffers [2][64][Dh+8] bf16 each, per-warp (m, l) [8][16] fp32 x 2,
    // per-thread partial scores [256][8] fp32
    return (size_t)2 * kAttnRows * (Dh + 8) * 2 + (size_t)kAttnBufs * 2 * kAttnTile * (Dh + 8) * 2 + 2 * 8 * kAttnRows * 4 +
           (size_t)256 * 8 * 4;
}

// Attention of up to 16 query rows of one (sequence, head) over one split of the position axis, by
// 256 threads, on tensor cores.  K/V chunks of 64 positions are fetched with cp.async into three
// buffers (the next two chunks load while this one is used).  Warp w owns positions 16 (w & 3) .. +15
// of each chunk and the output columns of half (w >> 2) of the head.  The two warps of a position
// group each contract half of the head dimension of the 16 x 16 score block S = Q K^T (Q as bf16
// hi + lo) and exchange the halves, so both hold S; each keeps its own running max / sum (equal in
// both, the sum of two halves being order-independent) and adds P V (P as bf16
// hi + lo) to its 16 x Dh/2 accumulators -- no exchange between warps until the end, where the
// four position groups are merged in shared memory.  Rows of this pass (positions >= len) take
// their keys / values from qkv (rotary, cache rounding) and the split that owns them appends them
// to the cache.  With one split the result goes straight to the out-projection operand; otherwise
// partials are written and the split that finishes last merges them.  All exponentials are base 2.
__device__ __noinline__ void attention_item(const FwdParams &p, int layer, int item, uint8_t *scratch, Shared *sh) {
    const int MT = (p.M + kAttnRows - 1) / kAttnRows;
    const int mt = item % MT, rest = item / MT;
    const int split = rest % p.n_split, bh = rest / p.n_split, b = bh / p.H, h = bh % p.H;
    const int Dh = p.Dh, d = p.d, pitch = Dh + 8;
    const uint32_t pitchB = (uint32_t)pitch * 2u;
    __nv_bfloat16 *Qhi = reinterpret_cast<__nv_bfloat16 *>(scratch);
    __nv_bfloat16 *Qlo = Qhi + kAttnRows * pitch;
    __nv_bfloat16 *KV = Qlo + kAttnRows * pitch;  // buffer i: K at KV + i * 2 * 64 * pitch, V 64 * pitch later
    float *mw = reinterpret_cast<float *>(KV + kAttnBufs * 2 * kAttnTile * pitch);
    float *lw = mw + 8 * kAttnRows;
    float *sx = lw + 8 * kAttnRows;  // score halves exchanged between the two warps of a position group
    float *o_acc = reinterpret_cast<float *>(KV);  // [4][16][Dh] fp32, reuses the chunk buffers after the loop

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int pg = warp & 3, dhh = warp >> 2;
    const int nk = Dh >> 4;          // k-steps of Q K^T; also 8-column output tiles per head half
    const int dh0 = dhh * (Dh >> 1);
    const int n_rows = staged_len(sh)[64 + b];
    const int len = staged_len(sh)[b];
    const int r0 = b * p.M, m_base = mt * kAttnRows;
    const int chunk = split_chunk(p, len + n_rows, kAttnTile);
    const int p_begin = split * chunk;
    const int p_end = min(p_begin + chunk, len + n_rows);
    const float sc = p.attn_scale * 1.4426950408889634f;  // scores in log2 units

    __nv_bfloat16 *kc = (__nv_bfloat16 *)(p.cache + (size_t)layer * p.layer_bytes) + ((size_t)(b * 2) * p.H + h) * p.S * Dh;
    __nv_bfloat16 *vc = kc + (size_t)p.H * p.S * Dh;
    const int vpr = Dh >> 3;  // 16-byte vectors per row
    auto load_chunk = [&](int c) {
        __nv_bfloat16 *Kb = KV + (size_t)(c % kAttnBufs) * 2 * kAttnTile * pitch, *Vb = Kb + kAttnTile * pitch;
        const int t0 = p_begin + c * kAttnTile, np = min(kAttnTile, p_end - t0);
        const int prow = tid >> 4, v8 = tid & 15;  // 16 threads per row, 16 rows per pass
        if (v8 < vpr) {
            if (t0 + kAttnTile <= len) {  // the common case: all 64 positions come from the cache
                const __nv_bfloat16 *ks = kc + (size_t)(t0 + prow) * Dh + v8 * 8, *vs = vc + (size_t)(t0 + prow) * Dh + v8 * 8;
                __nv_bfloat16 *dk = Kb + prow * pitch + v8 * 8, *dv = Vb + prow * pitch + v8 * 8;
#pragma unroll
                for (int q = 0; q < kAttnTile / 16; ++q) {
                    cp_async16(dk + q * 16 * pitch, ks + (size_t)q * 16 * Dh);
                    cp_async16(dv + q * 16 * pitch, vs + (size_t)q * 16 * Dh);
                }
            } else {
#pragma unroll 1
                for (int q = 0; q < kAttnTile / 16; ++q) {
                    const int pp = prow + 16 * q, pos = t0 + pp;
                    __nv_bfloat16 *dk = Kb + pp * pitch + v8 * 8, *dv = Vb + pp * pitch + v8 * 8;
                    if (pp >= np) {  // beyond the split: zeros (P is 0 there, but 0 * garbage must not be NaN)
                        *reinterpret_cast<uint4 *>(dk) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(dv) = make_uint4(0, 0, 0, 0);
                    } else if (pos < len) {
                        const size_t go = (size_t)pos * Dh + v8 * 8;
                        cp_async16(dk, kc + go);
                        cp_async16(dv, vc + go);
                    } else {  // a row of this pass: from qkv, position-encoded and rounded as the cache stores it
                        const int r = r0 + (pos - len);
                        const float *krow = p.qkv + (size_t)r * 3 * d + d + h * Dh;
                        float kf[8];
                        rope_vec8(p, krow, r, v8 * 8, kf);
                        const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(krow + d + v8 * 8));
                        const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(krow + d + v8 * 8 + 4));
                        const float vf[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                        __nv_bfloat16 kb[8], vb[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            kb[u] = __float2bfloat16_rn(kf[u]);
                            vb[u] = __float2bfloat16_rn(vf[u]);
                        }
                        const uint4 kq = *reinterpret_cast<uint4 *>(kb), vq = *reinterpret_cast<uint4 *>(vb);
                        *reinterpret_cast<uint4 *>(dk) = kq;
                        *reinterpret_cast<uint4 *>(dv) = vq;
                        if (mt == 0) {  // append: exactly one split owns this position
                            const size_t go = (size_t)pos * Dh + v8 * 8;
                            *reinterpret_cast<uint4 *>(kc + go) = kq;
                            *reinterpret_cast<uint4 *>(vc + go) = vq;
                        }
                    }
                }
            }
        }
        cp_async_commit();
    };

    float o[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int n_chunks = p_begin < p_end ? (p_end - p_begin + kAttnTile - 1) / kAttnTile : 0;

    // kAttnBufs - 1 chunks are always in flight; one group is committed per chunk slot so that
    // "at most kAttnBufs - 1 groups pending" means "chunk c has landed"
    for (int c = 0; c < kAttnBufs - 1; ++c) {
        if (c < n_chunks) load_chunk(c); else cp_async_commit();
    }
    // ---- Q rows (rotary applied) as bf16 hi / lo: thread = (row, 8 columns) ----
    {
        const int ml = tid >> 4, v8 = tid & 15, m = m_base + ml;
        if (v8 < vpr) {
            float q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) q[u] = 0.f;
            if (m < n_rows) rope_vec8(p, p.qkv + (size_t)(r0 + m) * 3 * d + h * Dh, r0 + m, v8 * 8, q);
            __nv_bfloat16 hq[8], lq[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                hq[u] = __float2bfloat16_rn(q[u]);
                lq[u] = __float2bfloat16_rn(q[u] - __bfloat162float(hq[u]));
            }
            *reinterpret_cast<uint4 *>(Qhi + ml * pitch + v8 * 8) = *reinterpret_cast<uint4 *>(hq);
            *reinterpret_cast<uint4 *>(Qlo + ml * pitch + v8 * 8) = *reinterpret_cast<uint4 *>(lq);
        }
    }
    for (int c = 0; c < n_chunks; ++c) {
        if (c + kAttnBufs - 1 < n_chunks) load_chunk(c + kAttnBufs - 1); else cp_async_commit();
        cp_async_wait<kAttnBufs - 1>();
        named_bar(3, kAttnThreadsP);  // chunk c (and, first time, Q) is in shared memory
        const __nv_bfloat16 *Kb = KV + (size_t)(c % kAttnBufs) * 2 * kAttnTile * pitch, *Vb = Kb + kAttnTile * pitch;
        const int pos0 = p_begin + c * kAttnTile + 16 * pg;  // this warp's 16 positions
        // ---- S = Q K^T for 16 rows x 16 positions; four independent accumulator sets (Q hi / lo x
        //      even / odd k-step) keep the dependent MMA chains short ----
        float s[2][4];
        {
            float sa[2][2][2][4];  // [hi|lo][even|odd][position tile][4]
#pragma unroll
            for (int x = 0; x < 2; ++x)
#pragma unroll
                for (int y = 0; y < 2; ++y)
#pragma unroll
                    for (int j = 0; j < 2; ++j) sa[x][y][j][0] = sa[x][y][j][1] = sa[x][y][j][2] = sa[x][y][j][3] = 0.f;
            const uint32_t qa = smem_u32(Qhi) + (uint32_t)(lane & 15) * pitchB + (uint32_t)(lane >> 4) * 16u;
            const uint32_t ql = qa + (uint32_t)kAttnRows * pitchB;
            const uint32_t ka = smem_u32(Kb) + (uint32_t)(16 * pg + (lane & 7) + 8 * (lane >> 4)) * pitchB + (uint32_t)((lane >> 3) & 1) * 16u;
            const int ks_lo = dhh ? (nk + 1) / 2 : 0, ks_hi = dhh ? nk : (nk + 1) / 2;  // this warp's half of Dh
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                if (ks >= ks_lo && ks < ks_hi) {
                    uint32_t a0, a1, a2, a3, c0, c1, c2, c3, k0, k1, k2, k3;
                    ldmatrix_x4(qa + ks * 32, a0, a1, a2, a3);
                    ldmatrix_x4(ql + ks * 32, c0, c1, c2, c3);
                    ldmatrix_x4(ka + ks * 32, k0, k1, k2, k3);  // (pos 0-7: k lo, k hi), (pos 8-15: k lo, k hi)
                    mma_bf16(sa[0][ks & 1][0], a0, a1, a2, a3, k0, k1);
                    mma_bf16(sa[1][ks & 1][0], c0, c1, c2, c3, k0, k1);
                    mma_bf16(sa[0][ks & 1][1], a0, a1, a2, a3, k2, k3);
                    mma_bf16(sa[1][ks & 1][1], c0, c1, c2, c3, k2, k3);
                }
            }
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) s[j][e] = (sa[0][0][j][e] + sa[0][1][j][e]) + (sa[1][0][j][e] + sa[1][1][j][e]);
            // exchange with the warp that holds the other half (same position group, same lane = same elements)
            float4 *mine = reinterpret_cast<float4 *>(sx + (size_t)tid * 8);
            mine[0] = make_float4(s[0][0], s[0][1], s[0][2], s[0][3]);
            mine[1] = make_float4(s[1][0], s[1][1], s[1][2], s[1][3]);
            named_bar(8 + pg, 64);
            const float4 *other = reinterpret_cast<const float4 *>(sx + (size_t)(tid ^ 128) * 8);
            const float4 o0 = other[0], o1 = other[1];
            s[0][0] += o0.x; s[0][1] += o0.y; s[0][2] += o0.z; s[0][3] += o0.w;
            s[1][0] += o1.x; s[1][1] += o1.y; s[1][2] += o1.z; s[1][3] += o1.w;
        }
        // ---- mask, running max / sum (rows g and g + 8) ----
        float pr[2][4];
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
            const int m = m_base + g + 8 * hrow;
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int pos = pos0 + 8 * j + 2 * t + e;
                    const bool vis = pos < p_end && pos <= len + m;
                    const float v = vis ? s[j][2 * hrow + e] * sc : -INFINITY;
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
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float pv = exp2f(s[j][2 * hrow + e] - m_new);
                        pr[j][2 * hrow + e] = pv;
                        sum += pv;
                    }
            } else {
#pragma unroll
                for (int j = 0; j < 2; ++j) pr[j][2 * hrow] = pr[j][2 * hrow + 1] = 0.f;
            }
            m_run[hrow] = m_new;
            l_run[hrow] = l_run[hrow] * f + sum;  // this thread's share; lanes are summed at the end
#pragma unroll
            for (int j = 0; j < 8; ++j) { o[j][2 * hrow] *= f; o[j][2 * hrow + 1] *= f; }
        }
        // ---- O += P V  (P as hi + lo; k = the 16 positions; n = this warp's Dh/2 columns) ----
        {
            uint32_t ph[4], pl[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {  // a0: (row g, k 2t..) a1: (row g+8, ..) a2: (row g, k 8+2t..) a3: (row g+8, ..)
                const int j = q >> 1, hrow = q & 1;
                const float x0 = pr[j][2 * hrow], x1 = pr[j][2 * hrow + 1];
                const __nv_bfloat162 hv = __floats2bfloat162_rn(x0, x1);
                ph[q] = *reinterpret_cast<const uint32_t *>(&hv);
                pl[q] = pack_bf16x2(x0 - __low2float(hv), x1 - __high2float(hv));
            }
            const uint32_t va = smem_u32(Vb) + (uint32_t)(16 * pg + (lane & 15)) * pitchB + (uint32_t)dh0 * 2u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < nk) {
                    uint32_t b0, b1;
                    ldmatrix_x2_trans(va + j * 16, b0, b1);
                    mma_bf16(o[j], ph[0], ph[1], ph[2], ph[3], b0, b1);
                    mma_bf16(o[j], pl[0], pl[1], pl[2], pl[3], b0, b1);
                }
            }
        }
        named_bar(3, kAttnThreadsP);  // everyone is done with this buffer before it is refilled
    }
    if (n_chunks == 0) named_bar(3, kAttnThreadsP);  // Q stores vs. later reuse of the scratch

    // ---- merge the four position groups ----
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
        l_run[hrow] += __shfl_xor_sync(0xffffffffu, l_run[hrow], 1);
        l_run[hrow] += __shfl_xor_sync(0xffffffffu, l_run[hrow], 2);
    }
    if (t == 0) {
        mw[warp * kAttnRows + g] = m_run[0];
        mw[warp * kAttnRows + g + 8] = m_run[1];
        lw[warp * kAttnRows + g] = l_run[0];
        lw[warp * kAttnRows + g + 8] = l_run[1];
    }
    named_bar(3, kAttnThreadsP);
    // every warp scales its block to the common maximum and stores it: o_part[pg][16][Dh] (fp32, in the
    // chunk buffers, free now); the output loop adds the four position groups in a fixed order
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
        const int row = g + 8 * hrow;
        float mx = -INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q) mx = fmaxf(mx, mw[q * kAttnRows + row]);
        const float f = (m_run[hrow] > -INFINITY) ? exp2f(m_run[hrow] - mx) : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < nk) {
                float2 v2 = make_float2(o[j][2 * hrow] * f, o[j][2 * hrow + 1] * f);
                *reinterpret_cast<float2 *>(o_acc + ((size_t)pg * kAttnRows + row) * Dh + dh0 + 8 * j + 2 * t) = v2;
            }
        }
    }
    named_bar(3, kAttnThreadsP);
    const bool direct = p.n_split == 1;
    // four output columns of one real row per work item
    auto store_ao4 = [&](int r, int col, float4 y) {
        const __nv_bfloat162 h01 = __floats2bfloat162_rn(y.x, y.y), h23 = __floats2bfloat162_rn(y.z, y.w);
        const __nv_bfloat162 l01 = __floats2bfloat162_rn(y.x - __low2float(h01), y.y - __high2float(h01));
        const __nv_bfloat162 l23 = __floats2bfloat162_rn(y.z - __low2float(h23), y.w - __high2float(h23));
        uint2 hv, lv;
        hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
        lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
        __nv_bfloat16 *base = p.op[OP_AO];
        *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r), col)) = hv;
        *reinterpret_cast<uint2 *>(base + op_off(p.rk, op_row(r) + 8, col)) = lv;
    };
    const int q4 = Dh >> 2;  // float4 per row
    const int rows_here = max(0, min(kAttnRows, p.M - m_base));
    for (int i = tid; i < rows_here * q4; i += kAttnThreadsP) {
        const int ml = i / q4, e = (i % q4) * 4, m = m_base + ml;
        float mx = -INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q) mx = fmaxf(mx, mw[q * kAttnRows + ml]);
        float L = 0.f;
        if (mx > -INFINITY) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float mq = mw[q * kAttnRows + ml];
                if (mq > -INFINITY) L += lw[q * kAttnRows + ml] * exp2f(mq - mx);
            }
        }
        const bool live = m < n_rows && L > 0.f;
        const int gs = kAttnRows * Dh;  // stride between position groups
        const float *oa = o_acc + ml * Dh + e;
        const float4 a0 = *reinterpret_cast<const float4 *>(oa), a1 = *reinterpret_cast<const float4 *>(oa + gs);
        const float4 a2 = *reinterpret_cast<const float4 *>(oa + 2 * gs), a3 = *reinterpret_cast<const float4 *>(oa + 3 * gs);
        float4 osum = make_float4((a0.x + a1.x) + (a2.x + a3.x), (a0.y + a1.y) + (a2.y + a3.y),
                                  (a0.z + a1.z) + (a2.z + a3.z), (a0.w + a1.w) + (a2.w + a3.w));
        if (!live) osum = make_float4(0.f, 0.f, 0.f, 0.f);
        if (direct) {
            const float inv = live ? 1.f / L : 0.f;
            store_ao4(r0 + m, h * Dh + e, make_float4(osum.x * inv, osum.y * inv, osum.z * inv, osum.w * inv));
        } else {
            const size_t slot = ((size_t)(r0 + m) * p.H + h) * p.n_split + split;
            if (e == 0) {
                p.part_m[slot] = live ? mx : -INFINITY;
                p.part_l[slot] = live ? L : 0.f;
            }
            *reinterpret_cast<float4 *>(p.part_o + slot * Dh + e) = osum;
        }
    }
    if (!direct) {
        // ticket: the item that finishes last for this (sequence, head) merges all partials
        __threadfence();
        named_bar(3, kAttnThreadsP);
        if (tid == 0) sh->flag = (atomicAdd(p.tickets + bh, 1u) == (unsigned)(p.n_split * MT - 1));
        named_bar(3, kAttnThreadsP);
        if (sh->flag) {
            __threadfence();
            merge_splits(p, r0, h, Dh);
            if (tid == 0) p.tickets[bh] = 0;  // ready for the next layer (a grid barrier lies between)
        }
    }
    named_bar(3, kAttnThreadsP);  // scratch is free for the next item
}

__device__ __forceinline__ void cp_async16_zfill(void *dst, const void *src, bool valid) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(valid ? 16 : 0) : "memory");
}

#include "attn_mma8.cuh"

// ---- attention on tcgen05 (head dim 128) ----------------------------------------------------------
// The same item as attention_item - up to 16 query rows of one (sequence, head) over one split of the
// position axis - with the two products on the 5th-generation tensor core and the scores and the
// output in tensor memory, 128 positions per chunk:
//   S^T [128 positions x 32]  = K chunk (the M = 128 operand, straight from the TMA copy of the cache)
//                               x Q rows (16 hi + 16 lo, the N = 32 operand)
//   O^T [128 head dims x 32] += V chunk read as its transpose (MN-major M = 128 operand) x P (16 hi + 16 lo)
// Roles: threads 0-127 = one position each (softmax: masks, running max shared through shared memory,
// P as bf16 hi + lo into the P tile, rescale of O^T when a maximum moved) and, at the end, one head
// dim each (output); warp 4: MMA issue; warp 5: TMA copies of K and V chunks into a 4-stage ring;
// warps 6-7: rows of this pass (positions >= len) - rotary, rounding, append to the cache - written
// into the chunk tiles over what the copy brought.  Positions behind them are masked (P = 0) and
// multiply whatever the cache holds there: kv_init zeroes the cache, and all later writes are
// finite rows of earlier passes, so 0 x stale is 0.  Per chunk 8 + 8 MMA steps of ~120 cycles against 1.5 us of HBM time for its
// 64 KB: the chunk loop is bandwidth-bound instead of a latency chain.
constexpr int kTcChunk = 128;
constexpr int kTcStages = 4;  // K / V ring stages of 32 KB: the bytes in flight set the chunk rate (3 stages: 2.7 us per chunk)
constexpr int kTcKvStage = kTcChunk * 128 * 2;  // one K or V chunk: two 64-column panels of 128 rows x 128 B
constexpr int kTcPBytes = 8192;  // one P tile (16 hi + 16 lo rows x 128 positions, bf16); two of them, used in turn
constexpr int kTcQOff = kTcStages * kTcKvStage, kTcPOff = kTcQOff + 8192, kTcMiscOff = kTcPOff + 2 * kTcPBytes;
constexpr int kTcScratchBytes = kTcMiscOff + 1536 + kAttnRows * 128 * 4;  // + per-thread running sums [16][128]
// Its mbarriers live outside the scratch (which the weight ring reuses), are initialised once per kernel
// and keep running: cnt[i] = phases barrier i has completed before the current item.  A parity wait is
// only meaningful for a waiter that follows every phase of its barrier in order and that the barrier
// cannot pass by two phases; the threads that patch this pass's rows into a chunk skip most chunks, so
// they do not wait on the ring's barriers: the MMA issuer, which follows every stage, tells them through
// `landed` when such a chunk has arrived, and hears back through `fixed`.
enum { AB_KV_FULL = 0, AB_KV_FREE = kTcStages, AB_S_FULL = 2 * kTcStages, AB_P_READY = AB_S_FULL + 2, AB_O_DONE /* two: chunk parity */,
       AB_FIXED = AB_O_DONE + 2, AB_LANDED, AB_COUNT };
// The running maximum of a row is only raised when a chunk's maximum exceeds it by more than this (log2 units):
// P then stays below 2^8, the sums and O^T absorb it, and the dependent rescale of O^T - which has to wait for the
// previous chunk's P V - becomes rare instead of happening in every other chunk.
constexpr float kTcMaxSlack = 8.f;

__device__ __forceinline__ void tc_ld_32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// eight columns from each of two places of this warp's lane quadrant, one round trip
__device__ __forceinline__ void tc_ld_2x8(uint32_t ta, uint32_t tb, float (&a)[8], float (&b)[8]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%16];\n"
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%8,%9,%10,%11,%12,%13,%14,%15}, [%17];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(ta), "r"(tb)
        : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) { a[i] = __uint_as_float(r[i]); b[i] = __uint_as_float(r[8 + i]); }
}
// one column from each of two places of this warp's lane quadrant
__device__ __forceinline__ void tc_ld_2(uint32_t ta, uint32_t tb, float &a, float &b) {
    uint32_t x, y;
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%2];\n"
        "tcgen05.ld.sync.aligned.32x32b.x1.b32 {%1}, [%3];\n"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(x), "=r"(y)
        : "r"(ta), "r"(tb)
        : "memory");
    a = __uint_as_float(x);
    b = __uint_as_float(y);
}
__device__ __forceinline__ void tc_st_32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
        "tcgen05.wait::st.sync.aligned;\n" ::"r"(taddr),
        "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
// shared-memory matrix descriptor, 128-byte swizzle, explicit leading / stride byte offsets
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// byte offset of (row, 16-byte chunk c) in a tile of 128-byte rows with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int row, int c) { return (uint32_t)(row * 128 + ((c ^ (row & 7)) << 4)); }

__device__ __noinline__ void attention_item_tc(const FwdParams &p, int layer, int item, uint8_t *scratch, Shared *sh) {
    const uint32_t tmem_base = sh->tmem_base;
    uint64_t *abar = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(sh) + sh->attn_bar_off);
    uint32_t *acnt = reinterpret_cast<uint32_t *>(abar + AB_COUNT);
    constexpr int Dh = 128;
    const int MT = (p.M + kAttnRows - 1) / kAttnRows;
    const int mt = item % MT, rest = item / MT;
    const int split = rest % p.n_split, bh = rest / p.n_split, b = bh / p.H, h = bh % p.H;
    const int d = p.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint8_t *ring = scratch, *qt = scratch + kTcQOff, *pt = scratch + kTcPOff;
    // [2][4][16] chunk maxima per warp: scores are one chunk ahead, so a fast warp may already write the next
    // chunk's maxima while a slow one still reads this chunk's
    float *wmax2 = reinterpret_cast<float *>(scratch + kTcMiscOff);
    float *wsum = wmax2 + 128;                                      // [4][16]
    float *wmrun = wsum + 64;                                       // [4][16] running maxima, one copy per warp
    float *fsh = wmrun + 64;                                        // [4][16] this chunk's rescale factors
    float *l_sh = fsh + 64;                                         // [16][128] running sums, one per (row, thread)
    uint64_t *kv_full = abar + AB_KV_FULL, *kv_free = abar + AB_KV_FREE;  // [kTcStages] each
    uint64_t *s_full = abar + AB_S_FULL;  // [2]: the scores are double-buffered in tensor memory
    uint64_t *p_ready = abar + AB_P_READY, *o_done = abar + AB_O_DONE, *fixed = abar + AB_FIXED, *landed = abar + AB_LANDED;

    const int n_rows = staged_len(sh)[64 + b];
    const int len = staged_len(sh)[b];
    const int r0 = b * p.M, m_base = mt * kAttnRows;
    const int rows_here = max(0, min(kAttnRows, p.M - m_base));
    const int chunk = split_chunk(p, len + n_rows, kTcChunk);
    const int p_begin = split * chunk;
    const int p_end = min(p_begin + chunk, len + n_rows);
    const int n_chunks = p_begin < p_end ? (p_end - p_begin + kTcChunk - 1) / kTcChunk : 0;
    const float sc = p.attn_scale * 1.4426950408889634f;  // scores in log2 units
    const uint32_t tS = tmem_base, tO = tmem_base + 64;  // scores of chunk c at tS + 32 (c & 1)
    __nv_bfloat16 *kc = (__nv_bfloat16 *)(p.cache + (size_t)layer * p.layer_bytes) + ((size_t)(b * 2) * p.H + h) * p.S * Dh;
    __nv_bfloat16 *vc = kc + (size_t)p.H * p.S * Dh;
    const int krow0 = layer * p.kv_rows_per_layer + ((b * 2) * p.H + h) * p.S, vrow0 = krow0 + p.H * p.S;

    // a wait that keeps the control flow of every role intact: once anything has timed out, waits fall through
    auto wait = [&](uint64_t *bar, uint32_t parity) {
        if (sh->abort) return;
        if (!mbar_spin_or_abort(bar, parity, sh)) {
            set_status(p.status, kTimeoutCode);
            sh->abort = 1;
        }
    };

    // phases completed before this item (written by thread 0 at the end of the previous item, behind a barrier)
    uint32_t c_full[kTcStages], c_free[kTcStages];
#pragma unroll
    for (int i = 0; i < kTcStages; ++i) { c_full[i] = acnt[AB_KV_FULL + i]; c_free[i] = acnt[AB_KV_FREE + i]; }
    const uint32_t c_s0 = acnt[AB_S_FULL], c_s1 = acnt[AB_S_FULL + 1];
    const uint32_t c_p = acnt[AB_P_READY], c_o0 = acnt[AB_O_DONE], c_o1 = acnt[AB_O_DONE + 1], c_fix = acnt[AB_FIXED], c_land = acnt[AB_LANDED];
    // P V of chunk c completes phase c >> 1 of o_done[c & 1]
    auto o_par = [&](int c) { return ((c & 1 ? c_o1 : c_o0) + (uint32_t)(c >> 1)) & 1u; };
    auto full_par = [&](int j) { return (c_full[j % kTcStages] + (uint32_t)(j / kTcStages)) & 1u; };          // stage j has landed
    auto free_par = [&](int j) { return ((c_free[j % kTcStages] + (uint32_t)(j / kTcStages)) & 1u) ^ 1u; };   // its slot was released
    int n_fix_total = 0;
    for (int c = 0; c < n_chunks; ++c) n_fix_total += (p_begin + (c + 1) * kTcChunk > len) ? 1 : 0;

    // The copies of the first chunks do not depend on the set-up below: start them now.
    auto issue_kv = [&](int j) {
        const int slot = j % kTcStages, c = j >> 1;
        const int row = ((j & 1) ? vrow0 : krow0) + p_begin + c * kTcChunk;
        uint8_t *dst = ring + slot * kTcKvStage;
        mbar_expect_tx(&kv_full[slot], kTcKvStage);
        tma_load_2d(dst, p.tm_kv_ptr, 0, row, &kv_full[slot]);
        tma_load_2d(dst + kTcKvStage / 2, p.tm_kv_ptr, 64, row, &kv_full[slot]);
    };
    const int n_early = min(kTcStages, 2 * n_chunks);
    if (warp == 5 && lane == 0 && !sh->abort) {
        fence_async_proxy();  // the previous user of these slots wrote them through the generic proxy
        for (int j = 0; j < n_early; ++j) issue_kv(j);
    }
    // ---- set-up: Q tile (rotary applied; 16 hi rows, 16 lo rows), P tile zeroed ----
    {
        const int ml = tid >> 4, v8 = tid & 15, m = m_base + ml;
        float q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) q[u] = 0.f;
        if (m < n_rows && ml < rows_here) rope_vec8(p, p.qkv + (size_t)(r0 + m) * 3 * d + h * Dh, r0 + m, v8 * 8, q);
        __nv_bfloat16 hq[8], lq[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            hq[u] = __float2bfloat16_rn(q[u]);
            lq[u] = __float2bfloat16_rn(q[u] - __bfloat162float(hq[u]));
        }
        uint8_t *panel = qt + (v8 >> 3) * 4096;
        *reinterpret_cast<uint4 *>(panel + sw128(ml, v8 & 7)) = *reinterpret_cast<uint4 *>(hq);
        *reinterpret_cast<uint4 *>(panel + sw128(16 + ml, v8 & 7)) = *reinterpret_cast<uint4 *>(lq);
#pragma unroll
        for (int i = 0; i < 4; ++i) reinterpret_cast<uint4 *>(pt)[4 * tid + i] = make_uint4(0, 0, 0, 0);  // both P tiles
    }
    fence_async_proxy();
    named_bar(3, kAttnThreadsP);

    if (warp == 5) {
        // ---------------- K / V chunk copies: stage j = 2 c (K), 2 c + 1 (V), slot j % kTcStages ----------------
        if (lane == 0) {
            int issued = n_early;
            for (int j = n_early; j < 2 * n_chunks && !sh->abort; ++j) {
                wait(&kv_free[j % kTcStages], free_par(j));
                if (sh->abort) break;
                issue_kv(j);
                ++issued;
            }
            if (sh->abort)  // error path only: copies still in flight
                for (int j = max(0, issued - kTcStages); j < issued; ++j) mbar_wait(&kv_full[j % kTcStages], full_par(j));
        }
        __syncwarp();
    } else if (warp == 4) {
        // ---------------- MMA issue ----------------
        if (lane == 0) {
            const uint32_t idS = umma_idesc_bf16(128, 32), idO = umma_idesc_bf16(128, 32) | (1u << 15);  // A of PV: MN-major
            const uint32_t qa = smem_u32(qt), pa = smem_u32(pt);
            int n_fix = 0;
            // S(c): scores of chunk c into buffer c & 1; issued one chunk ahead of P V so that it runs
            // while the softmax threads work on the previous chunk
            auto issue_s = [&](int c) {
                const int jk = 2 * c, jv = 2 * c + 1;
                const bool fix = p_begin + (c + 1) * kTcChunk > len;
                wait(&kv_full[jk % kTcStages], full_par(jk));
                if (fix) {  // both tiles are here: let the patching threads in, wait for them
                    wait(&kv_full[jv % kTcStages], full_par(jv));
                    if (!sh->abort) mbar_arrive(landed);
                    wait(fixed, (c_fix + n_fix) & 1u);
                    ++n_fix;
                }
                if (sh->abort) return;
                tc_fence_after();
                const uint32_t ka = smem_u32(ring + (jk % kTcStages) * kTcKvStage);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // k = 16 head dims per step; panel ks / 4
                    tc_mma_bf16(tS + 32 * (c & 1), umma_desc(ka + (ks >> 2) * (kTcKvStage / 2) + (ks & 3) * 32, 16, 1024),
                                umma_desc(qa + (ks >> 2) * 4096 + (ks & 3) * 32, 16, 1024), idS, ks ? 1u : 0u);
                tc_commit(&s_full[c & 1]);
                tc_commit(&kv_free[jk % kTcStages]);
            };
            if (n_chunks > 0) issue_s(0);
            for (int c = 0; c < n_chunks && !sh->abort; ++c) {
                const int jv = 2 * c + 1;
                if (c + 1 < n_chunks) issue_s(c + 1);
                wait(p_ready, (c_p + c) & 1u);
                wait(&kv_full[jv % kTcStages], full_par(jv));
                if (sh->abort) break;
                tc_fence_after();
                const uint32_t va = smem_u32(ring + (jv % kTcStages) * kTcKvStage);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // k = 16 positions per step: two 8-row groups of the V tile
                    tc_mma_bf16(tO, umma_desc(va + ks * 2048, kTcKvStage / 2, 1024),
                                umma_desc(pa + (c & 1) * kTcPBytes + (ks >> 2) * 4096 + (ks & 3) * 32, 16, 1024), idO, (c | ks) ? 1u : 0u);
                tc_commit(&o_done[c & 1]);
                tc_commit(&kv_free[jv % kTcStages]);
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ---------------- rows of this pass, chunk by chunk ----------------
        const int ft = tid - 192;  // 0..63
        int n_fixed = 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int base = p_begin + c * kTcChunk;
            if (base + kTcChunk <= len) continue;
            const int jk = 2 * c, jv = 2 * c + 1;
            uint8_t *kt = ring + (jk % kTcStages) * kTcKvStage, *vt = ring + (jv % kTcStages) * kTcKvStage;
            const int first = max(0, len - base), last = min(kTcChunk, len + n_rows - base);  // tile rows [first, last)
            // at most 32 rows x 16 vectors = 8 work items per thread: compute them all, then wait for the copies
            uint4 kq[8], vq[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = ft + 64 * u, pr = first + (i >> 4), v8 = i & 15;
                kq[u] = vq[u] = make_uint4(0, 0, 0, 0);
                if (pr < last) {
                    const int pos = base + pr, r = r0 + (pos - len);
                    const float *krow = p.qkv + (size_t)r * 3 * d + d + h * Dh;
                    float kf[8];
                    rope_vec8(p, krow, r, v8 * 8, kf);
                    const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(krow + d + v8 * 8));
                    const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(krow + d + v8 * 8 + 4));
                    const float vf[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                    __nv_bfloat16 kb[8], vb[8];
#pragma unroll
                    for (int w = 0; w < 8; ++w) {
                        kb[w] = __float2bfloat16_rn(kf[w]);
                        vb[w] = __float2bfloat16_rn(vf[w]);
                    }
                    kq[u] = *reinterpret_cast<uint4 *>(kb);
                    vq[u] = *reinterpret_cast<uint4 *>(vb);
                }
            }
            wait(landed, (c_land + (uint32_t)n_fixed) & 1u);
            ++n_fixed;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = ft + 64 * u, pr = first + (i >> 4), v8 = i & 15;
                if (pr < last) {
                    const uint32_t off = (uint32_t)(v8 >> 3) * (kTcKvStage / 2) + sw128(pr, v8 & 7);
                    *reinterpret_cast<uint4 *>(kt + off) = kq[u];
                    *reinterpret_cast<uint4 *>(vt + off) = vq[u];
                    if (mt == 0) {  // append: exactly one split owns this position (stores after all the loads)
                        const size_t go = (size_t)(base + pr) * Dh + v8 * 8;
                        *reinterpret_cast<uint4 *>(kc + go) = kq[u];
                        *reinterpret_cast<uint4 *>(vc + go) = vq[u];
                    }
                }
            }
            fence_async_proxy();
            mbar_arrive(fixed);
        }
    } else {
        // ---------------- softmax: thread = position tid of the chunk ----------------
        // Runtime loops over the real rows (usually 5 of 16) and per-row tensor-memory loads keep this
        // code small: it runs once per item and layer, so its instruction fetch is mostly cold.
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        float *lrow = l_sh + tid;
        for (int r = 0; r < rows_here; ++r) lrow[r * 128] = 0.f;
        if (lane < kAttnRows) { wmrun[warp * 16 + lane] = -INFINITY; fsh[warp * 16 + lane] = 1.f; }
        __syncwarp();
        for (int c = 0; c < n_chunks; ++c) {
            const int pos = p_begin + c * kTcChunk + tid;
            const uint32_t tSc = tS + 32 * (c & 1) + lane_sel;
            float *wmax = wmax2 + 64 * (c & 1);
            wait(&s_full[c & 1], ((c & 1 ? c_s1 : c_s0) + (uint32_t)(c >> 1)) & 1u);
            tc_fence_after();
            // the chunk's row maxima over its 128 positions; 8 rows per tensor-memory round trip, unrolled
            // over those 8 so that their shuffles and exponentials overlap
            const int nblk = (rows_here + 7) >> 3;
#pragma unroll 1
            for (int blk = 0; blk < nblk; ++blk) {
                float a[8], b2[8];
                tc_ld_2x8(tSc + 8 * blk, tSc + 16 + 8 * blk, a, b2);
                float mx[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = 8 * blk + i;
                    const bool vis = r < rows_here && pos < p_end && pos <= len + m_base + r;
                    mx[i] = vis ? (a[i] + b2[i]) * sc : -INFINITY;
                }
#pragma unroll
                for (int o = 16; o; o >>= 1)
#pragma unroll
                    for (int i = 0; i < 8; ++i) mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], o));
                if (lane < 8) {
                    float sel = mx[0];
#pragma unroll
                    for (int i = 1; i < 8; ++i) sel = lane == i ? mx[i] : sel;
                    wmax[warp * 16 + 8 * blk + lane] = sel;
                }
            }
            named_bar(6, 128);
            if (c > 1) wait(&o_done[c & 1], o_par(c - 2));  // this chunk's P tile was last read by P V of chunk c - 2
            bool moved = false;
            uint8_t *panel = pt + (c & 1) * kTcPBytes + (tid >> 6) * 4096;
            const int cc = (tid & 63) >> 3, e = (tid & 7) * 2;
#pragma unroll 1
            for (int blk = 0; blk < nblk; ++blk) {
                float a[8], b2[8];
                tc_ld_2x8(tSc + 8 * blk, tSc + 16 + 8 * blk, a, b2);
                float fl[8], ml[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = 8 * blk + i;
                    fl[i] = 1.f;
                    ml[i] = -INFINITY;
                    if (r < rows_here) {
                        const bool vis = pos < p_end && pos <= len + m_base + r;
                        const float v = vis ? (a[i] + b2[i]) * sc : -INFINITY;
                        const float mc = fmaxf(fmaxf(wmax[r], wmax[16 + r]), fmaxf(wmax[32 + r], wmax[48 + r]));
                        const float m_old = wmrun[warp * 16 + r];
                        const float m_new = (mc > m_old + kTcMaxSlack || m_old == -INFINITY) ? fmaxf(m_old, mc) : m_old;
                        float pv = 0.f;
                        if (m_new > -INFINITY) {
                            fl[i] = exp2f(m_old - m_new);  // 0 on the first non-empty chunk
                            pv = exp2f(v - m_new);
                        }
                        ml[i] = m_new;
                        moved = moved || (fl[i] != 1.f);  // the same in all 128 threads: they read the same maxima
                        lrow[r * 128] = lrow[r * 128] * fl[i] + pv;
                        // P as bf16 hi + lo into the P tile: row r (hi) / 16 + r (lo), column = this position
                        const __nv_bfloat16 hv = __float2bfloat16_rn(pv);
                        *reinterpret_cast<__nv_bfloat16 *>(panel + sw128(r, cc) + e) = hv;
                        *reinterpret_cast<__nv_bfloat16 *>(panel + sw128(16 + r, cc) + e) =
                            __float2bfloat16_rn(pv - __bfloat162float(hv));
                    }
                }
                __syncwarp();  // every lane has read this block's running maxima
                if (lane < 8 && 8 * blk + lane < rows_here) {
                    float msel = ml[0], fsel = fl[0];
#pragma unroll
                    for (int i = 1; i < 8; ++i) {
                        msel = lane == i ? ml[i] : msel;
                        fsel = lane == i ? fl[i] : fsel;
                    }
                    wmrun[warp * 16 + 8 * blk + lane] = msel;
                    fsh[warp * 16 + 8 * blk + lane] = fsel;
                }
            }
            __syncwarp();
            if (c > 0 && moved) {  // thread = head dim tid: scale the accumulated O^T, once P V of the previous chunk has written it
                wait(&o_done[(c - 1) & 1], o_par(c - 1));
                tc_fence_after();
                float o[32];
                tc_ld_32(tO + lane_sel, o);
#pragma unroll
                for (int r = 0; r < kAttnRows; ++r) {
                    const float f = fsh[warp * 16 + r];  // 1 for rows beyond rows_here
                    o[r] *= f;
                    o[16 + r] *= f;
                }
                tc_st_32(tO + lane_sel, o);
            }
            fence_async_proxy();
            tc_fence_before();
            mbar_arrive(p_ready);
        }
        // ---- the sums over positions, then thread = head dim tid: output or partial ----
#pragma unroll 1
        for (int r = 0; r < rows_here; ++r) {
            float t = lrow[r * 128];
#pragma unroll
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) wsum[warp * 16 + r] = t;
        }
        if (n_chunks > 1) wait(&o_done[(n_chunks - 2) & 1], o_par(n_chunks - 2));
        if (n_chunks > 0) {
            wait(&o_done[(n_chunks - 1) & 1], o_par(n_chunks - 1));
            tc_fence_after();
        }
        named_bar(6, 128);
        const bool direct = p.n_split == 1;
#pragma unroll 1
        for (int r = 0; r < rows_here; ++r) {
            const int m = m_base + r;
            const float L = (wsum[r] + wsum[16 + r]) + (wsum[32 + r] + wsum[48 + r]);
            const bool live = m < n_rows && L > 0.f && n_chunks > 0;
            float a = 0.f, b2 = 0.f;
            if (n_chunks > 0) tc_ld_2(tO + lane_sel + r, tO + lane_sel + 16 + r, a, b2);
            const float acc = live ? a + b2 : 0.f;
            if (direct) {
                store_hilo(p.op[OP_AO], p.rk, r0 + m, h * Dh + tid, live ? acc / L : 0.f);
            } else {
                const size_t slot = ((size_t)(r0 + m) * p.H + h) * p.n_split + split;
                if (tid == 0) {
                    p.part_m[slot] = live ? wmrun[r] : -INFINITY;
                    p.part_l[slot] = live ? L : 0.f;
                }
                p.part_o[slot * Dh + tid] = acc;
            }
        }
        tc_fence_before();
    }
    if (p.n_split != 1) {
        // ticket: the item that finishes last for this (sequence, head) merges all partials
        __threadfence();
        named_bar(3, kAttnThreadsP);
        if (tid == 0) sh->flag = (atomicAdd(p.tickets + bh, 1u) == (unsigned)(p.n_split * MT - 1));
        named_bar(3, kAttnThreadsP);
        if (sh->flag) {
            __threadfence();
            merge_splits(p, r0, h, Dh);
            if (tid == 0) p.tickets[bh] = 0;  // ready for the next layer (a grid barrier lies between)
        }
    }
    if (tid == 0) {
        for (int i = 0; i < kTcStages; ++i) {
            const uint32_t uses = (uint32_t)((2 * n_chunks + kTcStages - 1 - i) / kTcStages);  // stages j < 2 n_chunks with j % kTcStages == i
            acnt[AB_KV_FULL + i] = c_full[i] + uses;
            acnt[AB_KV_FREE + i] = c_free[i] + uses;
        }
        acnt[AB_S_FULL] = c_s0 + (uint32_t)((n_chunks + 1) / 2);
        acnt[AB_S_FULL + 1] = c_s1 + (uint32_t)(n_chunks / 2);
        acnt[AB_P_READY] = c_p + n_chunks;
        acnt[AB_O_DONE] = c_o0 + (uint32_t)((n_chunks + 1) / 2);
        acnt[AB_O_DONE + 1] = c_o1 + (uint32_t)(n_chunks / 2);
        acnt[AB_FIXED] = c_fix + n_fix_total;
        acnt[AB_LANDED] = c_land + n_fix_total;
    }
    named_bar(3, kAttnThreadsP);  // scratch, tensor memory and the counts are ready for the next item
}

__device__ __forceinline__ void attention_phase(const FwdParams &p, int layer, uint8_t *scratch, Shared *sh) {
    const int MT = (p.M + kAttnRows - 1) / kAttnRows;
    const int items = p.B * p.H * p.n_split * MT;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        if (p.attn_tc == 1) attention_item_tc(p, layer, item, scratch, sh);
        else if (p.attn_tc == 2 && p.Dh == 128) attention_item_mma8<128>(p, layer, item, scratch, sh);
        else if (p.attn_tc == 2) attention_item_mma8<64>(p, layer, item, scratch, sh);
        else attention_item(p, layer, item, scratch, sh);
    }
}

// Where the kernel's small state lives behind the ring (and the attention scratch) in shared memory.
struct SmemMap {
    uint64_t *fullW, *fullX, *empty, *accFull, *accEmpty, *mmaDone;
    uint32_t *tmem_slot;
    Shared *sh;
    double *red;
    float *epi_tile;
    volatile int *epi_ok;
    uint64_t *abar;
    uint32_t *acnt;
    RingPos *role_rp;  // [2]: the MMA issuer's and the operand issuer's walk of the ring, between GEMMs
    int *role_seg;     // [8]: per work warp, tile segments so far
    FwdParams *params; // the kernel parameters, copied once (see forward_kernel)
    int *seq;          // [128]: lengths, rows of this pass
    const float **ltab;  // [8 * kMaxStagedLayers + 2]
};
__device__ __forceinline__ SmemMap smem_map(const FwdParams &p, uint8_t *smem) {
    SmemMap m;
    const int S = p.stages;
    m.fullW = (uint64_t *)(smem + p.bar_off);
    m.fullX = m.fullW + S;
    m.empty = m.fullX + S;
    m.accFull = m.empty + S;
    m.accEmpty = m.accFull + 2;
    m.mmaDone = m.accEmpty + 2;
    m.tmem_slot = (uint32_t *)(m.mmaDone + 1);
    m.sh = (Shared *)(((uintptr_t)(m.mmaDone + 4) + 15) & ~(uintptr_t)15);
    m.red = (double *)(m.sh + 1);
    m.epi_tile = (float *)(m.red + 16);
    m.epi_ok = (volatile int *)(m.epi_tile + 8 * kEpiPitch);
    m.abar = (uint64_t *)(m.epi_tile + 8 * kEpiPitch + 4);
    m.acnt = (uint32_t *)(m.abar + AB_COUNT);
    m.role_rp = (RingPos *)(m.acnt + AB_COUNT);
    m.role_seg = (int *)(m.role_rp + 2);
    m.params = (FwdParams *)(((uintptr_t)(m.role_seg + 8) + 63) & ~(uintptr_t)63);
    m.seq = (int *)((uint8_t *)m.params + 960);
    m.ltab = (const float **)(m.seq + 128);
    return m;
}

// Run this CTA's units of GEMM gi (all 256 work threads call it; NT = padded rows / 8).  The units are
// contiguous in (tile, k-chunk) order, so they form one segment per tile touched; each segment is
// accumulated in tensor memory and reduced into the output once.  A function of its own, with the
// little state that survives from GEMM to GEMM kept in shared memory, so that the kernel's phase loop
// holds nothing across its calls: with 227 KB of shared memory there is next to no L1 left, and a
// value spilled to the stack costs an L2 round trip at every phase.
template <int NT>
__device__ __noinline__ void run_gemm(const FwdParams &p, int gi, uint8_t *smem) {
    constexpr int kRp = NT * 8;
    constexpr int kXBytes = 2 * kRp * kTileK * 2;
    constexpr int kStageBytes = kXBytes + kWTileBytesP;
    // M of the MMA: the operand tile's 2 kRp rows; the rows the MMA reads beyond them are the weight
    // tile's bytes (finite or not, they only reach accumulator lanes that nobody loads)
    constexpr int kM = 2 * kRp <= 64 ? 64 : 128;
    const SmemMap mp = smem_map(p, smem);
    const int S = p.stages, S1 = p.stages_lo;
    uint8_t *ring = smem;
    uint64_t *fullW = mp.fullW, *fullX = mp.fullX, *empty = mp.empty, *accFull = mp.accFull, *accEmpty = mp.accEmpty;
    Shared *sh = mp.sh;
    float *epi_tile = mp.epi_tile;
    volatile int *epi_ok = mp.epi_ok;
    const uint32_t tmem_base = sh->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool walks_ring = lane == 0 && (warp == kMmaWarp || warp == kXWarp);
    RingPos rp;
    if (walks_ring) rp = mp.role_rp[warp == kMmaWarp ? 0 : 1];
    int seg = mp.role_seg[warp];
    auto save_state = [&]() {
        if (walks_ring) mp.role_rp[warp == kMmaWarp ? 0 : 1] = rp;
        __syncwarp();
        if (lane == 0) mp.role_seg[warp] = seg;
        __syncwarp();
    };

            const GemmDesc g = gemm_desc(p, gi, staged_ltab(sh));
            int c0, c1;
            unit_range(p, g, c0, c1);
            if (c0 >= c1) return;  // (no state to save: nothing moved)
            const int tile0 = c0 / g.kchunks, tile1 = (c1 - 1) / g.kchunks;
            if (warp == kMmaWarp) {
                if (lane == 0 && !sh->abort) {
                    const uint32_t idesc = umma_idesc_bf16(kM, kTileNP);
                    int sg = seg, kc = c0 % g.kchunks;
                    bool first = true;
                    for (int c = c0; c < c1; ++c) {
                        uint32_t ph;
                        const int s = ring_next(rp, ring_lo_only(g, c - c0, S1), S, S1, ph), b = sg & 1;
                        bool ok = true;
                        if (first && sg >= 2) ok = mbar_wait_or_abort(&accEmpty[b], ((sg >> 1) - 1) & 1, sh);
                        ok = ok && mbar_wait_or_abort(&fullW[s], ph, sh) && mbar_wait_or_abort(&fullX[s], ph, sh);
                        if (!ok) {
                            set_status(p.status, kTimeoutCode);
                            sh->abort = 1;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t st = smem_u32(ring + (size_t)s * kStageBytes);
                        const uint64_t adesc = umma_desc_sw128(st), bdesc = umma_desc_sw128(st + kXBytes);
                        const uint32_t d_tmem = tmem_base + (uint32_t)(b * kAccStride);
#pragma unroll
                        for (int ks = 0; ks < kTileK / 16; ++ks)  // 32 bytes further along k inside the swizzle atom
                            tc_mma_bf16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, idesc, (first && ks == 0) ? 0u : 1u);
                        tc_commit(&empty[s]);
                        first = false;
                        ++kc;
                        if (kc == g.kchunks || c + 1 == c1) {
                            tc_commit(&accFull[b]);
                            ++sg;
                            first = true;
                            if (kc == g.kchunks) kc = 0;
                        }
                    }
                }
                __syncwarp();
            } else if (warp == kXWarp) {
                // operand tiles of this GEMM (their phase has been released: this runs after its barrier)
                bool ready = true;
                if (lane == 0 && !sh->abort && g.wait_attn) {
                    // the attention output is complete once every attention CTA of this layer has signalled
                    const unsigned *cnt = attn_done(p);
                    if (ld_acquire(cnt) < g.wait_attn) {
                        const long long t0 = clock64();
                        while (ld_acquire(cnt) < g.wait_attn) {
                            if (sh->abort || clock64() - t0 > sh->wait_limit) { ready = false; break; }
                        }
                    }
                    if (!ready) {
                        set_status(p.status, kTimeoutCode);
                        sh->abort = 1;
                    }
                }
                if (lane == 0 && ready && !sh->abort) {
                    fence_async_proxy();  // that phase's generic-proxy writes -> visible to the bulk copies
                    int kx = c0 % g.kchunks;
                    for (int c = c0; c < c1; ++c) {
                        uint32_t ph;
                        const int s = ring_next(rp, ring_lo_only(g, c - c0, S1), S, S1, ph);
                        if (!mbar_wait_or_abort(&empty[s], ph ^ 1u, sh)) {
                            rp.par ^= 1u << s;  // nothing was issued into s
                            set_status(p.status, kTimeoutCode);
                            sh->abort = 1;
                            break;
                        }
                        mbar_expect_tx(&fullX[s], kXBytes);
                        bulk_load_1d(ring + (size_t)s * kStageBytes, g.xop + (size_t)kx * (2 * kRp * kTileK), kXBytes,
                                     &fullX[s]);
                        if (++kx == g.kchunks) kx = 0;
                    }
                }
                __syncwarp();
            } else if (warp < kEpiWarps) {
                int sg = seg;
                const bool vec_ok = (((uintptr_t)g.out & 15) == 0) && ((g.ldo & 3) == 0) &&
                                    (!g.bias || ((uintptr_t)g.bias & 15) == 0);
                for (int t = tile0; t <= tile1; ++t, ++sg) {
                    const int b = sg & 1;
                    // the four warps take the same decision: the named barriers below need all of them
                    const bool mine = mbar_wait_or_abort(&accFull[b], (sg >> 1) & 1, sh);
                    if (lane == 0) epi_ok[warp] = mine ? 1 : 0;
                    named_bar(5, kEpiWarps * 32);
                    if (!(epi_ok[0] && epi_ok[1] && epi_ok[2] && epi_ok[3])) {
                        set_status(p.status, kTimeoutCode);
                        sh->abort = 1;
                        break;
                    }
                    tc_fence_after();
                    const bool has_k0 = (t > tile0) || (c0 % g.kchunks == 0);
                    const float *bias = (has_k0 && g.bias) ? g.bias : nullptr;
                    const int g8 = lane >> 2, t4 = lane & 3;
                    // Block q of 8 rows sits in accumulator lanes 32 q .. 32 q + 15 (M = 64) or 16 q .. 16 q + 15
                    // (M = 128); a warp reaches the 32 lanes of its own quadrant only.
#pragma unroll 1
                    for (int q = 0; q < NT; ++q) {
                        if (8 * q >= p.R) break;
                        const int wq = kM == 64 ? q : (q >> 1), half = kM == 64 ? 0 : (q & 1);
                        if (wq == warp) {
                            const uint32_t ta = tmem_base + ((uint32_t)(warp * 32 + half * 16) << 16) + (uint32_t)(b * kAccStride);
                            for (int cg = 0; cg < kTileNP / 64; ++cg) {  // 64 columns per tensor-memory round trip
                                if (t * kTileNP + cg * 64 >= g.N) break;
                                float v[32];
                                tc_ld_16x64(ta + (uint32_t)(cg * 64), v);
#pragma unroll
                                for (int k = 0; k < 8; ++k)
                                    *reinterpret_cast<float2 *>(epi_tile + g8 * kEpiPitch + cg * 64 + 8 * k + 2 * t4) =
                                        make_float2(v[4 * k] + v[4 * k + 2], v[4 * k + 1] + v[4 * k + 3]);
                            }
                        }
                        named_bar(5, kEpiWarps * 32);
                        const int rows_here = min(8, p.R - 8 * q);
                        for (int i = threadIdx.x; i < rows_here * (kTileNP / 4); i += kEpiWarps * 32) {
                            const int rr = i / (kTileNP / 4), c4 = (i % (kTileNP / 4)) * 4, n = t * kTileNP + c4;
                            if (n >= g.N) continue;
                            float4 v = *reinterpret_cast<const float4 *>(epi_tile + rr * kEpiPitch + c4);
                            float *dst = g.out + (size_t)(8 * q + rr) * g.ldo + n;
                            if (vec_ok && n + 3 < g.N) {
                                if (bias) {
                                    const float4 bb = __ldg(reinterpret_cast<const float4 *>(bias + n));
                                    v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                                }
                                red_add_v4(dst, v);
                            } else {
                                const float e[4] = {v.x, v.y, v.z, v.w};
                                for (int u = 0; u < 4; ++u)
                                    if (n + u < g.N) atomicAdd(dst + u, e[u] + (bias ? __ldg(bias + n + u) : 0.f));
                            }
                        }
                        named_bar(5, kEpiWarps * 32);  // the tile is free for the next block
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&accEmpty[b]);
                }
            }
            seg += tile1 - tile0 + 1;
            save_state();
}

// ---- the vocabulary-wide tail of a draft step, inside the kernel ---------------------------------
// After the LM head of a draft step every sequence's last fed row of logits is turned into q = softmax(row / T),
// exported, and sampled by inverse CDF with the step's uniform - the work of draft_tail_kernel, spread over the
// whole grid so that the kernel can go on to the next step without returning to the host.  CTA c owns the slice
// [c * per, (c + 1) * per) of the vocabulary; inside a CTA warp w works on sequences w, w + 8, ... with warp
// shuffles only.  Three phases, a grid barrier behind each:
//   1. per (sequence, CTA): max, argmax and sum of exp relative to that max over the slice;
//   2. every CTA combines the partials of all CTAs into (max, argmax, Z), writes its slice of q and the slice's
//      mass (fp64, index order: lane l holds a contiguous piece of the slice);
//   3. every CTA takes the prefix of the slice masses in CTA order; the lanes whose piece can hold the first
//      index with c_j > u S walk it and post the index (atomic minimum); the largest index with q > 0 is
//      posted too (the fallback when rounding leaves no index past u S);
// then CTA 0 writes the tokens and commits the rows fed in this step.
__device__ __forceinline__ int tail_per(const FwdParams &p) { return (((p.V + (int)gridDim.x - 1) / (int)gridDim.x) + 3) & ~3; }
__device__ __forceinline__ const float *tail_row(const FwdParams &p, const Shared *sh, int b) {
    int row = (b < 64 ? staged_len(sh)[64 + b] : __ldcg(p.ri.n_eff + b)) - 1;  // (staged behind the step's first barrier)
    if (row < 0) row = 0;
    return p.logits + ((size_t)b * p.M + row) * p.V;
}

// (All loops below fetch eight elements before they use the first: a load from L2 costs about a microsecond
// under the weight stream, and a slice is only a few hundred elements.)
__device__ __noinline__ void tail_partial(const FwdParams &p, const Shared *sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, G = (int)gridDim.x;
    const int per = tail_per(p), lo = min(p.V, (int)blockIdx.x * per), hi = min(p.V, lo + per);
    for (int b = warp; b < p.B; b += kConsumerWarps) {
        const float *lg = tail_row(p, sh, b);
        // running (max, argmax, sum of exp relative to the max) per lane, then over the warp
        float mx = -INFINITY, sum = 0.f;
        int am = 0x7fffffff;
        for (int jb = lo + lane; jb < hi; jb += 256) {
            float l[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) l[u] = jb + 32 * u < hi ? __ldcg(lg + jb + 32 * u) : -INFINITY;
            float m8 = mx;
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (l[u] > m8) { m8 = l[u]; am = jb + 32 * u; }  // ascending per lane: the first maximum
            if (p.inv_t != 0.f && m8 > -INFINITY) {
                sum *= expf((mx - m8) * p.inv_t);  // 0 while nothing has been summed
#pragma unroll
                for (int u = 0; u < 8; ++u) sum += expf((l[u] - m8) * p.inv_t);  // exp(-inf) = 0
            }
            mx = m8;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sum, o);
            const int oi = __shfl_xor_sync(0xffffffffu, am, o);
            const float m2 = fmaxf(mx, ov);
            if (m2 > -INFINITY) sum = sum * expf((mx - m2) * p.inv_t) + os * expf((ov - m2) * p.inv_t);
            if (ov > mx || (ov == mx && oi < am)) am = oi;
            mx = m2;
        }
        if (lane == 0) {
            p.tp_m[(size_t)b * G + blockIdx.x] = mx;
            p.tp_s[(size_t)b * G + blockIdx.x] = sum;
            p.tp_a[(size_t)b * G + blockIdx.x] = am;
        }
    }
}

// (max, argmax - lowest index among the maxima -, Z) of a sequence's row from the CTAs' partials; the same in every lane
__device__ __forceinline__ void tail_stats(const FwdParams &p, int b, float &mx, int &am, float &z) {
    const int lane = threadIdx.x & 31, G = (int)gridDim.x;
    float pm[8], ps[8];
    int pa[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {  // (grids of up to 256 CTAs)
        const int c = lane + 32 * k;
        pm[k] = c < G ? __ldcg(p.tp_m + (size_t)b * G + c) : -INFINITY;
        ps[k] = c < G ? __ldcg(p.tp_s + (size_t)b * G + c) : 0.f;
        pa[k] = c < G ? __ldcg(p.tp_a + (size_t)b * G + c) : 0x7fffffff;
    }
    mx = -INFINITY;
    am = 0x7fffffff;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        if (pm[k] > mx || (pm[k] == mx && pa[k] < am)) { mx = pm[k]; am = pa[k]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, mx, o);
        const int oi = __shfl_xor_sync(0xffffffffu, am, o);
        if (ov > mx || (ov == mx && oi < am)) { mx = ov; am = oi; }
    }
    double zz = 0.0;
    if (p.inv_t != 0.f) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (pm[k] > -INFINITY) zz += (double)ps[k] * (double)expf((pm[k] - mx) * p.inv_t);
    }
    zz = warp_sum(zz);
    z = (float)zz;
}
__device__ __forceinline__ float tail_prob(float logit, float mx, int am, float z, float inv_t, int j) {
    if (inv_t == 0.f) return j == am ? 1.f : 0.f;
    return expf((logit - mx) * inv_t) / z;
}

__device__ __noinline__ void tail_q(const FwdParams &p, const Shared *sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, G = (int)gridDim.x;
    const int per = tail_per(p), lo = min(p.V, (int)blockIdx.x * per), hi = min(p.V, lo + per);
    const int seg = (hi - lo + 31) / 32, j0 = min(hi, lo + lane * seg), j1 = min(hi, j0 + seg);
    for (int b = warp; b < p.B; b += kConsumerWarps) {
        const float *lg = tail_row(p, sh, b);
        float l[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) l[u] = j0 + u < j1 ? __ldcg(lg + j0 + u) : 0.f;  // (under the partials' latency)
        float mx, z;
        int am;
        tail_stats(p, b, mx, am, z);
        float *q = p.q_out + (size_t)b * p.q_stride + (size_t)p.cur_step * p.V;
        double local = 0.0;
        for (int jb = j0; jb < j1; jb += 8) {
            if (jb > j0) {
#pragma unroll
                for (int u = 0; u < 8; ++u) l[u] = jb + u < j1 ? __ldcg(lg + jb + u) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (jb + u < j1) {
                    const float w = tail_prob(l[u], mx, am, z, p.inv_t, jb + u);
                    q[jb + u] = w;
                    local += (double)w;
                }
        }
        local = warp_sum(local);  // (a sum of at most 32 pieces: the order does not matter at fp64 for a decision that
        if (lane == 0) p.tp_mass[(size_t)b * G + blockIdx.x] = local;  //  is excused within 1e-6 S of a step anyway)
    }
}

__device__ __noinline__ void tail_draw(const FwdParams &p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, G = (int)gridDim.x;
    const int per = tail_per(p), lo = min(p.V, (int)blockIdx.x * per), hi = min(p.V, lo + per);
    const int seg = (hi - lo + 31) / 32, j0 = min(hi, lo + lane * seg), j1 = min(hi, j0 + seg);
    for (int b = warp; b < p.B; b += kConsumerWarps) {
        // total and this CTA's offset from the slice masses (lane l takes CTAs l, l + 32, ...; fp64)
        double off = 0.0, S = 0.0;
        {
            double t[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) t[k] = lane + 32 * k < G ? __ldcg(p.tp_mass + (size_t)b * G + lane + 32 * k) : 0.0;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                S += t[k];
                if (lane + 32 * k < (int)blockIdx.x) off += t[k];
            }
            S = warp_sum(S);
            off = warp_sum(off);
        }
        const float *q = p.q_out + (size_t)b * p.q_stride + (size_t)p.cur_step * p.V;
        double local = 0.0;
        int last_pos = -1;
        for (int jb = j0; jb < j1; jb += 8) {
            float w[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) w[u] = jb + u < j1 ? __ldcg(q + jb + u) : 0.f;  // written by this very lane in the phase before
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                local += (double)w[u];
                if (w[u] > 0.f) last_pos = jb + u;
            }
        }
        double incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const double target = (double)__ldcg(p.u + (size_t)b * p.u_stride + p.cur_step) * S;
        double run = off + (incl - local);
        int hit = 0x7fffffff;
        if (S > 0.0 && (run + local > target || run > target)) {
            for (int j = j0; j < j1; ++j) {
                const float w = __ldcg(q + j);
                run += (double)w;
                if (w > 0.f && run > target) { hit = j; break; }  // a zero-weight index is never drawn
            }
        }
        // one atomic per warp, not per lane: thousands of atomics on one word would serialise in L2
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            hit = min(hit, __shfl_xor_sync(0xffffffffu, hit, o));
            last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
        }
        int32_t *slot = p.tail_hit + ((size_t)p.cur_step * p.B + b) * 2;
        if (lane == 0 && hit != 0x7fffffff) atomicMin(slot, hit);
        if (lane == 0 && last_pos >= 0) atomicMax(slot + 1, last_pos);
    }
}

// CTA 0: the tokens of this step, and the rows it fed become part of the cache
__device__ __noinline__ void tail_commit(const FwdParams &p) {
    if (blockIdx.x != 0) return;
    for (int b = threadIdx.x; b < p.B; b += kWorkThreads) {
        const int32_t *slot = p.tail_hit + ((size_t)p.cur_step * p.B + b) * 2;
        const int hit = __ldcg(slot), last = __ldcg(slot + 1);
        int tok = hit != 0x7fffffff ? hit : last;
        if (tok < 0) tok = max(0, min(__ldcg(p.tp_a + (size_t)b * gridDim.x), p.V - 1));  // a row without any probability
        p.tok_out[(size_t)b * p.tok_out_stride + p.cur_step] = tok;
        p.len_rw[b] = __ldcg(p.len_rw + b) + __ldcg(p.ri.n_eff + b);
    }
}

// ---- the kernel -----------------------------------------------------------------------------
// NT = padded rows / 8
template <int NT>
__global__ void __launch_bounds__(kPersistThreads, 1) forward_kernel(const __grid_constant__ FwdParams kp) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // The phase functions are not inlined and read their parameters through a reference; a reference into the
    // kernel-parameter bank makes every field a generic load at the head of each phase, so they get a copy in
    // shared memory instead (tensor maps stay where the copy engine can read them: pointers into kp / global).
    static_assert(sizeof(FwdParams) <= 960, "parameter copy area");
    FwdParams *psm = smem_map(kp, smem).params;
    for (int i = threadIdx.x; i < (int)(sizeof(FwdParams) / 4); i += blockDim.x)
        reinterpret_cast<uint32_t *>(psm)[i] = reinterpret_cast<const uint32_t *>(&kp)[i];
    __syncthreads();
    if (threadIdx.x == 0) psm->tm_kv_ptr = &kp.tm_kv;
    const FwdParams &p = *psm;  // (visible to everyone after the barrier below)
    constexpr int kRp = NT * 8;
    constexpr int kXBytes = 2 * kRp * kTileK * 2;  // operand tile (hi and lo rows), then the weight tile
    constexpr int kStageBytes = kXBytes + kWTileBytesP;
    const int S = p.stages, S1 = p.stages_lo;
    uint8_t *ring = smem;
    uint8_t *attn_scratch = smem + p.attn_smem_off;
    uint64_t *fullW = (uint64_t *)(smem + p.bar_off);
    uint64_t *fullX = fullW + S, *empty = fullX + S;
    uint64_t *accFull = empty + S, *accEmpty = accFull + 2, *mmaDone = accEmpty + 2;
    uint32_t *tmem_slot = (uint32_t *)(mmaDone + 1);
    Shared *sh = (Shared *)(((uintptr_t)(mmaDone + 4) + 15) & ~(uintptr_t)15);
    double *red = (double *)(sh + 1);
    float *epi_tile = (float *)(red + 16);
    uint64_t *abar = (uint64_t *)(epi_tile + 8 * kEpiPitch + 4);  // the tensor-core attention's barriers and counts
    uint32_t *acnt = (uint32_t *)(abar + AB_COUNT);
    RingPos *role_rp = (RingPos *)(acnt + AB_COUNT);  // the same places smem_map() gives
    int *role_seg = (int *)(role_rp + 2);
    int *seq_tab = smem_map(kp, smem).seq;
    const float **ltab = smem_map(kp, smem).ltab;
    if (kp.n_layers <= kMaxStagedLayers) {  // the layers' gain / bias pointers and the final norm's
        for (int i = threadIdx.x; i < 8 * kp.n_layers + 2; i += blockDim.x) {
            const int l = i >> 3, k = i & 7;
            ltab[i] = l < kp.n_layers ? (&layer_desc(kp.md, l)->ln1_g)[k] : (k == 0 ? kp.md->lnf_g : kp.md->lnf_b);
        }
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {  // tensor memory for the accumulators; released by the same warp at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "n"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&fullW[s], 1);
            mbar_init(&fullX[s], 1);
            mbar_init(&empty[s], 1);  // one tcgen05.commit per stage
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&accFull[b], 1);
            mbar_init(&accEmpty[b], kEpiWarps);
        }
        mbar_init(mmaDone, 1);
        for (int i = 0; i < AB_COUNT; ++i) {
            mbar_init(&abar[i], i == AB_P_READY ? 128 : i == AB_FIXED ? 64 : 1);  // landed: the MMA issuer alone
            acnt[i] = 0;
        }
        role_rp[0] = RingPos();
        role_rp[1] = RingPos();
        for (int i = 0; i < 8; ++i) role_seg[i] = 0;
        sh->released = 0;
        sh->abort = 0;
        sh->go = 1;
        sh->wait_limit = kp.wait_cycles > 0 ? kp.wait_cycles : kWaitCycles;
        sh->attn_bar_off = (uint32_t)((uint8_t *)abar - (uint8_t *)sh);
        sh->seq_off = (uint32_t)((uint8_t *)seq_tab - (uint8_t *)sh);
        sh->ltab_off = kp.n_layers <= kMaxStagedLayers ? (uint32_t)((uint8_t *)ltab - (uint8_t *)sh) : 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) sh->tmem_base = tmem_base;  // read after the next barrier only
    const int NG = n_gemms(p);

    if (warp == kConsumerWarps) {
        // =============================== producer ===============================
        // Weights never change, so this cursor runs as far ahead as the ring allows, across grid
        // barriers.  The loop is kept minimal (no divisions, no clock reads while it makes progress):
        // its rate bounds the weight stream.
        if (lane == 0) {
            RingPos rp;
            bool failed = false;
            int seen_release = 0;
            // a CTA that never runs an attention item (fewer items than CTAs) never uses the scratch: its
            // upper slots take weights at any time
            const bool scratch_used = (int)blockIdx.x < p.B * p.H * p.n_split * ((p.M + kAttnRows - 1) / kAttnRows);
            for (int gws = 0; gws < NG * p.n_steps && !failed; ++gws) {
                const int gw = ((gws / NG) << kStepShift) | (gws % NG);
                const GemmDesc dw = gemm_desc(p, gw);
                int c0, c1;
                unit_range(p, dw, c0, c1);
                if (c0 >= c1) continue;
                int tw = c0 / dw.kchunks, kw = c0 % dw.kchunks;
                for (int c = c0; c < c1; ++c) {
                    uint32_t ph;
                    const int s = ring_next(rp, ring_lo_only(dw, c - c0, S1), S, S1, ph);
                    if (s >= S1 && scratch_used && seen_release < dw.need_hi) {  // slot shared with the attention scratch
                        const long long t0 = clock64();
                        while ((seen_release = sh->released) < dw.need_hi) {
                            if (sh->abort || clock64() - t0 > sh->wait_limit) { failed = true; break; }
                        }
                        if (failed) { rp.par ^= 1u << s; break; }  // nothing was issued into s
                    }
                    if (!mbar_test_wait(&empty[s], ph ^ 1u)) {
                        const long long t0 = clock64();
                        while (!mbar_test_wait(&empty[s], ph ^ 1u)) {
                            if (sh->abort || clock64() - t0 > sh->wait_limit) { failed = true; break; }
                        }
                        if (failed) { rp.par ^= 1u << s; break; }  // nothing was issued into s
                    }
                    mbar_expect_tx(&fullW[s], kWTileBytesP);
                    tma_load_2d(ring + (size_t)s * kStageBytes + kXBytes, dw.tmW, kw * kTileK, tw * kTileNP, &fullW[s]);
                    if (++kw == dw.kchunks) { kw = 0; ++tw; }
                }
            }
            if (failed) {
                set_status(p.status, kTimeoutCode);
                sh->abort = 1;
            }
            // error path only: wait (bounded) for copies still in flight before the CTA may exit
            if (sh->abort)
                for (int s = 0; s < S; ++s)
                    if ((rp.used >> s) & 1u) mbar_wait(&fullW[s], ((rp.par >> s) & 1u) ^ 1u);
        }
    } else {
        // =============================== work warps ===============================
        int epoch = 0;  // grid barriers passed

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
                const float *const *lt = staged_ltab(sh);
                const LayerDesc *ld = layer_desc(p.md, l);
                const float *g1 = lt ? lt[8 * l + 0] : ld->ln1_g, *b1 = lt ? lt[8 * l + 1] : ld->ln1_b;
                if (p.parallel)
                    norm_phase(p, g1, b1, OP_XN1, lt ? lt[8 * l + 4] : ld->ln2_g, lt ? lt[8 * l + 5] : ld->ln2_b, OP_XN2, red);
                else norm_phase(p, g1, b1, OP_XN1, nullptr, nullptr, 0, red);
                grid_zero(p.qkv, p.R, 3 * p.d, 3 * p.d);
                if (p.parallel) grid_zero(p.t_in, p.R, p.d_in, p.d_in);
            } else if (p.want_logits) {
                const float *const *lt = staged_ltab(sh);
                norm_phase(p, lt ? lt[8 * p.n_layers] : p.md->lnf_g, lt ? lt[8 * p.n_layers + 1] : p.md->lnf_b, OP_XN1, nullptr,
                           nullptr, 0, red);
                grid_zero(p.logits, p.R, p.V, p.V);
            }
        };
        if (p.tail && blockIdx.x == 0)  // the draws' meeting places: smallest hit index / largest index with weight
            for (int i = threadIdx.x; i < p.n_steps * p.B * 2; i += kWorkThreads) p.tail_hit[i] = (i & 1) ? -1 : 0x7fffffff;
        bool go = true;
        for (int step = 0; step < p.n_steps && go; ++step) {
            const int gs = step << kStepShift;
            if (step > 0) {  // the rows of this step: one per sequence, the token the step before drew
                if (threadIdx.x == 0) psm->cur_step = step;
                named_bar(2, kWorkThreads);
            }
            // Set-up, embedding and the first norm of a row all run on the CTA that owns the row, so only
            // CTA-wide barriers separate them: one grid barrier in front of the first GEMM instead of two.
            setup_phase(p);
            named_bar(2, kWorkThreads);  // the row's position and validity are read back by the embedding
            embed_phase(p);
            named_bar(2, kWorkThreads);  // the embedding rows are read back by the norm
            norm_for_layer(0);
            go = grid_sync(p, sh, epoch);
            if (go && threadIdx.x < 64) {  // lengths and rows of this pass (written by the set-up of every row), for the
                const int b = threadIdx.x;  // attention items, which run behind further grid barriers
                seq_tab[b] = b < p.B ? __ldcg(p.len + b) : 0;
                seq_tab[64 + b] = b < p.B ? __ldcg(p.ri.n_eff + b) : 0;
            }
            for (int l = 0; l < p.n_layers && go; ++l) {
                run_gemm<NT>(p, gs | (4 * l + 0), smem);                  // qkv
                if (p.parallel) run_gemm<NT>(p, gs | (4 * l + 1), smem);       // MLP in (same block input)
                if (!(go = grid_sync(p, sh, epoch))) break;
                if (overlap_mlp_out(p)) {
                    act_phase(p);
                    if ((int)blockIdx.x < attention_ctas(p)) {
                        grid_arrive(p, sh, epoch);  // the activation is out; attention needs nothing from the others
                        attention_phase(p, l, attn_scratch, sh);
                        attn_signal(p, sh);
                    } else {
                        if (!(go = grid_sync(p, sh, epoch))) break;
                        run_gemm<NT>(p, gs | (4 * l + 2), smem);               // MLP out -> x, beside the attention items
                        run_gemm<NT>(p, gs | (4 * l + 3), smem);               // out-proj -> x, once the attention CTAs have signalled
                    }
                    if (!(go = grid_sync(p, sh, epoch))) break;
                } else if (p.parallel) {
                    attention_phase(p, l, attn_scratch, sh);
                    act_phase(p);
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    run_gemm<NT>(p, gs | (4 * l + 2), smem);                   // out-proj -> x
                    run_gemm<NT>(p, gs | (4 * l + 3), smem);                   // MLP out  -> x
                    if (!(go = grid_sync(p, sh, epoch))) break;
                } else {
                    attention_phase(p, l, attn_scratch, sh);
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    run_gemm<NT>(p, gs | (4 * l + 1), smem);                   // out-proj -> x
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    const float *const *lt = staged_ltab(sh);
                    const LayerDesc *ld = layer_desc(p.md, l);
                    norm_phase(p, lt ? lt[8 * l + 4] : ld->ln2_g, lt ? lt[8 * l + 5] : ld->ln2_b, OP_XN1, nullptr, nullptr, 0, red);
                    grid_zero(p.t_in, p.R, p.d_in, p.d_in);
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    run_gemm<NT>(p, gs | (4 * l + 2), smem);                   // MLP in
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    act_phase(p);
                    if (!(go = grid_sync(p, sh, epoch))) break;
                    run_gemm<NT>(p, gs | (4 * l + 3), smem);                   // MLP out -> x
                    if (!(go = grid_sync(p, sh, epoch))) break;
                }
                norm_for_layer(l + 1);
                if (!(go = grid_sync(p, sh, epoch))) break;
            }
            if (go && p.want_logits) run_gemm<NT>(p, gs | (4 * p.n_layers), smem);
            if (go && p.tail) {  // q, the draw and the commit of this step (see tail_partial)
                if (!(go = grid_sync(p, sh, epoch))) break;
                tail_partial(p, sh);
                if (!(go = grid_sync(p, sh, epoch))) break;
                tail_q(p, sh);
                if (!(go = grid_sync(p, sh, epoch))) break;
                tail_draw(p);
                if (!(go = grid_sync(p, sh, epoch))) break;
                tail_commit(p);
                if (!(go = grid_sync(p, sh, epoch))) break;
            }
        }
        if (go && p.tail && p.mailbox && blockIdx.x == 0 && threadIdx.x == 0) {  // the host's length bound follows (see report_max_len)
            int m = 0;
            for (int b = 0; b < p.B; ++b) m = max(m, __ldcg(p.len_rw + b));
            *reinterpret_cast<volatile unsigned long long *>(p.mailbox) = ((unsigned long long)p.mb_seq << 32) | (unsigned)m;
        }
        if (p.trace && blockIdx.x == 0 && threadIdx.x == 0) {
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            p.trace[epoch + 1] = t;
            p.trace[epoch + 2] = 0;
        }
        if (warp == kXWarp && lane == 0 && sh->abort) {  // error path only: copies still in flight
            const RingPos rp = role_rp[1];
            for (int s = 0; s < S; ++s)
                if ((rp.used >> s) & 1u) mbar_wait(&fullX[s], ((rp.par >> s) & 1u) ^ 1u);
        }
        if (warp == kMmaWarp) {  // nothing of this CTA may still be running on the tensor core
            if (lane == 0) {
                tc_commit(mmaDone);
                mbar_wait(mmaDone, 0);
            }
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
    }
}

}  // namespace ssd

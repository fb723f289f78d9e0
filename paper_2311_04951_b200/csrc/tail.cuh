// Vocabulary-wide tail of a step: temperature softmax statistics, the accept / reject scan,
// residual renormalise-and-resample or bonus draw, and the draft's "sample from q, export q".
// (Section "Speculative Sampling", Figure 2: the target model passes or refuses each draft token in
// turn and generates one token itself.)  No host round-trip: everything a decision
// needs stays on the device; reductions use warp shuffles, prefix sums run in fp64.
//
// One row of the vocabulary is worked on by a thread-block cluster of kTailCluster CTAs (one SM alone
// is issue- and latency-bound on a 50 K-entry row: ncu shows 52 % issue slots busy on the statistics
// and long-scoreboard stalls of 18 per issue on the draw).  CTA `rank` owns a contiguous slice of the
// row; block results are published in shared memory and read by the other CTAs of the cluster through
// distributed shared memory, always combined in rank order so that sums keep the index order.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace ssd {

namespace cg = cooperative_groups;

constexpr int kTailThreads = 1024;
constexpr int kTailCluster = 8;

// What a CTA publishes to its cluster.  Every exchange uses slots of its own, so one cluster barrier
// per exchange suffices; a kernel ends with a cluster barrier (nobody leaves while its slots are read).
struct ClusterSlots {
    float v[2];
    int i[6];
    double d[4];
};

// CTA `rank`'s slice [lo, hi) of a row of V entries: whole rows of 32 indices, split evenly.
__device__ __forceinline__ void tail_slice(int V, int rank, int &lo, int &hi) {
    const int rows = (V + 31) >> 5, per = (rows + kTailCluster - 1) / kTailCluster;
    lo = min(V, rank * per * 32);
    hi = min(V, lo + per * 32);
}

struct RowStat {
    float mx;      // max logit of the row
    float z;       // sum exp((l - mx) / T)
    int32_t amax;  // argmax (lowest index among maxima)
    int32_t pad;
};

// p_j of a row from its statistics; the one place this is computed, so the rows exported for
// inspection are bit-identical to the rows the decisions use.
__device__ __forceinline__ float prob_of(float logit, const RowStat &st, float inv_t, int j) {
    if (inv_t == 0.f) return j == st.amax ? 1.f : 0.f;  // greedy: one-hot at the argmax
    return expf((logit - st.mx) * inv_t) / st.z;
}

// Restriction of a row to its most probable tokens (top-k, then top-p on what top-k kept): token j stays iff
// its probability is >= thr, and the kept ones are divided by their mass.  mass == 0 means "no restriction".
struct RowFilter {
    float thr;
    float mass;
};
__device__ __forceinline__ float prob_f(float logit, const RowStat &st, const RowFilter &f, float inv_t, int j) {
    const float pr = prob_of(logit, st, inv_t, j);
    if (f.mass == 0.f || inv_t == 0.f) return pr;  // (a one-hot row is its own restriction)
    return pr >= f.thr ? pr / f.mass : 0.f;
}

// Block-wide (max, lowest index of max).
__device__ __forceinline__ void block_argmax(float v, int idx, float *sv, int *si, float &out_v, int &out_i) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, v, o);
        int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
    }
    __syncthreads();
    if (lane == 0) { sv[w] = v; si[w] = idx; }
    __syncthreads();
    if (w == 0) {
        v = lane < nw ? sv[lane] : -INFINITY;
        idx = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, v, o);
            int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        }
        if (lane == 0) { sv[0] = v; si[0] = idx; }
    }
    __syncthreads();
    out_v = sv[0];
    out_i = si[0];
}

// Row statistics of logits[row, :] by the whole cluster; every thread of every CTA returns the same RowStat.
__device__ __forceinline__ RowStat row_stats(const float *logits, int V, float inv_t, float *sv, int *si, double *sd,
                                             ClusterSlots *pub, cg::cluster_group &cl) {
    const int rank = (int)cl.block_rank();
    int lo, hi;
    tail_slice(V, rank, lo, hi);
    float mx = -INFINITY;
    int am = 0x7fffffff;
    // eight loads in flight per thread: the row comes from L2, and one latency per element is the whole cost
    for (int j0 = lo + threadIdx.x; j0 < hi; j0 += 8 * blockDim.x) {
        float l[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * blockDim.x;
            l[u] = j < hi ? __ldcg(logits + j) : -INFINITY;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (l[u] > mx) { mx = l[u]; am = j0 + u * blockDim.x; }  // strided ascending: first maximum per thread
    }
    float bmx;
    int bam;
    block_argmax(mx, am, sv, si, bmx, bam);
    if (threadIdx.x == 0) { pub->v[0] = bmx; pub->i[0] = bam; }
    cl.sync();
    RowStat st;
    st.mx = -INFINITY;
    st.amax = 0x7fffffff;
    for (int r = 0; r < kTailCluster; ++r) {  // lowest index among the maxima
        const ClusterSlots *o = cl.map_shared_rank(pub, r);
        const float v = o->v[0];
        const int i = o->i[0];
        if (v > st.mx || (v == st.mx && i < st.amax)) { st.mx = v; st.amax = i; }
    }
    double z = 0.0;
    if (inv_t != 0.f) {
        float part = 0.f;
        for (int j0 = lo + threadIdx.x; j0 < hi; j0 += 8 * blockDim.x) {
            float l[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u * blockDim.x;
                l[u] = j < hi ? __ldcg(logits + j) : -INFINITY;  // exp(-inf) = 0
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) part += expf((l[u] - st.mx) * inv_t);
        }
        const double zb = block_sum((double)part, sd);
        if (threadIdx.x == 0) pub->d[0] = zb;
        cl.sync();
        for (int r = 0; r < kTailCluster; ++r) z += cl.map_shared_rank(pub, r)->d[0];
    }
    st.z = (float)z;
    st.pad = 0;
    return st;
}

// Shared memory of the threshold search below.
struct FilterSmem {
    unsigned cnt[256];
    double mass[256];
    unsigned tot_cnt[256];
    double tot_mass[256];
    unsigned sel, cnt_above;
    double mass_above, total;
};

// The threshold of a restriction, by the whole cluster: the largest probability value t such that the tokens
// with p >= t (p >= lo only are looked at) number at least want_cnt (by_mass false) or weigh at least want_mass
// (by_mass true); if no t reaches it, the smallest value present.  Tokens equal to the threshold all stay.  A
// radix search over the fp32 bit pattern (probabilities are >= 0, so the patterns order like the values): four
// passes of eight bits, each a 256-bin histogram of counts and masses of the tokens that match the bits fixed
// so far, summed over the CTAs in rank order through distributed shared memory; the bins are walked from the
// top.  Returns the threshold and, through *kept_mass, the mass at or above it (fp64 sums; the walk order
// differs from a sorted running sum only in rounding).  The same result in every thread of the cluster.
template <typename ProbFn>
__device__ __forceinline__ float select_threshold(ProbFn prob, int V, float lo, bool by_mass, unsigned want_cnt,
                                                  double want_frac, FilterSmem *fs, cg::cluster_group &cl,
                                                  double *kept_mass) {
    const int rank = (int)cl.block_rank();
    int lo_i, hi_i;
    tail_slice(V, rank, lo_i, hi_i);
    unsigned prefix = 0;
    int nb = 0;
    double want_mass = 0.0;
    if (threadIdx.x == 0) { fs->cnt_above = 0; fs->mass_above = 0.0; }
    for (int pass = 0; pass < 4; ++pass) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) { fs->cnt[i] = 0; fs->mass[i] = 0.0; }
        __syncthreads();
        for (int j = lo_i + threadIdx.x; j < hi_i; j += blockDim.x) {
            const float pr = prob(j);
            const unsigned bits = __float_as_uint(pr);
            if (pr >= lo && (nb == 0 || (bits >> (32 - nb)) == prefix)) {
                const unsigned bin = (bits >> (24 - nb)) & 255u;
                atomicAdd(&fs->cnt[bin], 1u);
                atomicAdd(&fs->mass[bin], (double)pr);
            }
        }
        __syncthreads();
        cl.sync();  // every CTA's histogram is complete
        for (int i = threadIdx.x; i < 256; i += blockDim.x) {
            unsigned c = 0;
            double m = 0.0;
            for (int r = 0; r < kTailCluster; ++r) {
                const FilterSmem *o = cl.map_shared_rank(fs, r);
                c += o->cnt[i];
                m += o->mass[i];
            }
            fs->tot_cnt[i] = c;
            fs->tot_mass[i] = m;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            if (pass == 0) {  // the mass of everything looked at: the base of a mass target
                double t = 0.0;
                for (int i = 255; i >= 0; --i) t += fs->tot_mass[i];
                fs->total = t;
            }
            const double target = want_frac * fs->total;
            unsigned c = fs->cnt_above;
            double m = fs->mass_above;
            int sel = -1, lowest = -1;
            for (int i = 255; i >= 0; --i) {
                if (fs->tot_cnt[i] == 0) continue;
                lowest = i;
                const bool met = by_mass ? (m + fs->tot_mass[i] >= target) : (c + fs->tot_cnt[i] >= want_cnt);
                if (met) { sel = i; break; }
                c += fs->tot_cnt[i];
                m += fs->tot_mass[i];
            }
            if (sel < 0) {  // the target lies beyond everything there is: keep all (back off the last bin's sums)
                sel = lowest < 0 ? 0 : lowest;
                if (lowest >= 0) { c -= fs->tot_cnt[sel]; m -= fs->tot_mass[sel]; }
            }
            fs->sel = (unsigned)sel;
            fs->cnt_above = c;
            fs->mass_above = m;
        }
        __syncthreads();
        prefix = (prefix << 8) | fs->sel;
        nb += 8;
        want_mass = fs->mass_above + fs->tot_mass[fs->sel];
        cl.sync();  // all remote reads of this pass are done before the histograms are cleared
    }
    *kept_mass = want_mass;
    return __uint_as_float(prefix);
}

// The restriction of a row (top_k tokens, then the top_p nucleus of those), by the whole cluster.
__device__ __forceinline__ RowFilter row_filter(const float *logits, int V, const RowStat &st, float inv_t, int top_k,
                                                float top_p, FilterSmem *fs, cg::cluster_group &cl) {
    RowFilter f;
    f.thr = 0.f;
    f.mass = 0.f;
    const bool use_k = top_k > 0 && top_k < V, use_p = top_p > 0.f && top_p < 1.f;
    if (inv_t == 0.f || (!use_k && !use_p)) return f;
    auto prob = [&](int j) { return prob_of(__ldcg(logits + j), st, inv_t, j); };
    double mass = 0.0;
    float thr = 0.f;
    if (use_k) thr = select_threshold(prob, V, 0.f, false, (unsigned)top_k, 0.0, fs, cl, &mass);
    if (use_p) thr = select_threshold(prob, V, thr, true, 0u, (double)top_p, fs, cl, &mass);
    f.thr = thr;
    f.mass = (float)mass;
    return f;
}

// Inverse-CDF draw over V weights w(j) >= 0 by the whole cluster: the smallest j whose inclusive prefix
// sum exceeds u * S; prefix sums in index order, fp64.  If rounding leaves none: the largest j with
// w > 0.  Each CTA owns a slice, each thread a contiguous segment of it, so the prefix order is the
// index order: thread sums are scanned inside the CTA, CTA totals in rank order across the cluster.
// `slot` (0 or 1) selects the exchange slots, so that two draws in one kernel need no extra barrier.
// Returns S via *total; S and the drawn index are the same in every thread of the cluster.  S <= 0
// returns -1.
template <typename WeightFn>
__device__ __forceinline__ int inv_cdf_cluster(WeightFn w, int V, float u, double *sd, int *si, double *total,
                                               ClusterSlots *pub, cg::cluster_group &cl, int slot) {
    const int rank = (int)cl.block_rank();
    int lo, hi;
    tail_slice(V, rank, lo, hi);
    const int seg = (hi - lo + (int)blockDim.x - 1) / (int)blockDim.x;
    const int j0 = min(hi, lo + (int)threadIdx.x * seg), j1 = min(hi, j0 + seg);
    double local = 0.0;
    int last_pos = -1;
    for (int j = j0; j < j1; ++j) {
        float wj = w(j);
        local += (double)wj;
        if (wj > 0.f) last_pos = j;
    }
    // exclusive scan of the per-thread sums over the block (warp scan + scan of warp totals)
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) sd[wid] = incl;
    if (threadIdx.x == 0) { si[0] = 0x7fffffff; si[1] = -1; }
    __syncthreads();
    double warp_off = 0.0, T = 0.0;
    for (int k = 0; k < nw; ++k) {  // nw <= 32: short serial pass keeps the order fixed
        double t = sd[k];
        if (k < wid) warp_off += t;
        T += t;
    }
    if (threadIdx.x == 0) pub->d[1 + slot] = T;
    cl.sync();
    double cta_off = 0.0, S = 0.0;
    for (int r = 0; r < kTailCluster; ++r) {
        const double t = cl.map_shared_rank(pub, r)->d[1 + slot];
        if (r < rank) cta_off += t;
        S += t;
    }
    *total = S;
    if (!(S > 0.0)) return -1;  // the same decision in every CTA of the cluster
    const double target = (double)u * S;
    double run = cta_off + warp_off + (incl - local);
    int hit = 0x7fffffff;
    if (run + local > target || run > target) {
        for (int j = j0; j < j1; ++j) {
            const float wj = w(j);
            run += (double)wj;
            if (wj > 0.f && run > target) { hit = j; break; }  // a zero-weight index is never drawn
        }
    }
    if (hit != 0x7fffffff) atomicMin(&si[0], hit);
    if (last_pos >= 0) atomicMax(&si[1], last_pos);
    __syncthreads();
    if (threadIdx.x == 0) { pub->i[1 + 2 * slot] = si[0]; pub->i[2 + 2 * slot] = si[1]; }
    cl.sync();
    int first = 0x7fffffff, last = -1;
    for (int r = 0; r < kTailCluster; ++r) {
        const ClusterSlots *o = cl.map_shared_rank(pub, r);
        first = min(first, o->i[1 + 2 * slot]);
        last = max(last, o->i[2 + 2 * slot]);
    }
    return first != 0x7fffffff ? first : last;
}

struct VerifyArgs {
    const float *logits;    // [B, K+1, V]
    int K, V;
    const int32_t *rows;    // [B, K+1]: pending, x~_1..x~_K
    const float *q;         // [B, K, V]
    const float *u;         // [B, K+1]
    float inv_t;            // 1/T, 0 = greedy
    int32_t *n_accepted;    // [B]
    int32_t *next_token;
    int next_stride;
    float *p_debug;         // [B, K+1, V] or null
    int32_t *keep;          // [B] or null: n_accepted + 1 for kv_commit
    RowStat *stats;         // scratch [B, K+1]
    RowFilter *filt;        // scratch [B, K+1]
    int top_k;              // restriction of the target rows (0 / 1.0: none); q arrives already restricted
    float top_p;
};

// grid (kTailCluster (K+1), B), one cluster per row: statistics of every row (+ optional export of the p row)
__global__ void __cluster_dims__(kTailCluster, 1, 1) __launch_bounds__(kTailThreads) row_stats_kernel(VerifyArgs a) {
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ double sd[32];
    __shared__ ClusterSlots pub;
    __shared__ FilterSmem fs;
    cg::cluster_group cl = cg::this_cluster();
    const int i = blockIdx.x / kTailCluster, b = blockIdx.y;
    const float *lg = a.logits + ((size_t)b * (a.K + 1) + i) * a.V;
    RowStat st = row_stats(lg, a.V, a.inv_t, sv, si, sd, &pub, cl);
    const RowFilter fl = row_filter(lg, a.V, st, a.inv_t, a.filt ? a.top_k : 0, a.top_p, &fs, cl);  // (no room for it: no restriction)
    if (cl.block_rank() == 0 && threadIdx.x == 0) {
        a.stats[b * (a.K + 1) + i] = st;
        if (a.filt) a.filt[b * (a.K + 1) + i] = fl;
    }
    if (a.p_debug) {
        int lo, hi;
        tail_slice(a.V, (int)cl.block_rank(), lo, hi);
        float *p = a.p_debug + ((size_t)b * (a.K + 1) + i) * a.V;
        for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) p[j] = prob_f(lg[j], st, fl, a.inv_t, j);
    }
    cl.sync();
}

// grid (kTailCluster B), one cluster per sequence: accept scan, then residual / bonus draw
__global__ void __cluster_dims__(kTailCluster, 1, 1) __launch_bounds__(kTailThreads) verify_kernel(VerifyArgs a) {
    __shared__ double sd[32];
    __shared__ int si[32];
    __shared__ int s_acc;
    __shared__ ClusterSlots pub;
    cg::cluster_group cl = cg::this_cluster();
    const int b = blockIdx.x / kTailCluster, K = a.K, V = a.V;
    const RowStat *st = a.stats + b * (K + 1);
    const RowFilter none = {0.f, 0.f};
    if (threadIdx.x == 0) {  // (every CTA of the cluster takes the same few steps)
        int acc = 0;
        for (int i = 0; i < K; ++i) {
            int x = a.rows[b * (K + 1) + 1 + i];
            x = max(0, min(x, V - 1));
            const float px = prob_f(a.logits[((size_t)b * (K + 1) + i) * V + x], st[i], a.filt ? a.filt[b * (K + 1) + i] : none, a.inv_t, x);
            const float qx = a.q[((size_t)b * K + i) * V + x];
            // accept with probability min(1, p/q): u * q < p, one fp32 rounding of the product
            if (__fmul_rn(a.u[b * (K + 1) + i], qx) < px) ++acc; else break;
        }
        s_acc = acc;
    }
    __syncthreads();
    const int acc = s_acc;
    const float *lg = a.logits + ((size_t)b * (K + 1) + acc) * V;
    const RowStat rs = st[acc];
    const RowFilter rf = a.filt ? a.filt[b * (K + 1) + acc] : none;
    const float u = a.u[b * (K + 1) + K];
    const float inv_t = a.inv_t;
    double S;
    int y = -1;
    if (acc < K) {
        const float *qr = a.q + ((size_t)b * K + acc) * V;
        y = inv_cdf_cluster([&](int j) { return fmaxf(0.f, __fsub_rn(prob_f(lg[j], rs, rf, inv_t, j), qr[j])); }, V, u,
                            sd, si, &S, &pub, cl, 0);
    }
    if (y < 0)  // all accepted: bonus from p_{K+1}; or an all-zero residual: fall back to p
        y = inv_cdf_cluster([&](int j) { return prob_f(lg[j], rs, rf, inv_t, j); }, V, u, sd, si, &S, &pub, cl, 1);
    if (y < 0) y = rs.amax;  // a row whose probabilities all vanished (non-finite logits)
    if (cl.block_rank() == 0 && threadIdx.x == 0) {
        a.n_accepted[b] = acc;
        a.next_token[(size_t)b * a.next_stride] = y;
        if (a.keep) a.keep[b] = acc + 1;
    }
    cl.sync();
}

struct DraftTailArgs {
    const float *logits;  // [B, M, V] rows of the draft forward
    int M, V;
    const int32_t *n_eff; // [B] rows fed per sequence (the last one is sampled)
    float inv_t;
    const float *u; int u_stride;
    int32_t *token_out; int token_stride;
    float *q_out; size_t q_stride;
    int top_k;            // restriction of q (0 / 1.0: none)
    float top_p;
};

// grid (kTailCluster B), one cluster per sequence: q = softmax(last row / T), exported; x~ = inverse-CDF(q, u)
__global__ void __cluster_dims__(kTailCluster, 1, 1) __launch_bounds__(kTailThreads) draft_tail_kernel(DraftTailArgs a) {
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ double sd[32];
    __shared__ ClusterSlots pub;
    __shared__ FilterSmem fs;
    cg::cluster_group cl = cg::this_cluster();
    const int b = blockIdx.x / kTailCluster;
    int row = a.n_eff[b] - 1;
    if (row < 0) row = 0;
    const float *lg = a.logits + ((size_t)b * a.M + row) * a.V;
    const RowStat st = row_stats(lg, a.V, a.inv_t, sv, si, sd, &pub, cl);
    const RowFilter fl = row_filter(lg, a.V, st, a.inv_t, a.top_k, a.top_p, &fs, cl);
    float *q = a.q_out + (size_t)b * a.q_stride;
    int lo, hi;
    tail_slice(a.V, (int)cl.block_rank(), lo, hi);
    for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) q[j] = prob_f(lg[j], st, fl, a.inv_t, j);
    __syncthreads();  // the draw below reads this CTA's own slice of q
    double S;
    int y = inv_cdf_cluster([&](int j) { return q[j]; }, a.V, a.u[(size_t)b * a.u_stride], sd, si, &S, &pub, cl, 0);
    if (y < 0) y = st.amax;
    if (cl.block_rank() == 0 && threadIdx.x == 0) a.token_out[(size_t)b * a.token_stride] = y;
    cl.sync();
}

// ---------------- cache length bookkeeping ----------------
// Every kernel that changes the committed lengths runs as ONE block of 64 threads (at most 64 sequences)
// and afterwards reports the largest length to the host through a word of mapped host memory, tagged with
// the host's sequence number of the operation: (seq << 32) | max length.  The host plans attention splits
// from an upper bound of the lengths; with this word the bound follows the real lengths without a
// synchronisation (it adds what the operations queued behind `seq` can add at most).
__device__ __forceinline__ void report_max_len(int my_len, unsigned long long *mailbox, unsigned seq) {
    __shared__ int s_max[2];
    int v = my_len;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0 && mailbox) {
        const unsigned m = (unsigned)max(s_max[0], s_max[1]);
        *reinterpret_cast<volatile unsigned long long *>(mailbox) = ((unsigned long long)seq << 32) | m;
    }
}
// Keep n_keep[b] more rows.  A length that would pass the capacity S is clamped and recorded as
// SSD_E_CAPACITY in the sticky status word: rows that no forward wrote must not become context.
__global__ void kv_commit_kernel(int32_t *len, const int32_t *n_keep, int B, int S, int32_t *status,
                                 unsigned long long *mailbox, unsigned seq) {
    const int b = threadIdx.x;
    int v = 0;
    if (b < B) {
        v = len[b] + max(0, n_keep[b]);
        if (v > S) {
            v = S;
            set_status(status, -3);
        }
        len[b] = v;
    }
    report_max_len(v, mailbox, seq);
}
__global__ void kv_commit_rows_kernel(int32_t *len, const int32_t *n_eff, int B, unsigned long long *mailbox,
                                      unsigned seq) {
    const int b = threadIdx.x;
    int v = 0;
    if (b < B) {
        v = len[b] + n_eff[b];   // n_eff is what the forward's set-up found to fit
        len[b] = v;
    }
    report_max_len(v, mailbox, seq);
}
__global__ void kv_rollback_kernel(int32_t *len, const int32_t *new_len, int B, unsigned long long *mailbox,
                                   unsigned seq) {
    const int b = threadIdx.x;
    int v = 0;
    if (b < B) {
        v = max(0, min(len[b], new_len[b]));
        len[b] = v;
    }
    report_max_len(v, mailbox, seq);
}
// chunk c of a prompt pass: rows fed per sequence = clamp(n_tokens - c*C, 0, C)
__global__ void prefill_rows_kernel(const int32_t *n_tokens, int chunk, int C, int32_t *n_rows, int B) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) n_rows[b] = max(0, min(C, n_tokens[b] - chunk * C));
}

struct AdvanceArgs {
    int32_t *tlen, *dlen;  // target / draft committed lengths (dlen may be null)
    int32_t *rows;         // [B, K+1]
    int K, B;
    const int32_t *n_accepted, *next_token;
    int next_stride;
    int32_t *out_tokens; int out_cap; int32_t *out_count;
    int32_t *draft_in, *draft_n_in;
    unsigned long long *t_mailbox, *d_mailbox;  // see report_max_len
    unsigned t_seq, d_seq;
};

__device__ __forceinline__ void spec_advance_one(const AdvanceArgs &a, int b, int &t_new, int &d_new) {
    const int K = a.K;
    int acc = max(0, min(a.n_accepted[b], K));
    const int y = a.next_token[(size_t)b * a.next_stride];
    int32_t *row = a.rows + (size_t)b * (K + 1);
    const int n = a.tlen[b] + 1;  // committed tokens before this iteration
    if (a.out_tokens && a.out_count) {
        int c = a.out_count[b];
        for (int i = 0; i < acc; ++i, ++c)
            if (c < a.out_cap) a.out_tokens[(size_t)b * a.out_cap + c] = row[1 + i];
        if (c < a.out_cap) a.out_tokens[(size_t)b * a.out_cap + c] = y;
        a.out_count[b] = c + 1;
    } else if (a.out_count) {
        a.out_count[b] += acc + 1;
    }
    if (a.draft_in && a.draft_n_in) {
        if (acc == K && K > 0) {
            a.draft_in[2 * b] = row[K];
            a.draft_in[2 * b + 1] = y;
            a.draft_n_in[b] = 2;
        } else {
            a.draft_in[2 * b] = y;
            a.draft_in[2 * b + 1] = y;
            a.draft_n_in[b] = 1;
        }
    }
    t_new = a.tlen[b] + acc + 1;
    a.tlen[b] = t_new;
    if (a.dlen) {
        d_new = min(a.dlen[b], K > 0 ? min(n + acc, n + K - 1) : n + acc);
        a.dlen[b] = d_new;
    }
    row[0] = y;
}
__global__ void spec_advance_kernel(AdvanceArgs a) {  // one block of 64 threads
    const int b = threadIdx.x;
    int t_new = 0, d_new = 0;
    if (b < a.B) spec_advance_one(a, b, t_new, d_new);
    report_max_len(t_new, a.t_mailbox, a.t_seq);
    __syncthreads();  // the exchange slots are reused
    report_max_len(d_new, a.d_mailbox, a.d_seq);
}

}  // namespace ssd

// Included by persistent.cuh inside namespace ssd (it uses that file's parameter block, staged tables and helpers).
#pragma once

// ---- attention of up to eight query rows on warp-level MMAs, hi and lo in one tile -------------------
// The 16-row MMA tile has room for eight query rows twice: rows 0-7 carry the bf16 hi parts of the queries (and,
// in the second product, of the probabilities), rows 8-15 the lo parts, so ONE m16n8k16 step yields both terms
// and the thread that holds accumulator row g also holds row g + 8: hi + lo is an add in registers.  That is half
// the MMAs of attention_item for passes of at most eight rows - and on this part the legacy MMA rate (about one
// m16n8k16 per seven cycles per SM) is what bounds that form.  The rest follows the FP32 items: nothing is shared
// inside the loop.  A warp owns every eighth block of 16 positions; its K and V rows (8 KB) arrive by cp.async in
// a ring of two stages private to the warp, 16-byte pieces swizzled by the row so that ldmatrix reads them without
// bank conflicts; S = Q K^T (16 MMAs), running maximum / sum per row in the four threads that hold the row (the
// maximum is raised only past a slack of 2^8, so the output is rarely rescaled), P packed as hi / lo rows straight
// from the score registers (no exchange between threads), O += P V (16 MMAs).  The rows of the pass come from qkv
// (rotary, cache rounding) as one more block of warp 0; the split that owns them appends them to the cache.  The
// eight warps meet once, in shared memory (over the stages), at the end.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
constexpr int kM8Rows = 8, kM8Block = 16;             // query rows per item; positions per block
constexpr int kM8Slack = 8;
// bytes of a tile row in shared memory: the head's bf16 row padded to a power of two, so that the 16-byte pieces can be swizzled
__host__ __device__ constexpr int m8_row_bytes(int Dh) { return Dh <= 32 ? 64 : Dh <= 64 ? 128 : 256; }
__host__ __device__ constexpr int m8_stage_bytes(int Dh) { return 2 * kM8Block * m8_row_bytes(Dh); }   // K rows, then V rows
// stages of a warp's ring: two 8 KB stages at head 128; narrower heads take more of them for the same bytes on their way
__host__ __device__ constexpr int m8_stages(int Dh) { return Dh <= 64 ? 4 : 2; }
__host__ __device__ constexpr int m8_scratch_bytes(int Dh) {
    // two stages per warp (the warps' (max, sum, output) lie over them at the end), then the staged queries
    // ... then the staged queries (one tile) and the block of the pass's own rows (a K tile and a V tile)
    return 8 * m8_stages(Dh) * m8_stage_bytes(Dh) + 16 * m8_row_bytes(Dh) + m8_stage_bytes(Dh);
}

template <int DH>
__device__ __noinline__ void attention_item_mma8(const FwdParams &p, int layer, int item, uint8_t *scratch, Shared *sh) {
    constexpr int NK = DH / 16, ND = DH / 8, ROWB = m8_row_bytes(DH), GPR = DH / 8;  // k-steps; 8-column tiles; bytes of a tile row; 16-byte pieces of a head row
    static_assert(DH % 16 == 0 && DH <= 128 && ND % 2 == 0, "head dims that are multiples of 16");
    constexpr int STAGE = m8_stage_bytes(DH), NS = m8_stages(DH);
    const int split = item % p.n_split, bh = item / p.n_split, b = bh / p.H, h = bh % p.H;
    const int d = p.d;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int n_rows = staged_len(sh)[64 + b];
    const int len = staged_len(sh)[b];
    const int r0 = b * p.M;
    const int chunk = split_chunk(p, len + n_rows, kAttnTile);
    const int p_begin = split * chunk;
    const int p_end = min(p_begin + chunk, len + n_rows);
    const int c1 = min(p_end, len);                      // cached positions of this split: [p_begin, c1)
    const int nb = c1 > p_begin ? (c1 - p_begin + kM8Block - 1) / kM8Block : 0;
    const float sc = p.attn_scale * 1.4426950408889634f;  // scores in log2 units
    __nv_bfloat16 *kc = (__nv_bfloat16 *)(p.cache + (size_t)layer * p.layer_bytes) + ((size_t)(b * 2) * p.H + h) * p.S * DH;
    __nv_bfloat16 *vc = kc + (size_t)p.H * p.S * DH;
    uint8_t *wst = scratch + (size_t)warp * (NS * STAGE);   // this warp's stages
    // piece c of row r of a tile sits at r * ROWB + ((c ^ (r & 7)) << 4)
    // a lane copies 16-byte piece lc of rows lr, lr + RPI, ... of a block's K and V tiles
    static_assert((GPR & (GPR - 1)) == 0, "pieces per row: a power of two");
    constexpr int RPI = 32 / GPR;
    const int lr = lane / GPR, lc = lane % GPR;
    const uint32_t wst_u = smem_u32(wst) + (uint32_t)(lr * ROWB);
    auto issue = [&](int i) {  // block warp + 8 i of this warp into stage i % NS
        const int blk = warp + 8 * i, pos0 = p_begin + blk * kM8Block + lr;
        const uint32_t st = wst_u + (uint32_t)((i % NS) * STAGE);
        const size_t off0 = (size_t)pos0 * DH + lc * 8;
#pragma unroll 4
        for (int it = 0; it < kM8Block / RPI; ++it) {
            const int r = it * RPI + lr;
            const bool in = blk < nb && pos0 + it * RPI < c1;
            const size_t off = in ? off0 + (size_t)it * RPI * DH : 0;
            const uint32_t so = st + (uint32_t)(it * RPI * ROWB + ((lc ^ (r & 7)) << 4));
            const uint32_t nbytes = in ? 16u : 0u;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(so), "l"(kc + off), "r"(nbytes) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(so + kM8Block * ROWB), "l"(vc + off), "r"(nbytes) : "memory");
        }
        cp_async_commit();
    };
    const int my_blocks = nb > warp ? (nb - warp + 7) / 8 : 0;
#pragma unroll
    for (int i = 0; i < NS - 1; ++i) issue(i);

    // ---- the queries (rotary applied, in log2 units), staged once behind the stages as the MMA's A tile: row r
    //      as bf16 hi in tile row r, lo in tile row r + 8, pieces swizzled like the K / V tiles ----
    uint8_t *q_t = scratch + 8 * NS * STAGE;  // [16][DH] bf16
    for (int i = tid; i < kM8Rows * GPR; i += kAttnThreadsP) {
        const int r = i / GPR, c = i % GPR;
        float q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) q[u] = 0.f;
        if (r < n_rows) rope_vec8(p, p.qkv + (size_t)(r0 + r) * 3 * d + h * DH, r0 + r, c * 8, q);
        uint32_t hw[4], lw4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float x0 = q[2 * u] * sc, x1 = q[2 * u + 1] * sc;
            const __nv_bfloat162 hv = __floats2bfloat162_rn(x0, x1);
            hw[u] = *reinterpret_cast<const uint32_t *>(&hv);
            lw4[u] = pack_bf16x2(x0 - __low2float(hv), x1 - __high2float(hv));
        }
        const uint32_t so = (uint32_t)((c ^ (r & 7)) << 4);  // (r + 8) & 7 == r & 7
        *reinterpret_cast<uint4 *>(q_t + r * ROWB + so) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        *reinterpret_cast<uint4 *>(q_t + (r + 8) * ROWB + so) = make_uint4(lw4[0], lw4[1], lw4[2], lw4[3]);
    }
    // ---- the rows of this pass inside this split, as one more block (a K tile, a V tile) behind the query tile:
    //      every thread builds one or two 16-byte pieces (rotary, cache rounding); the split that owns the rows
    //      appends them to the cache ----
    uint8_t *n_t = q_t + 16 * ROWB;
    const bool has_new = p_end > len && p_end > p_begin;
    const int first = max(p_begin, len) - len;                              // first new row of this split
    const int cnt = has_new ? min(p_end - len, n_rows) - first : 0;         // new rows here (at most 8)
    if (has_new) {
        for (int i = tid; i < 2 * kM8Block * GPR; i += kAttnThreadsP) {
            const int kv = i / (kM8Block * GPR), j = (i / GPR) % kM8Block, c = i % GPR;
            uint4 w = make_uint4(0, 0, 0, 0);
            if (j < cnt) {
                const int rn = first + j, r = r0 + rn;
                const float *krow = p.qkv + (size_t)r * 3 * d + d + h * DH;
                float x[8];
                if (kv == 0) {
                    rope_vec8(p, krow, r, c * 8, x);
                } else {
                    const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(krow + d + c * 8));
                    const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(krow + d + c * 8 + 4));
                    x[0] = v0.x; x[1] = v0.y; x[2] = v0.z; x[3] = v0.w; x[4] = v1.x; x[5] = v1.y; x[6] = v1.z; x[7] = v1.w;
                }
                w = make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]), pack_bf16x2(x[4], x[5]), pack_bf16x2(x[6], x[7]));
                *reinterpret_cast<uint4 *>((kv ? vc : kc) + (size_t)(len + rn) * DH + c * 8) = w;  // append: exactly one split owns this position
            }
            *reinterpret_cast<uint4 *>(n_t + kv * (kM8Block * ROWB) + j * ROWB + ((c ^ (j & 7)) << 4)) = w;
        }
    }
    named_bar(3, kAttnThreadsP);
    // ldmatrix x4 of the A tile: (rows 0-7, k lo), (rows 8-15, k lo), (rows 0-7, k hi), (rows 8-15, k hi)
    const uint32_t qaddr = smem_u32(q_t) + (uint32_t)((lane & 15) * ROWB);
    const int qrow7 = lane & 7, qhalf = lane >> 4;

    float o[ND][4];
#pragma unroll
    for (int j = 0; j < ND; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;  // of row g (the four threads of a row hold the same maximum)
    // One block of 16 positions in the tile at `st` (K rows, then V rows): vis(j) = position j counts for row g.
    auto update = [&](const uint8_t *st, auto vis) {
        const uint32_t kb = smem_u32(st), vb = kb + kM8Block * ROWB;
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};  // positions 0-7 / 8-15
        {
            // ldmatrix x4: (pos 0-7, k lo), (pos 0-7, k hi), (pos 8-15, k lo), (pos 8-15, k hi)
            const int pr = (lane & 7) + 8 * (lane >> 4), half = (lane >> 3) & 1;
            const uint32_t ka = kb + (uint32_t)pr * ROWB;
#pragma unroll
            for (int ks = 0; ks < NK; ++ks) {
                uint32_t k0, k1, k2, k3, q0, q1, q2, q3;
                ldmatrix_x4(qaddr + (uint32_t)(((2 * ks + qhalf) ^ qrow7) << 4), q0, q1, q2, q3);
                ldmatrix_x4(ka + (uint32_t)(((2 * ks + half) ^ (pr & 7)) << 4), k0, k1, k2, k3);
                mma_bf16(s0, q0, q1, q2, q3, k0, k1);
                mma_bf16(s1, q0, q1, q2, q3, k2, k3);
            }
        }
        // row g: hi part in c0, c1, lo part in c2, c3; positions 2t, 2t + 1 (s0) and 8 + 2t, 9 + 2t (s1)
        float sv[4] = {s0[0] + s0[2], s0[1] + s0[3], s1[0] + s1[2], s1[1] + s1[3]};
        float mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            sv[e] = vis(2 * t + (e & 1) + 8 * (e >> 1)) ? sv[e] : -INFINITY;
            mx = fmaxf(mx, sv[e]);
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = (mx > m_run + (float)kM8Slack || m_run == -INFINITY) ? fmaxf(m_run, mx) : m_run;
        float pv[4] = {0.f, 0.f, 0.f, 0.f};
        if (m_new > -INFINITY) {
            const float f = exp2f(m_run - m_new);  // 0 on the first non-empty block
            if (f != 1.f) {
                l_run *= f;
#pragma unroll
                for (int j = 0; j < ND; ++j) { o[j][0] *= f; o[j][1] *= f; o[j][2] *= f; o[j][3] *= f; }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) pv[e] = exp2f(sv[e] - m_new);
            l_run += (pv[0] + pv[1]) + (pv[2] + pv[3]);  // this thread's positions; the row's four threads are summed at the end
        }
        m_run = m_new;
        // P as the A operand: tile row g = hi, row g + 8 = lo, straight from this thread's registers
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(pv[0], pv[1]), h1 = __floats2bfloat162_rn(pv[2], pv[3]);
        const uint32_t a0 = *reinterpret_cast<const uint32_t *>(&h0), a2 = *reinterpret_cast<const uint32_t *>(&h1);
        const uint32_t a1 = pack_bf16x2(pv[0] - __low2float(h0), pv[1] - __high2float(h0));
        const uint32_t a3 = pack_bf16x2(pv[2] - __low2float(h1), pv[3] - __high2float(h1));
        {
            // ldmatrix x4 trans: lanes 0-15 the 16 positions of column piece 2 j2, lanes 16-31 of piece 2 j2 + 1
            const int pr = lane & 15, hi = lane >> 4;
            const uint32_t va = vb + (uint32_t)pr * ROWB;
#pragma unroll
            for (int j2 = 0; j2 < ND / 2; ++j2) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(va + (uint32_t)(((2 * j2 + hi) ^ (pr & 7)) << 4), b0, b1, b2, b3);
                mma_bf16(o[2 * j2], a0, a1, a2, a3, b0, b1);
                mma_bf16(o[2 * j2 + 1], a0, a1, a2, a3, b2, b3);
            }
        }
    };
    // the block of the pass's own rows: warp 0, first (the order of the blocks does not matter to the running
    // maximum / sum), while the copies of its first cached blocks are on their way
    if (warp == 0 && has_new) update(n_t, [&](int j) { return j < cnt && first + j <= g; });
#pragma unroll 1
    for (int i = 0; i < my_blocks; ++i) {
        __syncwarp();            // every lane is done reading the stage block i - 1 used
        issue(i + NS - 1);
        cp_async_wait<NS - 1>();   // this thread's copies of block i have landed ...
        __syncwarp();            // ... and every other lane's
        const int base = p_begin + (warp + 8 * i) * kM8Block;
        update(wst + (i % NS) * STAGE, [&](int j) { return base + j < c1; });
    }
    cp_async_wait<0>();
    __syncwarp();
    // ---- the four threads of a row, then the eight warps (their partial results lie over the stages) ----
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    named_bar(3, kAttnThreadsP);  // every warp is done with its stages
    float *mw = reinterpret_cast<float *>(scratch);  // [8 warps][8 rows] maxima, then sums, then [8][8][DH] outputs
    float *lw = mw + 64, *ow = lw + 64;
    if (t == 0) {
        mw[warp * 8 + g] = m_run;
        lw[warp * 8 + g] = l_run;
    }
#pragma unroll
    for (int j = 0; j < ND; ++j)
        *reinterpret_cast<float2 *>(ow + ((size_t)warp * 8 + g) * DH + 8 * j + 2 * t) = make_float2(o[j][0] + o[j][2], o[j][1] + o[j][3]);
    named_bar(3, kAttnThreadsP);
    const bool direct = p.n_split == 1;
    constexpr int q4 = DH >> 2;
    const int rows_here = min(kM8Rows, p.M);
    for (int i = tid; i < rows_here * q4; i += kAttnThreadsP) {
        const int r = i / q4, e = (i % q4) * 4;
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < 8; ++w) mx = fmaxf(mx, mw[w * 8 + r]);
        float L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mx > -INFINITY) {
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const float mq = mw[w * 8 + r];
                if (mq > -INFINITY) {
                    const float f = exp2f(mq - mx);
                    const float4 a = *reinterpret_cast<const float4 *>(ow + ((size_t)w * 8 + r) * DH + e);
                    L = fmaf(lw[w * 8 + r], f, L);
                    acc.x = fmaf(a.x, f, acc.x); acc.y = fmaf(a.y, f, acc.y); acc.z = fmaf(a.z, f, acc.z); acc.w = fmaf(a.w, f, acc.w);
                }
            }
        }
        const bool live = r < n_rows && L > 0.f;
        if (!live) acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (direct) {
            const float inv = live ? 1.f / L : 0.f;
            store_ao4(p, r0 + r, h * DH + e, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
        } else {
            const size_t slot = ((size_t)(r0 + r) * p.H + h) * p.n_split + split;
            if (e == 0) {
                p.part_m[slot] = live ? mx : -INFINITY;
                p.part_l[slot] = live ? L : 0.f;
            }
            *reinterpret_cast<float4 *>(p.part_o + slot * DH + e) = acc;
        }
    }
    if (!direct) {
        // ticket: the item that finishes last for this (sequence, head) merges all partials
        __threadfence();
        named_bar(3, kAttnThreadsP);
        if (tid == 0) sh->flag = (atomicAdd(p.tickets + bh, 1u) == (unsigned)(p.n_split - 1));
        named_bar(3, kAttnThreadsP);
        if (sh->flag) {
            __threadfence();
            merge_splits(p, r0, h, DH);
            if (tid == 0) p.tickets[bh] = 0;  // ready for the next layer (a grid barrier lies between)
        }
    }
    named_bar(3, kAttnThreadsP);  // scratch is free for the next item
}

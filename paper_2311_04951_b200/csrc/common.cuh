// Shared device helpers of the verification path: status word, bf16 splitting, reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ssd {

constexpr int kMaxRows = 64;        // rows of one forward (sequences x rows per sequence)
constexpr int kMaxRowsPerSeq = 32;  // K + 1
constexpr int kHeaderInts = 64;     // cache header: [0] status, [1] reserved ..., then len[], keep[]

// Sticky device-side status: first error wins.
__device__ __forceinline__ void set_status(int32_t *status, int32_t code) {
    if (status) atomicCAS(status, 0, code);
}

// An fp32 activation as the sum of two bf16 values (hi = RNE(v), lo = RNE(v - hi)): the tensor
// cores multiply bf16 x bf16 exactly and accumulate in fp32, so W*hi + W*lo reproduces the
// fp32 activation to ~2^-17 relative instead of bf16's 2^-9.
struct Operand {
    float *f32;           // fp32 models: plain fp32 operand [rows, ld]
    __nv_bfloat16 *hi;    // bf16 models: split operand [rows_padded, ld] x 2
    __nv_bfloat16 *lo;
    int ld;
};

__device__ __forceinline__ void store_operand(const Operand &o, int r, int i, float v) {
    size_t idx = (size_t)r * o.ld + i;
    if (o.f32) {
        o.f32[idx] = v;
    } else {
        __nv_bfloat16 h = __float2bfloat16_rn(v);
        o.hi[idx] = h;
        o.lo[idx] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide reductions through shared scratch (>= 32 entries); every thread gets the result.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T *scratch) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[w] = v;
    __syncthreads();
    T t = (threadIdx.x < nw) ? scratch[threadIdx.x] : T(0);
    if (w == 0) {
        t = warp_sum(t);
        if (lane == 0) scratch[0] = t;
    }
    __syncthreads();
    t = scratch[0];
    return t;
}

__device__ __forceinline__ float block_max(float v, float *scratch) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) scratch[w] = v;
    __syncthreads();
    float t = (threadIdx.x < nw) ? scratch[threadIdx.x] : -INFINITY;
    if (w == 0) {
        t = warp_max(t);
        if (lane == 0) scratch[0] = t;
    }
    __syncthreads();
    t = scratch[0];
    return t;
}

// Per-row bookkeeping of one forward, filled by setup_rows_kernel.
struct RowInfo {
    int32_t *seq;    // [R] sequence of row r
    int32_t *pos;    // [R] absolute position of row r (len[seq] + j)
    int32_t *valid;  // [R] 1 if the row is fed (j < n_rows[seq] and the sequence fits)
    int32_t *n_eff;  // [B] rows actually fed per sequence
    float *rope_cos; // [R, rotary_dim/2]
    float *rope_sin;
};

}  // namespace ssd

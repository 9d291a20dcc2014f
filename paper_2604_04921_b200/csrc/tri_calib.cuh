// Calibration statistics (Sections 3.3 and 4.1, Appendix B.5): per query head and band the running sums
// behind E[q_f] (complex mean of the pre-RoPE query component), E|q_f| (mean magnitude) and the mean
// resultant length R_f = |E q_f| / E|q_f|.  A pure streaming reduction: every query row is read once.
//
// k_calib_partial  grid (blocks, heads): a block walks a contiguous range of tokens of one head, 4 or 8 tokens
//                  per warp at a time, 4 components per lane and token (one 8- or 16-byte load each).  Sums run
//                  in fp32 for 32 tokens, then move to fp64; the block's 192 sums go to its own slot, no atomics.
// k_calib_merge    adds the block slots of a head into the running state in a fixed order (bit-reproducible).
// k_calib_finish   state -> means and R_f.
#pragma once
#include "tri_common.cuh"

namespace tri {

constexpr int kCalibThreads = 256;
constexpr int kCalibWarps = kCalibThreads / 32;
constexpr int kCalibSums = kHeadDim + kBands;      // 128 component sums + 64 magnitude sums per head
constexpr int kCalibFlush = 32;                    // tokens a lane adds in fp32 before moving on to fp64

struct CalibParams {
    const void *q;            // [T][heads][128], bf16 (KIND 0) or fp32 (KIND 1)
    int64_t T, stride_tok, stride_head;   // strides in elements
    int32_t per_block;        // tokens per block
    double *partials;         // [heads][gridDim.x][192]
};

// sqrt to ~2^-22 relative in one special-function instruction (the results are averaged and rounded to fp32).
__device__ __forceinline__ float approx_sqrt(float x)
{
    float r;
    asm("sqrt.approx.f32 %0, %1;\n" : "=f"(r) : "f"(x));
    return r;
}

// Four consecutive components as raw words (bf16: 8 bytes, fp32: 16 bytes; unused words are 0) and their values.
template <int KIND>
__device__ __forceinline__ uint4 load_raw(const void *base, int64_t elem)
{
    // volatile: the U loads of a trip are issued back to back, ahead of the arithmetic on any of them
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (KIND == 0)
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];\n"
                     : "=r"(v.x), "=r"(v.y) : "l"(reinterpret_cast<const uint16_t *>(base) + elem));
    else
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(reinterpret_cast<const float *>(base) + elem));
    return v;
}
template <int KIND>
__device__ __forceinline__ float4 widen(uint4 v)
{
    if (KIND == 0)
        return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                           __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
    return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w));
}

// Slots of a lane: 0..3 the sums of components 4 lane .. 4 lane + 3; 4..7 magnitude sums.
//   LAYOUT 0 (pairs (2f, 2f+1)): the lane owns bands 2 lane and 2 lane + 1 (slots 4, 5).
//   LAYOUT 1 (pairs (f, f+64)):  lanes 0..15 hold the real parts of bands 4 lane .. 4 lane + 3, lanes 16..31
//                                the imaginary parts; lanes 0..15 own the four magnitudes (slots 4..7).
// grid (blocks, heads): a block owns a contiguous token range of one head; its warps take U tokens each per
// trip.  (One head per warp, with a block's warps on adjacent heads of the same tokens, measured half as fast.)
template <int LAYOUT, int KIND>
__global__ void __launch_bounds__(kCalibThreads) k_calib_partial(const CalibParams p)
{
    constexpr int U = KIND == 0 ? 8 : 4;     // tokens per warp and trip: U independent loads in flight per lane
    __shared__ double red[kCalibWarps][32][8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int head = blockIdx.y;
    const int64_t t_begin = (int64_t)blockIdx.x * p.per_block;
    const int64_t t_end = min(t_begin + (int64_t)p.per_block, p.T);
    double acc[8];
    float part[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { acc[i] = 0.0; part[i] = 0.f; }
    const int64_t row0 = (int64_t)head * p.stride_head + 4 * lane;
    int pending = 0;
    for (int64_t t = t_begin + U * warp; t < t_end; t += U * kCalibWarps) {
        uint4 raw[U];
#pragma unroll
        for (int j = 0; j < U; ++j)
            raw[j] = t + j < t_end ? load_raw<KIND>(p.q, (t + j) * p.stride_tok + row0) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const float4 x = widen<KIND>(raw[j]);
            part[0] += x.x; part[1] += x.y; part[2] += x.z; part[3] += x.w;
            if (LAYOUT == 0) {
                part[4] += approx_sqrt(x.x * x.x + x.y * x.y);
                part[5] += approx_sqrt(x.z * x.z + x.w * x.w);
            } else {
                const float ox = __shfl_xor_sync(0xffffffffu, x.x, 16), oy = __shfl_xor_sync(0xffffffffu, x.y, 16);
                const float oz = __shfl_xor_sync(0xffffffffu, x.z, 16), ow = __shfl_xor_sync(0xffffffffu, x.w, 16);
                part[4] += approx_sqrt(x.x * x.x + ox * ox);
                part[5] += approx_sqrt(x.y * x.y + oy * oy);
                part[6] += approx_sqrt(x.z * x.z + oz * oz);
                part[7] += approx_sqrt(x.w * x.w + ow * ow);
            }
        }
        pending += U;
        if (pending >= kCalibFlush) {
#pragma unroll
            for (int i = 0; i < 8; ++i) { acc[i] += (double)part[i]; part[i] = 0.f; }
            pending = 0;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) red[warp][lane][i] = acc[i] + (double)part[i];
    __syncthreads();
    // thread (lane l, slot i) adds the warps in order and writes the sum to its place among the 192
    {
        const int l = threadIdx.x >> 3, i = threadIdx.x & 7;
        double s = 0.0;
        for (int w = 0; w < kCalibWarps; ++w) s += red[w][l][i];
        int dst = -1;
        if (i < 4) dst = 4 * l + i;
        else if (LAYOUT == 0) { if (i < 6) dst = kHeadDim + 2 * l + (i - 4); }
        else if (l < 16) dst = kHeadDim + 4 * l + (i - 4);
        if (dst >= 0) p.partials[((int64_t)head * gridDim.x + blockIdx.x) * kCalibSums + dst] = s;
    }
}

// state: [heads][192] running sums, then one double holding the number of tokens seen so far.
__global__ void __launch_bounds__(kCalibSums) k_calib_merge(const double *__restrict__ partials, int nblocks, int64_t T,
                                                             double *state, int heads)
{
    const int head = blockIdx.x, i = threadIdx.x;
    double s = 0.0;
    for (int b = 0; b < nblocks; ++b) s += partials[((int64_t)head * nblocks + b) * kCalibSums + i];
    state[(int64_t)head * kCalibSums + i] += s;
    if (head == 0 && i == 0) state[(int64_t)heads * kCalibSums] += (double)T;
}

template <int LAYOUT>
__global__ void __launch_bounds__(kBands) k_calib_finish(const double *__restrict__ state, int heads, float *q_center,
                                                          float *q_mean_norm, float *mrl)
{
    const int head = blockIdx.x, f = threadIdx.x;
    const double n = state[(int64_t)heads * kCalibSums];
    const double *s = state + (int64_t)head * kCalibSums;
    const int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
    const double cr = n > 0.0 ? s[ir] / n : 0.0, ci = n > 0.0 ? s[ii] / n : 0.0;
    const double mn = n > 0.0 ? s[kHeadDim + f] / n : 0.0;
    q_center[(int64_t)head * kHeadDim + ir] = (float)cr;
    q_center[(int64_t)head * kHeadDim + ii] = (float)ci;
    q_mean_norm[(int64_t)head * kBands + f] = (float)mn;
    if (mrl) mrl[(int64_t)head * kBands + f] = mn > 0.0 ? (float)(sqrt(cr * cr + ci * ci) / mn) : 0.f;
}

}  // namespace tri

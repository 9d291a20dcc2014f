// Raw scoring of keys cached BEFORE RoPE (the k_f of Section 4.1 as they are): fp32 vectors scored in double
// (k_kind 1, the reference-style path of the tiny configuration) and bf16 vectors scored in fp32 with tabulated
// distance phasors (k_kind 2).  Same grid, outputs and partial sums as the post-RoPE kernels.
#pragma once
#include "tri_score.cuh"

namespace tri {

// ---------------------------------------------------------------------------------------
// Raw scoring of fp32 pre-RoPE keys (k_kind 1): the reference-style slow path, all in double.
//   S~^(g)(k) = sum_f Re( conj(k_f) * E[q_f]^(g) * Dbar_f * e^{i omega_f (p_q - p_k)} ) + sum_f m_f |k_f|
// Same grid, outputs and partial sums as the bf16 kernel; one thread per key.
// ---------------------------------------------------------------------------------------
template <int LAYOUT>
__global__ void __launch_bounds__(kScoreThreads)
k_score_f32_pre(const ScoreParams p, const double *__restrict__ omega, const double2 *__restrict__ dbar,
                const int64_t *__restrict__ cur_pos)
{
    __shared__ double red[kScoreWarps][kMaxGroup][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n || n <= skip_limit(p, u)) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int64_t pq = cur_pos[s];
    double a1[kMaxGroup], a2[kMaxGroup];
    for (int g = 0; g < kMaxGroup; ++g) { a1[g] = 0.0; a2[g] = 0.0; }

    for (int key = key_begin + tid; key < key_end; key += kScoreThreads) {
        int64_t off = row_offset(p.src, l, s, h, key);
        if (off < 0) {
            if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
            continue;
        }
        const float *row = reinterpret_cast<const float *>(p.src.k) + off;
        int64_t pk = p.src.positions ? (int64_t)p.src.positions[(int64_t)u * p.src.n_max + key] : (int64_t)key;
        double Delta = (double)(pq - pk);
        double acc[kMaxGroup];
        for (int g = 0; g < kMaxGroup; ++g) acc[g] = 0.0;
        for (int f = 0; f < kBands; ++f) {
            int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
            double kr = row[ir], ki = row[ii];
            double sn, cs;
            sincos(omega[f] * Delta, &sn, &cs);
            double2 d = dbar[f];
            double pr = cs * d.x - sn * d.y, pi = cs * d.y + sn * d.x;   // Dbar_f e^{i omega_f Delta}
            double mag = sqrt(kr * kr + ki * ki);
            for (int g = 0; g < G; ++g) {
                const float *c = p.qc + ((int64_t)l * p.H * G + (int64_t)h * G + g) * kHeadDim;
                double cr = c[ir], ci = c[ii];
                double tr = cr * pr - ci * pi, ti = cr * pi + ci * pr;     // E[q_f] * phasor
                double m = p.mw[((int64_t)l * p.H * G + (int64_t)h * G + g) * kBands + f];
                acc[g] += kr * tr + ki * ti + m * mag;
            }
        }
        for (int g = 0; g < G; ++g) {
            float y = (float)acc[g];
            p.raw[((int64_t)u * p.src.n_max + key) * G + g] = y;
            a1[g] += (double)y;
            a2[g] += (double)y * (double)y;
        }
    }
    for (int g = 0; g < G; ++g) {
        double a = a1[g], b = a2[g];
        for (int m = 1; m < 32; m <<= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, m);
            b += __shfl_xor_sync(0xffffffffu, b, m);
        }
        if (lane == 0) { red[warp][g][0] = a; red[warp][g][1] = b; }
    }
    __syncthreads();
    if (tid < G) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < kScoreWarps; ++w) { a += red[w][tid][0]; b += red[w][tid][1]; }
        p.partials[((int64_t)u * p.nchunks + chunk) * G + tid] = make_double2(a, b);
    }
}

// ---------------------------------------------------------------------------------------
// Raw scoring of bf16 pre-RoPE keys (k_kind 2) in fp32, one thread per key.
//   S~^(g)(k) = sum_f Re( conj(k_f) * E[q_f]^(g) * Dbar_f * e^{i omega_f Delta} ) + sum_f m_f |k_f|,   Delta = p_q - p_k >= 0
// The phasor of a distance comes from two tables built in double when the context is created, stored band-major so
// that neighbouring keys (neighbouring distances) read neighbouring entries:
//   rot_lo[f][b] = Dbar_f e^{i omega_f b}            b = Delta % 512
//   rot_hi[f][a] = e^{i omega_f 512 a}               a = Delta / 512 < kRotHi
// Their product carries the phasor to ~2e-7, whatever the angle.  Same grid, outputs and partial sums as the other
// scoring kernels.  A distance outside the tables is reported through device_status and that key scores 0.
// ---------------------------------------------------------------------------------------
constexpr int kRotLo = 512, kRotHi = 4096;            // distances up to 2,097,151

// GP: the group size rounded up to 4, 8 or 16 (accumulators per thread).
template <int LAYOUT, int GP>
__global__ void __launch_bounds__(kScoreThreads)
k_score_bf16_pre(const ScoreParams p, const float2 *__restrict__ rot_lo, const float2 *__restrict__ rot_hi,
                 const int64_t *__restrict__ cur_pos)
{
    // statistics of the group's heads, head-minor so that one 16-byte load serves four heads: Re E[q_f], Im E[q_f], m_f
    __shared__ __align__(16) float qr_s[kBands][GP], qi_s[kBands][GP], mw_s[kBands][GP];
    __shared__ double red[kScoreWarps][kMaxGroup][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n || n <= skip_limit(p, u)) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int64_t pq = cur_pos[s];
    for (int i = tid; i < GP * kBands; i += kScoreThreads) {
        const int g = i / kBands, f = i - g * kBands;
        if (g >= G) { qr_s[f][g] = 0.f; qi_s[f][g] = 0.f; mw_s[f][g] = 0.f; continue; }
        const int64_t qh = (int64_t)l * p.H * G + (int64_t)h * G + g;
        const int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
        qr_s[f][g] = p.qc[qh * kHeadDim + ir];
        qi_s[f][g] = p.qc[qh * kHeadDim + ii];
        mw_s[f][g] = p.mw[qh * kBands + f];
    }
    __syncthreads();
    float a1[GP], a2[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) { a1[g] = 0.f; a2[g] = 0.f; }

    for (int key = key_begin + tid; key < key_end; key += kScoreThreads) {
        const int64_t off = row_offset(p.src, l, s, h, key);
        const int64_t pk = p.src.positions ? (int64_t)p.src.positions[(int64_t)u * p.src.n_max + key] : (int64_t)key;
        const int64_t Delta = pq - pk;
        float acc[GP];
#pragma unroll
        for (int g = 0; g < GP; ++g) acc[g] = 0.f;
        if (off < 0 || Delta < 0 || Delta >= (int64_t)kRotLo * kRotHi) {
            if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
        } else {
            const uint4 *row = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(p.src.k) + off);
            const int a = (int)(Delta >> 9), b = (int)(Delta & (kRotLo - 1));
#pragma unroll 2
            for (int c = 0; c < 8; ++c) {                  // 8 bands per step: two 16-byte pieces of the row
                uint4 x, y;
                if (LAYOUT == 0) { x = __ldg(row + 2 * c); y = __ldg(row + 2 * c + 1); }     // (re, im) pairs of bands 8c .. 8c + 7
                else { x = __ldg(row + c); y = __ldg(row + 8 + c); }                         // real parts | imaginary parts
                const uint32_t wx[4] = {x.x, x.y, x.z, x.w}, wy[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int f = 8 * c + j;
                    float kr, ki;
                    if (LAYOUT == 0) {
                        const uint32_t w = j < 4 ? wx[j] : wy[j - 4];
                        kr = __uint_as_float(w << 16); ki = __uint_as_float(w & 0xffff0000u);
                    } else {
                        const uint32_t wr = wx[j >> 1], wi = wy[j >> 1];
                        kr = (j & 1) ? __uint_as_float(wr & 0xffff0000u) : __uint_as_float(wr << 16);
                        ki = (j & 1) ? __uint_as_float(wi & 0xffff0000u) : __uint_as_float(wi << 16);
                    }
                    const float2 lo = __ldg(rot_lo + f * kRotLo + b), hi = __ldg(rot_hi + f * kRotHi + a);
                    const float pr = lo.x * hi.x - lo.y * hi.y, pi = lo.x * hi.y + lo.y * hi.x;   // Dbar_f e^{i omega_f Delta}
                    const float tr = kr * pr + ki * pi, ti = kr * pi - ki * pr;                   // conj(k_f) * phasor
                    const float mag = sqrtf(kr * kr + ki * ki);
#pragma unroll
                    for (int g4 = 0; g4 < GP; g4 += 4) {  // heads beyond G have zero statistics in shared memory
                        const float4 qr = *reinterpret_cast<const float4 *>(&qr_s[f][g4]), qi = *reinterpret_cast<const float4 *>(&qi_s[f][g4]);
                        const float4 mw = *reinterpret_cast<const float4 *>(&mw_s[f][g4]);
                        acc[g4] += tr * qr.x - ti * qi.x + mw.x * mag;
                        acc[g4 + 1] += tr * qr.y - ti * qi.y + mw.y * mag;
                        acc[g4 + 2] += tr * qr.z - ti * qi.z + mw.z * mag;
                        acc[g4 + 3] += tr * qr.w - ti * qi.w + mw.w * mag;
                    }
                }
            }
        }
#pragma unroll
        for (int g = 0; g < GP; ++g)
            if (g < G) {
                p.raw[((int64_t)u * p.src.n_max + key) * G + g] = acc[g];
                a1[g] += acc[g];
                a2[g] = fmaf(acc[g], acc[g], a2[g]);
            }
    }
#pragma unroll
    for (int g = 0; g < GP; ++g) {
        double a = a1[g], b = a2[g];
        for (int m = 1; m < 32; m <<= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, m);
            b += __shfl_xor_sync(0xffffffffu, b, m);
        }
        if (lane == 0) { red[warp][g][0] = a; red[warp][g][1] = b; }
    }
    __syncthreads();
    if (tid < G) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < kScoreWarps; ++w) { a += red[w][tid][0]; b += red[w][tid][1]; }
        p.partials[((int64_t)u * p.nchunks + chunk) * G + tid] = make_double2(a, b);
    }
}

}  // namespace tri

// Scoring kernels: phasor fold, raw scores S~^(g)(k), GQA z-score + max (Sections 4.1-4.3).
//
// Why one dot product is enough.  Keys are cached post-RoPE, k~_f = k_f e^{i omega_f p_k}
// (Appendix B.1).  One term of the trigonometric series (Section 4.1) is
//     |E q_f| |k_f| cos(omega_f (Delta + delta) + arg E q_f - arg k_f)
//   = Re( E q_f * conj(k_f) * e^{i omega_f (p_q - p_k + delta)} )
//   = Re( conj(k~_f) * E q_f * e^{i omega_f (p_q + delta)} ),
// so the key's own position cancels and the average over the offset set D (Section 4.2) only
// touches the query side:
//     mean_delta S_trig = sum_f Re( conj(k~_f) * W_f ),   W_f = E q_f * e^{i omega_f p_q} * Dbar_f,
//     Dbar_f = (1/|D|) sum_{delta in D} e^{i omega_f delta}.
// That is a 128-wide real dot product of the cached row with a per-(sequence, query head)
// vector; the norm term (Section 4.2) is a 64-wide dot product of the band magnitudes
// |k~_f| = |k_f| with m_f = E|q_f| - |E q_f|.
#pragma once
#include "tri_common.cuh"

namespace tri {

// ---------------------------------------------------------------------------------------
// Fold, step 1: E[s][f] = e^{i omega_f p_q[s]} * Dbar_f in double (angles reach ~1e5 rad).
// grid = S blocks of 64 threads.
// ---------------------------------------------------------------------------------------
__global__ void k_fold_phasors(const double *__restrict__ omega, const double2 *__restrict__ dbar,
                               const int64_t *__restrict__ cur_pos, double2 *__restrict__ E)
{
    int s = blockIdx.x, f = threadIdx.x;
    double sn, cs;
    sincos(omega[f] * (double)cur_pos[s], &sn, &cs);
    double2 d = dbar[f];
    E[s * kBands + f] = make_double2(cs * d.x - sn * d.y, cs * d.y + sn * d.x);
}

// ---------------------------------------------------------------------------------------
// small PTX helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_sqrt(float x)
{
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;\n" : "=f"(r) : "f"(x));
    return r;
}

// Packed fp32 pairs (sm_100 f32x2 arithmetic): two lanes per instruction.
__device__ __forceinline__ uint64_t pack2(float a, float b)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &a, float &b)
{
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint32_t bf16_hi_bits(float w)   // bf16(w), round to nearest even
{
    uint32_t b = __float_as_uint(w);
    b += 0x7fffu + ((b >> 16) & 1u);
    return b >> 16;
}

struct ScoreParams {
    View src;
    int32_t S, H, G;
    int32_t u0;           // first unit of this launch (a round may be issued as several launches over unit ranges)
    int32_t skip_upto;    // units of at most this many keys are not scored (the fused round keeps them whole); 0 = score all
    const int32_t *unit_budgets;   // [U] or NULL: with skip_upto > 0, the per-unit value min(unit_budgets[u], skip_upto) applies
    int32_t chunk;        // keys per block (multiple of 16)
    int32_t nchunks;      // blocks per unit
    const double2 *E;     // [S][64]  e^{i omega_f p_q} Dbar_f
    const float *qc;      // [L][H*G][128]  E[q_f]
    const float *mw;      // [L][H*G][64]   norm weights m_f
    const uint8_t *bt;    // tcgen05 kernel: folded B operand images, [U] trig and [L*H] norm (see k_fold_operands)
    const uint8_t *bn;
    float *raw;           // [U][n_max][G]
    double2 *partials;    // [U][nchunks][G]  (sum, sum of squares) of raw over the block's keys
    int32_t *device_status;
};

// Units of at most this many keys are left unscored by the fused round (it keeps them whole).
__device__ __forceinline__ int skip_limit(const ScoreParams &p, int u)
{
    return (p.unit_budgets && p.skip_upto > 0) ? min(max(__ldg(p.unit_budgets + u), 0), p.skip_upto) : p.skip_upto;
}

// mu_g and 1/sigma_g of one unit from the per-block partial sums, added in a fixed order so that every
// block (and every kernel) that asks gets the same bits.  Threads 0 .. 255 of the block take part:
// 16 lanes per head, lane i adds blocks i, i+16, ...; then a fixed butterfly.  Results land in shared
// memory; the caller synchronises.  A head whose scores are equal up to fp32 resolution gets 1/sigma = 0
// (it then contributes z = 0: Section 4.3 with sigma_g = 0).
__device__ __forceinline__ void unit_mean_rstd(const double2 *__restrict__ part, int G, int used, int n,
                                               float *mu_s, float *rs_s)
{
    const int tid = threadIdx.x;
    if (tid >= 16 * kMaxGroup) return;          // whole warps only: the shuffles below stay converged
    int g = tid >> 4, i = tid & 15;
    double a = 0.0, b = 0.0;
    if (g < G)
        for (int c = i; c < used; c += 16) {
            double2 v = part[(int64_t)c * G + g];
            a += v.x;
            b += v.y;
        }
    for (int m = 1; m < 16; m <<= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, m);
        b += __shfl_xor_sync(0xffffffffu, b, m);
    }
    if (g < G && i == 0) {
        double mu = a / (double)n;
        double var = b / (double)n - mu * mu;
        double rs = (var > 1e-12 * mu * mu && var > 0.0) ? rsqrt(var) : 0.0;
        mu_s[g] = (float)mu;
        rs_s[g] = (float)rs;
    }
}

// z-score + max over the group for one key (Section 4.3), from its G raw scores.
__device__ __forceinline__ float zmax4(float4 x, const float *mu_s, const float *rs_s)
{
    return fmaxf(fmaxf((x.x - mu_s[0]) * rs_s[0], (x.y - mu_s[1]) * rs_s[1]),
                 fmaxf((x.z - mu_s[2]) * rs_s[2], (x.w - mu_s[3]) * rs_s[3]));
}
__device__ __forceinline__ float zmax8(const float4 *row, const float *mu_s, const float *rs_s)
{
    return fmaxf(zmax4(row[0], mu_s, rs_s), zmax4(row[1], mu_s + 4, rs_s + 4));
}
__device__ __forceinline__ float zmax(const float *row, int G, const float *mu_s, const float *rs_s)
{
    float z = -INFINITY;
    for (int g = 0; g < G; ++g) z = fmaxf(z, (row[g] - mu_s[g]) * rs_s[g]);
    return z;
}

// ---------------------------------------------------------------------------------------
// GQA normalise-then-aggregate (Section 4.3): S_final(k) = max_g (raw_g(k) - mu_g) / sigma_g.
// Same grid as the scoring kernel.  mu, sigma come from the per-block partial sums, added in a
// fixed order so that every block of a unit (and every run) sees the same bits.
// ---------------------------------------------------------------------------------------
struct NormParams {
    const float *raw;           // [U][n_max][G]
    const double2 *partials;    // [U][nchunks][G]
    const int32_t *seq_lens;
    float *scores;              // [U][n_max]
    int32_t S, H, G, n_max, chunk, nchunks, u0;
};

__global__ void __launch_bounds__(256) k_normalize(const NormParams p)
{
    __shared__ float mu_s[kMaxGroup], rs_s[kMaxGroup];
    const int tid = threadIdx.x;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int s = (u / p.H) % p.S;
    const int n = min(__ldg(p.seq_lens + s), p.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int used = (n + p.chunk - 1) / p.chunk;
    unit_mean_rstd(p.partials + (int64_t)u * p.nchunks * G, G, used, n, mu_s, rs_s);
    __syncthreads();
    const float *rawu = p.raw + (int64_t)u * p.n_max * G;
    float *out = p.scores + (int64_t)u * p.n_max;
    if (G == 4) {
        for (int key = key_begin + tid; key < key_end; key += 256)
            out[key] = zmax4(*reinterpret_cast<const float4 *>(rawu + (int64_t)key * 4), mu_s, rs_s);
    } else if (G == 8) {
        for (int key = key_begin + tid; key < key_end; key += 256)
            out[key] = zmax8(reinterpret_cast<const float4 *>(rawu + (int64_t)key * 8), mu_s, rs_s);
    } else {
        for (int key = key_begin + tid; key < key_end; key += 256)
            out[key] = zmax(rawu + (int64_t)key * G, G, mu_s, rs_s);
    }
}

}  // namespace tri

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

__device__ __forceinline__ void mma_tf32_1688(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
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

// Upper part of an fp32 that is exactly representable in tf32 (10 explicit mantissa bits).  With
// lo = x - hi (exact), hi + lo carries x to ~2^-22 through two tf32 MMAs.
__device__ __forceinline__ uint32_t to_tf32(float x) { return __float_as_uint(x) & 0xffffe000u; }

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

// Magnitudes of two bands held as bf16 (re, im) pairs in xa and xb, split for tf32:
// hi = (hi_a, hi_b) as tf32 bit patterns, lo = the exact remainders.
__device__ __forceinline__ void band_mags2(uint32_t xa, uint32_t xb, uint32_t &hi_a, uint32_t &hi_b,
                                           uint32_t &lo_a, uint32_t &lo_b)
{
    uint64_t re = pack2(__uint_as_float(xa << 16), __uint_as_float(xb << 16));
    uint64_t im = pack2(__uint_as_float(xa & 0xffff0000u), __uint_as_float(xb & 0xffff0000u));
    float sa, sb;
    unpack2(fma2(re, re, mul2(im, im)), sa, sb);
    float ma = fast_sqrt(sa), mb = fast_sqrt(sb);
    hi_a = to_tf32(ma);
    hi_b = to_tf32(mb);
    float la, lb;
    unpack2(sub2(pack2(ma, mb), pack2(__uint_as_float(hi_a), __uint_as_float(hi_b))), la, lb);
    lo_a = __float_as_uint(la);
    lo_b = __float_as_uint(lb);
}

// 16-byte streaming load of cache rows: read once, keep out of L1.
__device__ __forceinline__ uint4 ld_stream(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
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
    int32_t chunk;        // keys per block (multiple of 16)
    int32_t nchunks;      // blocks per unit
    const double2 *E;     // [S][64]  e^{i omega_f p_q} Dbar_f
    const float *qc;      // [L][H*G][128]  E[q_f]
    const float *mw;      // [L][H*G][64]   norm weights m_f
    float *raw;           // [U][n_max][G]
    double2 *partials;    // [U][nchunks][G]  (sum, sum of squares) of raw over the block's keys
    int32_t *device_status;
};

// Band geometry of one thread's share of a 16-key tile.
//
// Thread (q = lane/4, t = lane%4) of a warp loads, for rows q and q+8 of the tile, the four
// 16-byte pieces c = t + 4j (j = 0..3) of the 256-byte row; piece c holds dims 8c..8c+7, its
// register r (0..3) dims 8c+2r, 8c+2r+1.  The k index of the MMAs is a free permutation, so these
// registers are used as A fragments directly:
//   bf16 m16n8k16, step s = 2j + e:  (a0, a1) = register 2e of rows (q, q+8), (a2, a3) = register 2e+1
//        => k slots (2t, 2t+1) <-> dims 8c+4e, 8c+4e+1;  slots (2t+8, 2t+9) <-> dims 8c+4e+2, 8c+4e+3.
// The B fragments are built with the same map, so the contraction runs over all 128 dims.
template <int LAYOUT>
__device__ __forceinline__ int band_of(int t, int j, int r, int half)
{
    // band whose magnitude is formed from (piece j, register r [, half]) of thread t
    if (LAYOUT == 0) return 4 * (t + 4 * j) + r;   // register = (re, im) of one band
    return 8 * (t + 4 * j) + 2 * r + half;          // j in {0,1}: re from piece j, im from piece j+2
}

// ---------------------------------------------------------------------------------------
// Raw scoring of bf16 post-RoPE keys on the tensor cores.
//   grid = U * nchunks blocks, 256 threads; block (u, chunk) scores keys [chunk*C, (chunk+1)*C).
//   NT = number of 8-column MMA tiles: columns (2i, 2i+1) of tile nt carry the (hi, lo) bf16
//   halves of W for query head g = 4*nt + i, so thread t ends up with head 4*nt + t of rows q, q+8.
// ---------------------------------------------------------------------------------------
template <int NT, int LAYOUT>
__global__ void __launch_bounds__(kScoreThreads)
k_score_bf16(const ScoreParams p)
{
    __shared__ float Wf[NT * 4][kHeadDim];            // W as fp32, dims in cache order
    __shared__ float Mf[NT * 4][kBands];              // norm weights
    __shared__ uint2 trigB[NT][8][32];                // bf16x2 B fragments
    __shared__ uint2 normB[NT][8][32];                // tf32 B fragments
    __shared__ double red[kScoreWarps][NT * 4][2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.x / p.nchunks, chunk = blockIdx.x - u * p.nchunks;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;

    // ---- fold, step 2: W_f^(g) = E[q_f]^(g) * E[s][f]  (double), split for the tensor cores ----
    for (int i = tid; i < NT * 4 * kBands; i += kScoreThreads) {
        int g = i / kBands, f = i - g * kBands;
        float wr = 0.f, wi = 0.f, m = 0.f;
        if (g < G) {
            const float *c = p.qc + ((int64_t)l * p.H * G + (int64_t)h * G + g) * kHeadDim;
            int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
            double cr = c[ir], ci = c[ii];
            double2 e = p.E[s * kBands + f];
            wr = (float)(cr * e.x - ci * e.y);
            wi = (float)(cr * e.y + ci * e.x);
            m = p.mw[((int64_t)l * p.H * G + (int64_t)h * G + g) * kBands + f];
            Wf[g][ir] = wr;
            Wf[g][ii] = wi;
            Mf[g][f] = m;
        } else {
            int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
            Wf[g][ir] = 0.f;
            Wf[g][ii] = 0.f;
            Mf[g][f] = 0.f;
        }
    }
    __syncthreads();
    for (int i = tid; i < NT * 8 * 32; i += kScoreThreads) {
        int ln = i & 31, st = (i >> 5) & 7, nt = i >> 8;
        int col = ln >> 2, t = ln & 3;          // B fragment: column = lane/4, k slots from lane%4
        int g = 4 * nt + (col >> 1), part = col & 1;
        int j = st >> 1, e = st & 1;
        // trig: k slots (2t, 2t+1) and (2t+8, 2t+9)
        int dA = 8 * (t + 4 * j) + 4 * e;
        uint32_t w[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            float v = Wf[g][dA + x];
            uint32_t hi = bf16_hi_bits(v);
            if (part == 0) w[x] = hi;
            else w[x] = bf16_hi_bits(v - __uint_as_float(hi << 16));
        }
        trigB[nt][st][ln] = make_uint2(w[0] | (w[1] << 16), w[2] | (w[3] << 16));
        // norm: tf32 step st covers two bands per thread, k slot t and t+4
        int b0, b1;
        if (LAYOUT == 0) { b0 = band_of<0>(t, j, 2 * e, 0); b1 = band_of<0>(t, j, 2 * e + 1, 0); }
        else { int jj = st >> 2, r = st & 3; b0 = band_of<1>(t, jj, r, 0); b1 = band_of<1>(t, jj, r, 1); }
        float m0 = Mf[g][b0], m1 = Mf[g][b1];
        uint32_t h0 = to_tf32(m0), h1 = to_tf32(m1);
        if (part == 0) normB[nt][st][ln] = make_uint2(h0, h1);
        else normB[nt][st][ln] = make_uint2(__float_as_uint(m0 - __uint_as_float(h0)),
                                            __float_as_uint(m1 - __uint_as_float(h1)));
    }
    __syncthreads();

    const int q = lane >> 2, t = lane & 3;
    float s1[NT], s2[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { s1[nt] = 0.f; s2[nt] = 0.f; }

    const char *kbase = p.src.k;
    const int ntiles = (key_end - key_begin + kTileKeys - 1) / kTileKeys;
    for (int tile = warp; tile < ntiles; tile += kScoreWarps) {
        const int r0 = key_begin + tile * kTileKeys + q, r1 = r0 + 8;
        const bool v0 = r0 < key_end, v1 = r1 < key_end;
        uint4 A0[4], A1[4];
        {
            int64_t o0 = v0 ? row_offset(p.src, l, s, h, r0) : -1;
            int64_t o1 = v1 ? row_offset(p.src, l, s, h, r1) : -1;
            if ((v0 && o0 < 0) || (v1 && o1 < 0)) {
                if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
            }
            const char *p0 = kbase + o0 * 2 + t * 16, *p1 = kbase + o1 * 2 + t * 16;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                A0[j] = o0 >= 0 ? ld_stream(p0 + j * 64) : make_uint4(0, 0, 0, 0);
                A1[j] = o1 >= 0 ? ld_stream(p1 + j * 64) : make_uint4(0, 0, 0, 0);
            }
        }
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }

        // trigonometric part: K[16 x 128] * W[128 x 8NT] on bf16 tensor cores, fp32 accumulate
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t *x0 = reinterpret_cast<const uint32_t *>(&A0[j]);
            const uint32_t *x1 = reinterpret_cast<const uint32_t *>(&A1[j]);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    uint2 b = trigB[nt][2 * j + e][lane];
                    mma_bf16_16816(acc[nt], x0[2 * e], x1[2 * e], x0[2 * e + 1], x1[2 * e + 1], b.x, b.y);
                }
            }
        }
        // norm part: band magnitudes (fp32, split hi + lo for tf32) times m_f
        if (LAYOUT == 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t *x0 = reinterpret_cast<const uint32_t *>(&A0[j]);
                const uint32_t *x1 = reinterpret_cast<const uint32_t *>(&A1[j]);
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    // pair the same band of rows q and q+8: (a0, a1) and (a2, a3) are then born adjacent
                    uint32_t h00, h01, l00, l01, h10, h11, l10, l11;
                    band_mags2(x0[2 * e], x1[2 * e], h00, h10, l00, l10);           // k slot t
                    band_mags2(x0[2 * e + 1], x1[2 * e + 1], h01, h11, l01, l11);   // k slot t+4
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        uint2 b = normB[nt][2 * j + e][lane];
                        mma_tf32_1688(acc[nt], h00, h10, h01, h11, b.x, b.y);
                        mma_tf32_1688(acc[nt], l00, l10, l01, l11, b.x, b.y);
                    }
                }
            }
        } else {
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const uint32_t *xr0 = reinterpret_cast<const uint32_t *>(&A0[jj]);
                const uint32_t *xi0 = reinterpret_cast<const uint32_t *>(&A0[jj + 2]);
                const uint32_t *xr1 = reinterpret_cast<const uint32_t *>(&A1[jj]);
                const uint32_t *xi1 = reinterpret_cast<const uint32_t *>(&A1[jj + 2]);
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    float m0[2], m1[2];
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {
                        float re0 = __uint_as_float(hf ? (xr0[r] & 0xffff0000u) : (xr0[r] << 16));
                        float im0 = __uint_as_float(hf ? (xi0[r] & 0xffff0000u) : (xi0[r] << 16));
                        float re1 = __uint_as_float(hf ? (xr1[r] & 0xffff0000u) : (xr1[r] << 16));
                        float im1 = __uint_as_float(hf ? (xi1[r] & 0xffff0000u) : (xi1[r] << 16));
                        m0[hf] = fast_sqrt(fmaf(re0, re0, im0 * im0));
                        m1[hf] = fast_sqrt(fmaf(re1, re1, im1 * im1));
                    }
                    uint32_t h00 = to_tf32(m0[0]), h10 = to_tf32(m1[0]), h01 = to_tf32(m0[1]), h11 = to_tf32(m1[1]);
                    uint32_t l00 = __float_as_uint(m0[0] - __uint_as_float(h00));
                    uint32_t l10 = __float_as_uint(m1[0] - __uint_as_float(h10));
                    uint32_t l01 = __float_as_uint(m0[1] - __uint_as_float(h01));
                    uint32_t l11 = __float_as_uint(m1[1] - __uint_as_float(h11));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        uint2 b = normB[nt][4 * jj + r][lane];
                        mma_tf32_1688(acc[nt], h00, h10, h01, h11, b.x, b.y);
                        mma_tf32_1688(acc[nt], l00, l10, l01, l11, b.x, b.y);
                    }
                }
            }
        }

        // columns (2t, 2t+1) of tile nt are the hi and lo halves of head 4nt + t
        float *rawu = p.raw + (int64_t)u * p.src.n_max * G;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            int g = 4 * nt + t;
            float y0 = acc[nt][0] + acc[nt][1], y1 = acc[nt][2] + acc[nt][3];
            if (g < G) {
                if (v0) { rawu[(int64_t)r0 * G + g] = y0; s1[nt] += y0; s2[nt] = fmaf(y0, y0, s2[nt]); }
                if (v1) { rawu[(int64_t)r1 * G + g] = y1; s1[nt] += y1; s2[nt] = fmaf(y1, y1, s2[nt]); }
            }
        }
    }

    // ---- per-block (sum, sum^2) in a fixed order: lanes with equal t, then warps ----
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        double a = s1[nt], b = s2[nt];
#pragma unroll
        for (int m = 4; m < 32; m <<= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, m);
            b += __shfl_xor_sync(0xffffffffu, b, m);
        }
        if (q == 0) { red[warp][4 * nt + t][0] = a; red[warp][4 * nt + t][1] = b; }
    }
    __syncthreads();
    if (tid < G) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < kScoreWarps; ++w) { a += red[w][tid][0]; b += red[w][tid][1]; }
        p.partials[((int64_t)u * p.nchunks + chunk) * G + tid] = make_double2(a, b);
    }
}

// ---------------------------------------------------------------------------------------
// Raw scoring of fp32 pre-RoPE keys (k_kind 1): the reference-style slow path, all in double.
//   S~^(g)(k) = sum_f Re( conj(k_f) * E[q_f]^(g) * Dbar_f * e^{i omega_f (p_q - p_k)} ) + sum_f m_f |k_f|
// Same grid, outputs and partial sums as k_score_bf16; one thread per key.
// ---------------------------------------------------------------------------------------
template <int LAYOUT>
__global__ void __launch_bounds__(kScoreThreads)
k_score_f32_pre(const ScoreParams p, const double *__restrict__ omega, const double2 *__restrict__ dbar,
                const int64_t *__restrict__ cur_pos)
{
    __shared__ double red[kScoreWarps][kMaxGroup][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.x / p.nchunks, chunk = blockIdx.x - u * p.nchunks;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n) return;
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
// GQA normalise-then-aggregate (Section 4.3): S_final(k) = max_g (raw_g(k) - mu_g) / sigma_g.
// Same grid as the scoring kernel.  mu, sigma come from the per-block partial sums, added in a
// fixed order so that every block of a unit (and every run) sees the same bits.
// ---------------------------------------------------------------------------------------
struct NormParams {
    const float *raw;           // [U][n_max][G]
    const double2 *partials;    // [U][nchunks][G]
    const int32_t *seq_lens;
    float *scores;              // [U][n_max]
    int32_t S, H, G, n_max, chunk, nchunks;
};

__global__ void __launch_bounds__(256) k_normalize(const NormParams p)
{
    __shared__ float mu_s[kMaxGroup], rs_s[kMaxGroup];
    const int tid = threadIdx.x;
    const int u = blockIdx.x / p.nchunks, chunk = blockIdx.x - u * p.nchunks;
    const int s = (u / p.H) % p.S;
    const int n = min(__ldg(p.seq_lens + s), p.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int used = (n + p.chunk - 1) / p.chunk;
    {
        // 16 lanes per head: lane i adds blocks i, i+16, ...; then a fixed butterfly
        int g = tid >> 4, i = tid & 15;
        double a = 0.0, b = 0.0;
        if (g < G)
            for (int c = i; c < used; c += 16) {
                double2 v = p.partials[((int64_t)u * p.nchunks + c) * G + g];
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
            // scores equal up to fp32 resolution: sigma = 0, the head contributes z = 0
            double rs = (var > 1e-12 * mu * mu && var > 0.0) ? rsqrt(var) : 0.0;
            mu_s[g] = (float)mu;
            rs_s[g] = (float)rs;
        }
    }
    __syncthreads();
    const float *rawu = p.raw + (int64_t)u * p.n_max * G;
    float *out = p.scores + (int64_t)u * p.n_max;
    if (G == 4) {
        const float m0 = mu_s[0], m1 = mu_s[1], m2 = mu_s[2], m3 = mu_s[3];
        const float r0 = rs_s[0], r1 = rs_s[1], r2 = rs_s[2], r3 = rs_s[3];
        for (int key = key_begin + tid; key < key_end; key += 256) {
            float4 x = *reinterpret_cast<const float4 *>(rawu + (int64_t)key * 4);
            float z = fmaxf(fmaxf((x.x - m0) * r0, (x.y - m1) * r1), fmaxf((x.z - m2) * r2, (x.w - m3) * r3));
            out[key] = z;
        }
    } else {
        for (int key = key_begin + tid; key < key_end; key += 256) {
            float z = -INFINITY;
            for (int g = 0; g < G; ++g) z = fmaxf(z, (rawu[(int64_t)key * G + g] - mu_s[g]) * rs_s[g]);
            out[key] = z;
        }
    }
}

}  // namespace tri

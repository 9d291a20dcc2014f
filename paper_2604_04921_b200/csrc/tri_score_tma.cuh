// Raw scoring of bf16 post-RoPE keys: TMA -> swizzled shared memory -> ldmatrix -> tensor cores.
//
// Data movement.  The cache (contiguous or paged) is described to the TMA unit as a rank-5 bf16
// tensor (dim, row-in-page-or-unit, KV head, sequence-or-page, layer).  Every warp runs its own
// pipeline: for each of its 16-key tiles lane 0 issues two tiled bulk-tensor loads (left and right
// 64-element halves of the 16 rows, 2 KB each, 128-byte swizzle) that complete on a per-(warp, stage)
// mbarrier.  The warp waits (bounded), pulls the tile into registers with 8 ldmatrix.x4 -- which
// yields the A fragments of mma.m16n8k16 directly -- and immediately re-arms the stage with the
// tile kStages ahead, so the copy engine stays kStages tiles in front of the arithmetic.
//
// Arithmetic per k-step s (dims 16s..16s+15 of 16 keys):
//   trig   one bf16 MMA of the fragment with the (hi, lo)-split W              (Sections 4.1, 4.2)
//   norm   the fragment's four registers are four (re, im) pairs = four bands; the eight magnitudes of two
//          k-steps, split into a bf16 value and a bf16 residual, are the A fragments of two more bf16 MMAs
//          against m_f, itself split the same way into two columns per head           (Section 4.2)
// both accumulate into the same fp32 accumulator: thread (q, t) ends with S~ of head 4nt + t for keys
// q and q+8 of the tile.
#pragma once
#include <cuda.h>

#include "tri_score.cuh"

namespace tri {

constexpr int kStages = 2;
constexpr int kTileBytes = kTileKeys * kHeadDim * 2;                       // 4096
constexpr int kScoreDynSmem = kScoreWarps * kStages * kTileBytes;          // 65536: three blocks per SM
constexpr uint32_t kWaitPolls = 1u << 22;                                  // bound on every mbarrier wait

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Waits for the phase with the given parity; gives up after `polls` polls and returns false.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t polls = kWaitPolls)
{
    for (uint32_t i = 0; i < polls; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];\n" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

__device__ __forceinline__ uint32_t cvt_bf16x2(float upper, float lower)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(upper), "f"(lower));
    return r;
}
// Two band magnitudes straight from packed bf16 words, with the mixed-precision FMA of sm_100 (bf16 x bf16 + fp32 in
// one instruction, the product exact): no unpacking of the operands.
//   PAIRED = false: word a = (re, im) of one band, word b = (re, im) of another      -> |a|, |b|
//   PAIRED = true : word a = real parts of two bands, word b = their imaginary parts -> |(a.lo, b.lo)|, |(a.hi, b.hi)|
// Result: `hi` = the two magnitudes rounded to bf16 (first in the lower half), `lo` = the bf16 of what the rounding
// left over (m - hi, again one mixed FMA each): hi + lo carries each magnitude to ~2^-17.
#define TRI_MAG_PAIR_ASM(T, NEG1, X0, Y0, X1, Y1)                                         \
    asm("{\n"                                                                             \
        ".reg .b16 a0, a1, b0, b1, h0, h1, neg1;\n"                                       \
        ".reg .f32 s0, s1, m0, m1, r0, r1;\n"                                             \
        "mov.b32 {a0, a1}, %2;\n"                                                         \
        "mov.b32 {b0, b1}, %3;\n"                                                         \
        "mov.b16 neg1, " NEG1 ";\n" /* -1.0 */                                            \
        "fma.rn.f32." T " s0, " X0 ", " X0 ", 0f00000000;\n"                              \
        "fma.rn.f32." T " s1, " X1 ", " X1 ", 0f00000000;\n"                              \
        "fma.rn.f32." T " s0, " Y0 ", " Y0 ", s0;\n"                                      \
        "fma.rn.f32." T " s1, " Y1 ", " Y1 ", s1;\n"                                      \
        "sqrt.approx.ftz.f32 m0, s0;\n"                                                   \
        "sqrt.approx.ftz.f32 m1, s1;\n"                                                   \
        "cvt.rn." T "x2.f32 %0, m1, m0;\n"                                                \
        "mov.b32 {h0, h1}, %0;\n"                                                         \
        "fma.rn.f32." T " r0, h0, neg1, m0;\n"                                            \
        "fma.rn.f32." T " r1, h1, neg1, m1;\n"                                            \
        "cvt.rn." T "x2.f32 %1, r1, r0;\n"                                                \
        "}\n"                                                                             \
        : "=&r"(hi), "=r"(lo)                                                             \
        : "r"(a), "r"(b))

// F16 = false: the words hold bf16 pairs and so do the results; true: f16 (the 8-bit key path widens its keys to f16).
template <bool PAIRED, bool F16 = false>
__device__ __forceinline__ void mag_pair(uint32_t a, uint32_t b, uint32_t &hi, uint32_t &lo)
{
    if (F16) {
        if (PAIRED) TRI_MAG_PAIR_ASM("f16", "0xBC00", "a0", "b0", "a1", "b1");
        else TRI_MAG_PAIR_ASM("f16", "0xBC00", "a0", "a1", "b0", "b1");
    } else {
        if (PAIRED) TRI_MAG_PAIR_ASM("bf16", "0xBF80", "a0", "b0", "a1", "b1");
        else TRI_MAG_PAIR_ASM("bf16", "0xBF80", "a0", "a1", "b0", "b1");
    }
}
#undef TRI_MAG_PAIR_ASM

// ---- 8-bit keys (e4m3): widened exactly to f16 in registers, then the same two contractions on f16 tensor-core MMAs ----
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The two e4m3 values in the lower (upper) half of w as an f16 pair; every e4m3 value is an f16 value.
__device__ __forceinline__ void e4m3x4_to_f16x2(uint32_t w, uint32_t &lo, uint32_t &hi)
{
    asm("{\n.reg .b16 a, b;\nmov.b32 {a, b}, %2;\ncvt.rn.f16x2.e4m3x2 %0, a;\ncvt.rn.f16x2.e4m3x2 %1, b;\n}\n"
        : "=r"(lo), "=r"(hi) : "r"(w));
}
__device__ __forceinline__ uint32_t f16_bits(float w)          // f16(w), round to nearest even
{
    uint16_t r;
    asm("cvt.rn.f16.f32 %0, %1;\n" : "=h"(r) : "f"(w));
    return r;
}
__device__ __forceinline__ float f16_value(uint32_t bits)
{
    float r;
    asm("cvt.f32.f16 %0, %1;\n" : "=f"(r) : "h"((uint16_t)bits));
    return r;
}

// KEY8 = false: bf16 keys, tiles of two 64-element halves.  KEY8 = true: e4m3 keys, 128-byte rows, one box per tile;
// a 32-bit register of the 8-bit fragment holds dims 4t .. 4t+3 of its k-step, so slot x of lane t stands for dim
// 4t + x (not 2t + (x & 1) + 8 (x >> 1)): the B fragments are folded in the same order and the sum over k is the same.
template <int NT, int LAYOUT, bool KEY8 = false>
__global__ void __launch_bounds__(kScoreThreads, 3)
k_score_tma(const __grid_constant__ CUtensorMap tmap, const ScoreParams p)
{
    constexpr int kTileB = KEY8 ? kTileBytes / 2 : kTileBytes;          // bytes of one 16-key tile
    extern __shared__ __align__(1024) uint8_t tiles[];   // [warp][stage][half][16 rows][128 B]
    __shared__ uint2 trigB[NT][8][32];
    __shared__ uint2 normB[NT][4][32];
    __shared__ double red[kScoreWarps][NT * 4][2];
    __shared__ __align__(8) uint64_t bars[kScoreWarps][kStages];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n || n <= skip_limit(p, u)) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int ntiles = (key_end - key_begin + kTileKeys - 1) / kTileKeys;
    const int my_n = warp < ntiles ? (ntiles - warp + kScoreWarps - 1) / kScoreWarps : 0;

    const uint32_t my_tiles = smem_u32(tiles) + warp * (kStages * kTileB);
    const uint32_t my_bars = smem_u32(&bars[warp][0]);

    // lane 0 of each warp arms stage `it % kStages` with tile `it` of this warp
    auto issue = [&](int it) {
        const int stage = it % kStages;
        const int row = key_begin + (warp + kScoreWarps * it) * kTileKeys;
        int c1 = row, c3 = s;
        if (p.src.paged) {
            const int pg = p.src.page_shift >= 0 ? row >> p.src.page_shift : row / p.src.page_size;
            int page = __ldg(p.src.page_table + (int64_t)s * p.src.max_pages_per_seq + pg);
            if (p.src.n_pages > 0 && (page < 0 || page >= p.src.n_pages)) {
                if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                page = 0;                          // stay inside the pool; the unit's output is unspecified
            }
            c1 = row - pg * p.src.page_size;
            c3 = page;
        }
        const uint32_t bar = my_bars + stage * 8, dst = my_tiles + stage * kTileB;
        mbar_expect_tx(bar, kTileB);
        tma_load_5d(dst, &tmap, bar, 0, c1, h, c3, l);
        if (!KEY8) tma_load_5d(dst + kTileBytes / 2, &tmap, bar, kHeadDim / 2, c1, h, c3, l);
    };

    if (lane == 0) {
        for (int st = 0; st < kStages; ++st) mbar_init(my_bars + st * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        for (int it = 0; it < kStages && it < my_n; ++it) issue(it);
    }

    // ---- fold, step 2 (overlaps the first loads): W_f^(g) = E[q_f]^(g) * E[s][f], straight into the B fragments
    // of the MMAs, each value split into a bf16 and the bf16 of its residual (two columns per head) ----
    for (int i = tid; i < NT * 8 * 32; i += kScoreThreads) {
        const int ln = i & 31, st = (i >> 5) & 7, nt = i >> 8;
        const int col = ln >> 2, t = ln & 3;          // B fragment: column = lane/4, k slots from lane%4
        const int g = 4 * nt + (col >> 1), part = col & 1;
        const int64_t qh = (int64_t)l * p.H * G + (int64_t)h * G + g;
        const float *c = p.qc + qh * kHeadDim;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (g < G) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {            // k slots 2t, 2t+1, 2t+8, 2t+9 of step st = dims of the key row
                const int d = KEY8 ? 16 * st + 4 * t + x : 16 * st + 2 * t + (x & 1) + 8 * (x >> 1);
                const int f = LAYOUT == 0 ? d >> 1 : d & (kBands - 1);
                const bool imag = LAYOUT == 0 ? (d & 1) : (d >= kBands);
                const int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
                const double cr = c[ir], ci = c[ii];
                const double2 e = p.E[s * kBands + f];
                const float v = imag ? (float)(cr * e.y + ci * e.x) : (float)(cr * e.x - ci * e.y);
                if (KEY8) {
                    const uint32_t hi = f16_bits(v);
                    w[x] = part == 0 ? hi : f16_bits(v - f16_value(hi));
                } else {
                    const uint32_t hi = bf16_hi_bits(v);
                    w[x] = part == 0 ? hi : bf16_hi_bits(v - __uint_as_float(hi << 16));
                }
            }
        }
        trigB[nt][st][ln] = make_uint2(w[0] | (w[1] << 16), w[2] | (w[3] << 16));
        // norm: B fragment of pair st < 4 (k-steps 2 st and 2 st + 1 of the keys): k slots 2t, 2t+1, 2t+8, 2t+9
        // stand for the bands whose magnitudes the main loop puts there
        if (st < 4) {
            int bnd[4];
            if (KEY8 && LAYOUT == 0) { bnd[0] = 16 * st + 2 * t; bnd[1] = bnd[0] + 1; bnd[2] = 16 * st + 8 + 2 * t; bnd[3] = bnd[2] + 1; }
            else if (KEY8) { bnd[0] = 16 * st + 4 * t; bnd[1] = bnd[0] + 1; bnd[2] = bnd[0] + 2; bnd[3] = bnd[0] + 3; }
            else if (LAYOUT == 0) { bnd[0] = 16 * st + t; bnd[1] = 16 * st + 4 + t; bnd[2] = 16 * st + 8 + t; bnd[3] = 16 * st + 12 + t; }
            else { bnd[0] = 16 * st + 2 * t; bnd[1] = bnd[0] + 1; bnd[2] = 16 * st + 8 + 2 * t; bnd[3] = bnd[2] + 1; }
            uint32_t m[4] = {0u, 0u, 0u, 0u};
            if (g < G) {
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const float v = p.mw[qh * kBands + bnd[x]];
                    if (KEY8) {
                        const uint32_t hi = f16_bits(v);
                        m[x] = part == 0 ? hi : f16_bits(v - f16_value(hi));
                    } else {
                        const uint32_t hi = bf16_hi_bits(v);
                        m[x] = part == 0 ? hi : bf16_hi_bits(v - __uint_as_float(hi << 16));
                    }
                }
            }
            normB[nt][st][ln] = make_uint2(m[0] | (m[1] << 16), m[2] | (m[3] << 16));
        }
    }
    __syncthreads();

    const int q = lane >> 2, t = lane & 3;
    float s1[NT], s2[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { s1[nt] = 0.f; s2[nt] = 0.f; }
    // ldmatrix source of this lane inside a tile: row lane%16, 16-byte chunk 2*(s%4) + lane/16 of half s/4,
    // chunk index XORed with row%8 (128-byte swizzle)
    const int lrow = lane & 15, lsel = lane >> 4;
    float *rawu = p.raw + (int64_t)u * p.src.n_max * G;
    bool timed_out = false;

    for (int it = 0; it < my_n; ++it) {
        const int stage = it % kStages;
        const uint32_t bar = my_bars + stage * 8, base = my_tiles + stage * kTileB;
        if (!mbar_wait_bounded(bar, (it / kStages) & 1)) { timed_out = true; break; }
        uint32_t X[8][4];
        if (KEY8) {
            // one ldmatrix.x4 per 32 dims: registers = (row q | row q+8) x (dims 4t..4t+3 | 16+4t..16+4t+3) of the step;
            // each widens to the A fragments of two f16 MMAs (slots: dims 4t, 4t+1 | row+8 | dims 4t+2, 4t+3 | row+8)
#pragma unroll
            for (int s32 = 0; s32 < 4; ++s32) {
                uint32_t r[4];
                const int c = 2 * s32 + lsel;
                ldmatrix_x4(r, base + lrow * 128 + ((c ^ (lrow & 7)) << 4));
                e4m3x4_to_f16x2(r[0], X[2 * s32][0], X[2 * s32][2]);
                e4m3x4_to_f16x2(r[1], X[2 * s32][1], X[2 * s32][3]);
                e4m3x4_to_f16x2(r[2], X[2 * s32 + 1][0], X[2 * s32 + 1][2]);
                e4m3x4_to_f16x2(r[3], X[2 * s32 + 1][1], X[2 * s32 + 1][3]);
            }
        } else {
#pragma unroll
            for (int st = 0; st < 8; ++st) {
                const int c = 2 * (st & 3) + lsel;
                ldmatrix_x4(X[st], base + (st >> 2) * (kTileBytes / 2) + lrow * 128 + ((c ^ (lrow & 7)) << 4));
            }
        }
        __syncwarp();
        if (lane == 0 && it + kStages < my_n) {
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            issue(it + kStages);
        }

        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
        for (int st = 0; st < 8; ++st) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                uint2 b = trigB[nt][st][lane];
                if (KEY8) mma_f16_16816(acc[nt], X[st][0], X[st][1], X[st][2], X[st][3], b.x, b.y);
                else mma_bf16_16816(acc[nt], X[st][0], X[st][1], X[st][2], X[st][3], b.x, b.y);
            }
        }
#pragma unroll
        for (int pr = 0; pr < 4; ++pr) {
            uint32_t hA[4], lA[4];
            if (LAYOUT == 0) {
                const uint32_t *a = X[2 * pr], *b = X[2 * pr + 1];      // one register = (re, im) of one band
                mag_pair<false, KEY8>(a[0], a[2], hA[0], lA[0]);
                mag_pair<false, KEY8>(a[1], a[3], hA[1], lA[1]);
                mag_pair<false, KEY8>(b[0], b[2], hA[2], lA[2]);
                mag_pair<false, KEY8>(b[1], b[3], hA[3], lA[3]);
            } else {
                const uint32_t *re = X[pr], *im = X[pr + 4];            // two bands per register, re and im apart
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    mag_pair<true, KEY8>(re[x], im[x], hA[x], lA[x]);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint2 b = normB[nt][pr][lane];
                if (KEY8) {
                    mma_f16_16816(acc[nt], hA[0], hA[1], hA[2], hA[3], b.x, b.y);
                    mma_f16_16816(acc[nt], lA[0], lA[1], lA[2], lA[3], b.x, b.y);
                } else {
                    mma_bf16_16816(acc[nt], hA[0], hA[1], hA[2], hA[3], b.x, b.y);
                    mma_bf16_16816(acc[nt], lA[0], lA[1], lA[2], lA[3], b.x, b.y);
                }
            }
        }

        // columns (2t, 2t+1) of MMA tile nt are the hi and lo halves of head 4nt + t
        const int r0 = key_begin + (warp + kScoreWarps * it) * kTileKeys + q, r1 = r0 + 8;
        const bool v0 = r0 < key_end, v1 = r1 < key_end;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int g = 4 * nt + t;
            const float y0 = acc[nt][0] + acc[nt][1], y1 = acc[nt][2] + acc[nt][3];
            if (g < G) {
                if (v0) { rawu[(int64_t)r0 * G + g] = y0; s1[nt] += y0; s2[nt] = fmaf(y0, y0, s2[nt]); }
                if (v1) { rawu[(int64_t)r1 * G + g] = y1; s1[nt] += y1; s2[nt] = fmaf(y1, y1, s2[nt]); }
            }
        }
    }
    if (timed_out) {
        // a copy did not land within the bound: report it, give copies still in flight one more bounded
        // chance to land in this block's shared memory, and fall through to the block's normal exit
        if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_TIMEOUT);
        for (int st = 0; st < kStages; ++st) (void)mbar_wait_bounded(my_bars + st * 8, 0);
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

// One warp, one barrier that never completes: the wait must run out and report it (see tri_selftest_bounded_wait).
__global__ void k_selftest_wait(int32_t *device_status)
{
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    const bool done = mbar_wait_bounded(b, 0, 1u << 12);
    if (!done && threadIdx.x == 0) atomicExch(device_status, (int)TRI_ERR_TIMEOUT);
}

}  // namespace tri

// Raw scoring of bf16 post-RoPE keys on the 5th-generation tensor cores: TMA -> swizzled shared memory ->
// tcgen05.mma with the accumulator in tensor memory.
//
// A thread block streams its chunk of one unit in tiles of 128 keys.  Per tile:
//   producer warp   bulk-tensor copies of the 128 rows (16 boxes of 16 rows x 64 dims, 128-byte swizzle) into one of
//                   two key stages; the stage doubles as the K-major A operand of the trigonometric contraction
//   8 compute warps two threads per key row read the row back from shared memory, form the 64 band magnitudes
//                   |k_f| (packed f32x2 arithmetic, sqrt.approx), split each into a bf16 and the bf16 of its
//                   residual, and store them as a second K-major A operand (64 "hi" columns | 64 "lo" columns)
//   MMA warp        one thread issues 8 + 8 tcgen05.mma (M = 128 keys, N = NCOL, K = 16 each):
//                       acc  = K_tile [128 x 128] * Wsplit^T     W_f^(g) = E[q_f] e^{i omega_f p_q} Dbar_f  (Sections 4.1, 4.2)
//                       acc += Mag    [128 x 128] * msplit^T     m_f = weight of |k_f| in the norm term      (Section 4.2)
//                   column 2g of the accumulator is the bf16 part of head g's weights, column 2g + 1 the bf16 of
//                   their residual, so S~^(g) = acc[2g] + acc[2g + 1]; then tcgen05.commit frees the key stage and
//                   publishes the accumulator (two accumulators alternate)
//   compute warps   (one tile later, under the next tile's MMAs) tcgen05.ld their row's columns, add the two
//                   halves, store the raw scores and keep sum / sum of squares per head.
// Every mbarrier wait is bounded; a wait that runs out sets TRI_ERR_TIMEOUT in device_status, all roles fall
// through to the common exit, and the tensor memory is released there.
#pragma once
#include <cuda.h>

#include "tri_score_tma.cuh"

namespace tri {

constexpr int kUTile = 128;                              // keys per tile = rows of one tcgen05.mma
constexpr int kUStages = 2;                              // key stages
constexpr int kUBlockBytes = kUTile * 128;               // 16384: 128 rows x 64 bf16, one swizzled K-major block
constexpr int kUTileBytes = 2 * kUBlockBytes;            // dims 0..63 | dims 64..127
constexpr int kUComputeWarps = 8;
constexpr int kUThreads = (kUComputeWarps + 2) * 32;     // + producer warp + MMA warp
constexpr int kUTmemCols = 64;                           // two accumulators of up to 32 columns

constexpr int umma_smem_bytes(int ncol) { return kUStages * kUTileBytes + kUTileBytes + 2 * (2 * ncol * 128) + 1024; }

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_desc_sw128(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = ncol.
__host__ __device__ constexpr uint32_t tc_idesc_bf16(int ncol)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(ncol >> 3) << 17) | ((uint32_t)(kUTile >> 4) << 24);
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float (&v)[8])
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// Byte offset of 16-byte chunk `c` of row `r` inside a swizzled K-major block (rows of 128 bytes).
__device__ __forceinline__ uint32_t sw128(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// NCOL: accumulator columns = 2 per query head, 16 (G <= 8) or 32 (G <= 16).
template <int NCOL, int LAYOUT>
__global__ void __launch_bounds__(kUThreads, NCOL == 16 ? 2 : 1)
k_score_umma(const __grid_constant__ CUtensorMap tmap, const ScoreParams p)
{
    constexpr int HPT = NCOL / 4;                 // heads per compute thread (its half of the columns)
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t bar_kfull[kUStages], bar_kempty[kUStages], bar_accfull[2], bar_magfull;
    __shared__ uint32_t tmem_base_s;
    __shared__ int gave_up;
    __shared__ double red[kUComputeWarps][HPT][2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n || n <= p.skip_upto) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int ntiles = (key_end - key_begin + kUTile - 1) / kUTile;

    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;        // operands need 1024-byte alignment
    const uint32_t sm_k = base, sm_mag = base + kUStages * kUTileBytes, sm_bt = sm_mag + kUTileBytes,
                   sm_bn = sm_bt + 2 * NCOL * 128;
    const uint32_t b_kfull = smem_u32(bar_kfull), b_kempty = smem_u32(bar_kempty), b_accfull = smem_u32(bar_accfull),
                   b_magfull = smem_u32(&bar_magfull);

    // ---------------- set-up ----------------
    if (tid == 0) {
        for (int i = 0; i < kUStages; ++i) { mbar_init(b_kfull + 8 * i, 1); mbar_init(b_kempty + 8 * i, 1); }
        mbar_init(b_accfull, 1); mbar_init(b_accfull + 8, 1);
        mbar_init(b_magfull, kUComputeWarps * 32);
        gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == kUComputeWarps + 1) {             // the MMA warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_s)),
                     "r"(kUTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    // fold, step 2: the two B operands.  Row = accumulator column (2g: bf16 of the weight, 2g + 1: bf16 of its
    // residual), 128 K-major entries per row in two swizzled blocks of 64.
    if (warp < kUComputeWarps) {
        for (int i = tid; i < NCOL * 16; i += kUComputeWarps * 32) {      // one 16-byte chunk (8 entries) per step
            const int col = i >> 4, c16 = i & 15;                        // chunk c16 of row col: entries 8 c16 .. 8 c16 + 7
            const int g = col >> 1, part = col & 1;
            const int64_t qh = (int64_t)l * p.H * G + (int64_t)h * G + g;
            uint32_t wt[8], wn[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                wt[x] = 0u; wn[x] = 0u;
                if (g < G) {
                    const int d = 8 * c16 + x;                          // trig: entry = dim d of the key row
                    const int f = LAYOUT == 0 ? d >> 1 : d & (kBands - 1);
                    const bool imag = LAYOUT == 0 ? (d & 1) : (d >= kBands);
                    const int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
                    const double cr = p.qc[qh * kHeadDim + ir], ci = p.qc[qh * kHeadDim + ii];
                    const double2 e = p.E[s * kBands + f];
                    const float v = imag ? (float)(cr * e.y + ci * e.x) : (float)(cr * e.x - ci * e.y);
                    const uint32_t hi = bf16_hi_bits(v);
                    wt[x] = part == 0 ? hi : bf16_hi_bits(v - __uint_as_float(hi << 16));
                    const float m = p.mw[qh * kBands + (d & (kBands - 1))];   // norm: entry = band (hi block | lo block)
                    const uint32_t mh = bf16_hi_bits(m);
                    wn[x] = part == 0 ? mh : bf16_hi_bits(m - __uint_as_float(mh << 16));
                }
            }
            const uint32_t off = (uint32_t)(c16 >> 3) * (NCOL * 128) + sw128(col, c16 & 7);
            sts128(sm_bt + off, make_uint4(wt[0] | (wt[1] << 16), wt[2] | (wt[3] << 16), wt[4] | (wt[5] << 16), wt[6] | (wt[7] << 16)));
            sts128(sm_bn + off, make_uint4(wn[0] | (wn[1] << 16), wn[2] | (wn[3] << 16), wn[4] | (wn[5] << 16), wn[6] | (wn[7] << 16)));
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp == kUComputeWarps) {
        // ---------------- producer ----------------
        for (int t = 0; t < ntiles; ++t) {
            const int st = t % kUStages;
            bool ok = t < kUStages || mbar_wait_bounded(b_kempty + 8 * st, ((t / kUStages) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { gave_up = 1; break; }
            const int row0 = key_begin + t * kUTile;
            const int nsub = min(kUTile / kTileKeys, (key_end - row0 + kTileKeys - 1) / kTileKeys);
            if (lane == 0) mbar_expect_tx(b_kfull + 8 * st, (uint32_t)nsub * kTileBytes);
            __syncwarp();
            if (lane < 2 * nsub) {
                const int sub = lane >> 1, half = lane & 1;
                const int row = row0 + sub * kTileKeys;
                int c1 = row, c3 = s;
                if (p.src.paged) {
                    const int pg = p.src.page_shift >= 0 ? row >> p.src.page_shift : row / p.src.page_size;
                    int page = __ldg(p.src.page_table + (int64_t)s * p.src.max_pages_per_seq + pg);
                    if (p.src.n_pages > 0 && (page < 0 || page >= p.src.n_pages)) {
                        if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                        page = 0;                      // stay inside the pool; the unit's output is unspecified
                    }
                    c1 = row - pg * p.src.page_size;
                    c3 = page;
                }
                tma_load_5d(sm_k + st * kUTileBytes + half * kUBlockBytes + sub * (kTileKeys * 128), &tmap, b_kfull + 8 * st,
                            half * (kHeadDim / 2), c1, h, c3, l);
            }
        }
    } else if (warp == kUComputeWarps + 1) {
        // ---------------- MMA issue ----------------
        constexpr uint32_t idesc = tc_idesc_bf16(NCOL);
        for (int t = 0; t < ntiles; ++t) {
            const int st = t % kUStages, a = t & 1;
            bool ok = mbar_wait_bounded(b_kfull + 8 * st, (t / kUStages) & 1) && mbar_wait_bounded(b_magfull, t & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { gave_up = 1; break; }
            tc_fence_after();
            if (lane == 0) {
                const uint32_t acc = tmem + a * 32;
                const uint32_t ka = sm_k + st * kUTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    tc_mma_bf16(acc, tc_desc_sw128(ka + (k >> 2) * kUBlockBytes + (k & 3) * 32),
                                tc_desc_sw128(sm_bt + (k >> 2) * (NCOL * 128) + (k & 3) * 32), idesc, k > 0);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    tc_mma_bf16(acc, tc_desc_sw128(sm_mag + (k >> 2) * kUBlockBytes + (k & 3) * 32),
                                tc_desc_sw128(sm_bn + (k >> 2) * (NCOL * 128) + (k & 3) * 32), idesc, 1u);
                tc_commit(b_kempty + 8 * st);      // the stage (and the magnitude buffer) may be overwritten
                tc_commit(b_accfull + 8 * a);      // the accumulator may be read
            }
            __syncwarp();
        }
    } else {
        // ---------------- magnitudes and epilogue ----------------
        const int row = (warp & 3) * 32 + lane;      // key row of the tile = tensor-memory lane this warp may read
        const int hs = warp >> 2;                    // which half of the bands (magnitudes) / of the columns (epilogue)
        const int g0 = hs * HPT;                     // first head of this thread's columns
        float s1[HPT], s2[HPT];
#pragma unroll
        for (int i = 0; i < HPT; ++i) { s1[i] = 0.f; s2[i] = 0.f; }
        float *rawu = p.raw + (int64_t)u * p.src.n_max * G;

        for (int t = 0; t <= ntiles; ++t) {
            bool ok = true;
            if (t < ntiles) ok = mbar_wait_bounded(b_kfull + 8 * (t % kUStages), (t / kUStages) & 1);
            if (ok && t >= 1) ok = mbar_wait_bounded(b_accfull + 8 * ((t - 1) & 1), ((t - 1) >> 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { gave_up = 1; break; }
            tc_fence_after();
            if (t < ntiles) {
                const uint32_t ka = sm_k + (t % kUStages) * kUTileBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {        // 8 bands per step -> one 16-byte chunk of "hi" and one of "lo"
                    uint32_t hi[4], lo[4];
                    if (LAYOUT == 0) {               // a register = (re, im) of one band; block hs holds bands 32 hs ..
                        const uint4 a = lds128(ka + hs * kUBlockBytes + sw128(row, 2 * i));
                        const uint4 b = lds128(ka + hs * kUBlockBytes + sw128(row, 2 * i + 1));
                        mag_pair(bf16_lo(a.x), bf16_hi(a.x), bf16_lo(a.y), bf16_hi(a.y), hi[0], lo[0]);
                        mag_pair(bf16_lo(a.z), bf16_hi(a.z), bf16_lo(a.w), bf16_hi(a.w), hi[1], lo[1]);
                        mag_pair(bf16_lo(b.x), bf16_hi(b.x), bf16_lo(b.y), bf16_hi(b.y), hi[2], lo[2]);
                        mag_pair(bf16_lo(b.z), bf16_hi(b.z), bf16_lo(b.w), bf16_hi(b.w), hi[3], lo[3]);
                    } else {                         // real parts in block 0, imaginary parts in block 1, two bands per register
                        const uint4 re = lds128(ka + sw128(row, 4 * hs + i));
                        const uint4 im = lds128(ka + kUBlockBytes + sw128(row, 4 * hs + i));
                        mag_pair(bf16_lo(re.x), bf16_lo(im.x), bf16_hi(re.x), bf16_hi(im.x), hi[0], lo[0]);
                        mag_pair(bf16_lo(re.y), bf16_lo(im.y), bf16_hi(re.y), bf16_hi(im.y), hi[1], lo[1]);
                        mag_pair(bf16_lo(re.z), bf16_lo(im.z), bf16_hi(re.z), bf16_hi(im.z), hi[2], lo[2]);
                        mag_pair(bf16_lo(re.w), bf16_lo(im.w), bf16_hi(re.w), bf16_hi(im.w), hi[3], lo[3]);
                    }
                    const uint32_t off = sw128(row, 4 * hs + i);          // bands 32 hs + 8 i .. + 7
                    sts128(sm_mag + off, make_uint4(hi[0], hi[1], hi[2], hi[3]));
                    sts128(sm_mag + kUBlockBytes + off, make_uint4(lo[0], lo[1], lo[2], lo[3]));
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                mbar_arrive(b_magfull);
            }
            if (t >= 1 && g0 < G) {
                const int key = key_begin + (t - 1) * kUTile + row;
                const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + ((t - 1) & 1) * 32 + hs * (NCOL / 2);
                float y[HPT];
                {
                    float v[8];
                    tc_ld8(taddr, v);
#pragma unroll
                    for (int i = 0; i < 4; ++i) y[i] = v[2 * i] + v[2 * i + 1];
                    if (HPT == 8) {
                        tc_ld8(taddr + 8, v);
#pragma unroll
                        for (int i = 0; i < 4; ++i) y[(4 + i) % HPT] = v[2 * i] + v[2 * i + 1];
                    }
                }
                if (key < key_end) {
                    float *dst = rawu + (int64_t)key * G + g0;
                    if ((G & 3) == 0) {
#pragma unroll
                        for (int i = 0; i < HPT; i += 4)
                            if (g0 + i < G) *reinterpret_cast<float4 *>(dst + i) = make_float4(y[i], y[i + 1], y[i + 2], y[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < HPT; ++i)
                            if (g0 + i < G) dst[i] = y[i];
                    }
#pragma unroll
                    for (int i = 0; i < HPT; ++i) { s1[i] += y[i]; s2[i] = fmaf(y[i], y[i], s2[i]); }
                }
            }
            tc_fence_before();
        }

        // per-block (sum, sum^2) in a fixed order: lanes (butterfly), then the four warps that share a head
#pragma unroll
        for (int i = 0; i < HPT; ++i) {
            double a = s1[i], b = s2[i];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                a += __shfl_xor_sync(0xffffffffu, a, m);
                b += __shfl_xor_sync(0xffffffffu, b, m);
            }
            if (lane == 0) { red[warp][i][0] = a; red[warp][i][1] = b; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid < G && !gave_up) {
        const int hs = tid / HPT, i = tid - hs * HPT;
        double a = 0.0, b = 0.0;
        for (int w = 0; w < 4; ++w) { a += red[hs * 4 + w][i][0]; b += red[hs * 4 + w][i][1]; }
        p.partials[((int64_t)u * p.nchunks + chunk) * G + tid] = make_double2(a, b);
    }
    if (gave_up) {
        // a wait ran out: report it, and give copies still in flight one more bounded chance to land in this block's
        // shared memory before the block exits
        if (tid == 0 && p.device_status) atomicExch(p.device_status, (int)TRI_ERR_TIMEOUT);
        if (warp == kUComputeWarps)
            for (int t = 0; t < 2 * kUStages; ++t) (void)mbar_wait_bounded(b_kfull + 8 * (t % kUStages), (t / kUStages) & 1, 1u << 16);
    }
    if (warp == kUComputeWarps + 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kUTmemCols) : "memory");
    }
}

}  // namespace tri

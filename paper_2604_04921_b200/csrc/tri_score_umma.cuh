// Raw scoring of bf16 post-RoPE keys on the 5th-generation tensor cores: TMA -> swizzled shared memory ->
// tcgen05.mma with accumulator and magnitude operand in tensor memory.
//
// A thread block streams its chunk of one unit in tiles of 128 keys.  Per tile:
//   producer warp   bulk-tensor copies of the 128 rows (16 boxes of 16 rows x 64 dims, 128-byte swizzle) into one of
//                   three key stages; a stage is at once the K-major A operand of the trigonometric contraction
//   8 compute warps two threads per key row read the row back from shared memory, form the 64 band magnitudes
//                   |k_f| (packed f32x2 arithmetic, sqrt.approx), split each into a bf16 and the bf16 of its
//                   residual and write them with tcgen05.st into tensor memory as a second A operand
//                   (columns: 64 "hi" entries | 64 "lo" entries, two bf16 per 32-bit cell); two such buffers alternate
//   MMA warp        one thread issues 8 + 8 tcgen05.mma (M = 128 keys, N = NCOL, K = 16 each):
//                       acc  = K_tile [128 x 128] * Wsplit^T     W_f^(g) = E[q_f] e^{i omega_f p_q} Dbar_f  (Sections 4.1, 4.2)
//                       acc += Mag    [128 x 128] * msplit^T     m_f = weight of |k_f| in the norm term      (Section 4.2)
//                   the first as soon as the keys have landed, the second when the magnitudes are in place.  Column
//                   2g of the accumulator is the bf16 part of head g's weights, column 2g + 1 the bf16 of their
//                   residual, so S~^(g) = acc[2g] + acc[2g + 1]; tcgen05.commit then frees the key stage and
//                   publishes the accumulator (two accumulators alternate)
//   compute warps   (one tile later, under the next tile's MMAs) tcgen05.ld their row's columns, add the two
//                   halves, store the raw scores and keep sum / sum of squares per head.
// Every mbarrier wait is bounded and sleeps between polls; a wait that runs out sets TRI_ERR_TIMEOUT in device_status, all roles fall
// through to the common exit, and the tensor memory is released there.
#pragma once
#include <cuda.h>

#include "tri_score_tma.cuh"

namespace tri {

constexpr int kUTile = 128;                              // keys per tile = rows of one tcgen05.mma
#ifndef TRI_UMMA_BLOCKS_PER_SM
#define TRI_UMMA_BLOCKS_PER_SM 3
#endif
// Three blocks per SM: two key stages, one magnitude operand, 128 tensor-memory columns each.
// Two blocks per SM: three key stages, two magnitude operands, 256 columns each.
constexpr int kUBlocksPerSM = TRI_UMMA_BLOCKS_PER_SM;
constexpr int kUStages = kUBlocksPerSM == 3 ? 2 : 3;     // key stages
constexpr int kUMagBufs = kUBlocksPerSM == 3 ? 1 : 2;
constexpr int kUBlockBytes = kUTile * 128;               // 16384: 128 rows x 64 bf16, one swizzled K-major block
constexpr int kUTileBytes = 2 * kUBlockBytes;            // dims 0..63 | dims 64..127
constexpr int kUComputeWarps = 8;
constexpr int kUThreads = (kUComputeWarps + 2) * 32;     // + producer warp + MMA warp
constexpr int kUTmemCols = kUBlocksPerSM == 3 ? 128 : 256;   // columns 0..63: two accumulators; from 64: the magnitude operand(s)
constexpr int kUMagCol = 64, kUMagCols = 64;

constexpr int umma_smem_bytes(int ncol) { return kUStages * kUTileBytes + 2 * (2 * ncol * 128) + 1024; }

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
// Bounded wait that sleeps between polls: a warp waiting for another role of the block must not spend the
// issue slots the other blocks of the SM compute with.  One poll at once, then `nap` nanoseconds of sleep before
// each further poll; after kNapPolls polls the caller gives up.
constexpr uint32_t kNapPolls = 1u << 20;
#ifndef TRI_UMMA_NAP
#define TRI_UMMA_NAP 64
#endif
template <uint32_t NAP = TRI_UMMA_NAP>
__device__ __forceinline__ bool mbar_wait_parked(uint32_t bar, uint32_t parity, uint32_t polls = kNapPolls)
{
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < polls; ++i) {
        if (NAP) __nanosleep(NAP);
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}
// Plain (untiled) bulk copy global -> shared, completing on an mbarrier; 16-byte aligned addresses and size.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
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
// The same with the A operand in tensor memory (rows = lanes, two bf16 per 32-bit column).
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_st8_unused(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tc_st4(uint32_t taddr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(taddr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
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
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// Byte offset of 16-byte chunk `c` of row `r` inside a swizzled K-major block (rows of 128 bytes).
__device__ __forceinline__ uint32_t sw128(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// Fold, step 2, for the tcgen05 kernel: the B operands as ready-to-copy shared-memory images.
//   trig  [U][2 blocks][NCOL rows][128 B]   row = accumulator column (2g: bf16 of W^(g), 2g + 1: bf16 of its residual),
//                                           entry d = dim d of the key row; swizzled exactly as the kernel's shared memory
//   norm  [L*H][2 blocks][NCOL rows][128 B] entry k = band k % 64 (block 0 meets the "hi" magnitudes, block 1 the "lo")
// grid = units of the call, 16 * NCOL threads: one 16-byte chunk each.  The norm image does not depend on the
// sequence; the blocks of sequence 0 write it.
struct OperandParams {
    const double2 *E;     // [S][64]
    const float *qc;      // [L][H*G][128]
    const float *mw;      // [L][H*G][64]
    uint8_t *bt, *bn;
    int32_t S, H, G;
};

template <int NCOL, int LAYOUT>
__global__ void __launch_bounds__(NCOL * 16) k_fold_operands(const OperandParams p)
{
    const int u = blockIdx.x, i = threadIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int G = p.G;
    const int col = i >> 4, c16 = i & 15;                        // chunk c16 of row col: entries 8 c16 .. 8 c16 + 7
    const int g = col >> 1, part = col & 1;
    const int64_t qh = (int64_t)l * p.H * G + (int64_t)h * G + g;
    uint32_t wt[8], wn[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        wt[x] = 0u; wn[x] = 0u;
        if (g < G) {
            const int d = 8 * c16 + x;
            const int f = LAYOUT == 0 ? d >> 1 : d & (kBands - 1);
            const bool imag = LAYOUT == 0 ? (d & 1) : (d >= kBands);
            const int ir = LAYOUT == 0 ? 2 * f : f, ii = LAYOUT == 0 ? 2 * f + 1 : f + kBands;
            const double cr = p.qc[qh * kHeadDim + ir], ci = p.qc[qh * kHeadDim + ii];
            const double2 e = p.E[s * kBands + f];
            const float v = imag ? (float)(cr * e.y + ci * e.x) : (float)(cr * e.x - ci * e.y);
            const uint32_t hi = bf16_hi_bits(v);
            wt[x] = part == 0 ? hi : bf16_hi_bits(v - __uint_as_float(hi << 16));
            const float m = p.mw[qh * kBands + (d & (kBands - 1))];
            const uint32_t mh = bf16_hi_bits(m);
            wn[x] = part == 0 ? mh : bf16_hi_bits(m - __uint_as_float(mh << 16));
        }
    }
    const uint32_t off = (uint32_t)(c16 >> 3) * (NCOL * 128) + sw128(col, c16 & 7);
    *reinterpret_cast<uint4 *>(p.bt + (int64_t)u * (NCOL * 256) + off) =
        make_uint4(wt[0] | (wt[1] << 16), wt[2] | (wt[3] << 16), wt[4] | (wt[5] << 16), wt[6] | (wt[7] << 16));
    if (s == 0)
        *reinterpret_cast<uint4 *>(p.bn + ((int64_t)l * p.H + h) * (NCOL * 256) + off) =
            make_uint4(wn[0] | (wn[1] << 16), wn[2] | (wn[3] << 16), wn[4] | (wn[5] << 16), wn[6] | (wn[7] << 16));
}

// NCOL: accumulator columns = 2 per query head, 16 (G <= 8) or 32 (G <= 16).
template <int NCOL, int LAYOUT>
__global__ void __launch_bounds__(kUThreads, NCOL == 16 ? kUBlocksPerSM : kUBlocksPerSM - 1)
k_score_umma(const __grid_constant__ CUtensorMap tmap, const ScoreParams p)
{
    constexpr int HPT = NCOL / 4;                 // heads per compute thread (its half of the columns)
    extern __shared__ uint8_t dyn_smem[];
    __shared__ __align__(8) uint64_t bar_kfull[kUStages], bar_kempty[kUStages], bar_accfull[2], bar_accempty[2], bar_magfull[2], bar_bfull;
    __shared__ uint32_t tmem_base_s;
    __shared__ int gave_up;
    __shared__ double red[kUComputeWarps][HPT][2];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ub = blockIdx.x / p.nchunks, chunk = blockIdx.x - ub * p.nchunks, u = p.u0 + ub;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int n = min(__ldg(p.src.seq_lens + s), p.src.n_max);
    const int key_begin = chunk * p.chunk;
    if (key_begin >= n || n <= skip_limit(p, u)) return;
    const int key_end = min(key_begin + p.chunk, n);
    const int G = p.G;
    const int ntiles = (key_end - key_begin + kUTile - 1) / kUTile;

    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;        // operands need 1024-byte alignment
    const uint32_t sm_k = base, sm_bt = base + kUStages * kUTileBytes, sm_bn = sm_bt + 2 * NCOL * 128;
    const uint8_t *gk = dyn_smem + (base - smem_u32(dyn_smem));        // the key stages through a generic pointer
    const uint32_t b_kfull = smem_u32(bar_kfull), b_kempty = smem_u32(bar_kempty), b_accfull = smem_u32(bar_accfull),
                   b_accempty = smem_u32(bar_accempty), b_magfull = smem_u32(bar_magfull), b_bfull = smem_u32(&bar_bfull);

    // ---------------- set-up ----------------
    if (tid == 0) {
        for (int i = 0; i < kUStages; ++i) { mbar_init(b_kfull + 8 * i, 1); mbar_init(b_kempty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(b_accfull + 8 * i, 1);
            mbar_init(b_accempty + 8 * i, kUComputeWarps);      // one arrival per compute warp
            mbar_init(b_magfull + 8 * i, kUComputeWarps);       // (with one magnitude operand only the first is used)
        }
        mbar_init(b_bfull, 1);
        gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        // the two B operands (weights of the trigonometric and of the norm contraction), folded by k_fold_operands
        mbar_expect_tx(b_bfull, 2 * NCOL * 256);
        bulk_load(sm_bt, p.bt + (int64_t)u * (NCOL * 256), NCOL * 256, b_bfull);
        bulk_load(sm_bn, p.bn + ((int64_t)l * p.H + h) * (NCOL * 256), NCOL * 256, b_bfull);
    }
    if (warp == kUComputeWarps + 1) {             // the MMA warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_s)),
                     "r"(kUTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp == kUComputeWarps) {
        // ---------------- producer ----------------
        // lane (2 sub + half) copies one 16-row box of a tile.  Where its box of tile t lies (for paged keys a page-table
        // entry) is looked up one tile ahead, so that the lookup's latency is spent under the wait for the stage, not after it
        const int sub = lane >> 1, half = lane & 1;
        auto locate = [&](int t, int &c1, int &c3) {
            const int row = key_begin + t * kUTile + sub * kTileKeys;
            c1 = row; c3 = s;
            if (p.src.paged && t < ntiles && row < key_end) {
                const int pg = p.src.page_shift >= 0 ? row >> p.src.page_shift : row / p.src.page_size;
                int page = __ldg(p.src.page_table + (int64_t)s * p.src.max_pages_per_seq + pg);
                if (p.src.n_pages > 0 && (page < 0 || page >= p.src.n_pages)) {
                    if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                    page = 0;                      // stay inside the pool; the unit's output is unspecified
                }
                c1 = row - pg * p.src.page_size;
                c3 = page;
            }
        };
        int c1, c3;
        locate(0, c1, c3);
        for (int t = 0; t < ntiles; ++t) {
            const int st = t % kUStages;
            bool ok = t < kUStages || mbar_wait_parked(b_kempty + 8 * st, ((t / kUStages) - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { gave_up = 1; break; }
            const int row0 = key_begin + t * kUTile;
            const int nsub = min(kUTile / kTileKeys, (key_end - row0 + kTileKeys - 1) / kTileKeys);
            if (lane == 0) mbar_expect_tx(b_kfull + 8 * st, (uint32_t)nsub * kTileBytes);
            __syncwarp();
            if (lane < 2 * nsub)
                tma_load_5d(sm_k + st * kUTileBytes + half * kUBlockBytes + sub * (kTileKeys * 128), &tmap, b_kfull + 8 * st,
                            half * (kHeadDim / 2), c1, h, c3, l);
            locate(t + 1, c1, c3);
        }
    } else if (warp == kUComputeWarps + 1) {
        // ---------------- MMA issue ----------------
        constexpr uint32_t idesc = tc_idesc_bf16(NCOL);
        if (!__all_sync(0xffffffffu, mbar_wait_parked(b_bfull, 0))) gave_up = 1;
        for (int t = 0; t < ntiles && !gave_up; ++t) {
            const int st = t % kUStages, a = t & 1;
            const uint32_t acc = tmem + a * 32;
            // trigonometric part: needs the keys, and the accumulator read out by the epilogue of tile t - 2
            bool ok = mbar_wait_parked(b_kfull + 8 * st, (t / kUStages) & 1) &&
                      (t < 2 || mbar_wait_parked(b_accempty + 8 * a, ((t >> 1) - 1) & 1));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { gave_up = 1; break; }
            tc_fence_after();
            if (lane == 0) {
                const uint32_t ka = sm_k + st * kUTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    tc_mma_bf16(acc, tc_desc_sw128(ka + (k >> 2) * kUBlockBytes + (k & 3) * 32),
                                tc_desc_sw128(sm_bt + (k >> 2) * (NCOL * 128) + (k & 3) * 32), idesc, k > 0);
            }
            __syncwarp();
            // norm part: needs the magnitudes of this tile
            const int mb = kUMagBufs == 2 ? a : 0;
            ok = __all_sync(0xffffffffu, mbar_wait_parked(b_magfull + 8 * mb, (kUMagBufs == 2 ? t >> 1 : t) & 1));
            if (!ok) { gave_up = 1; break; }
            tc_fence_after();
            if (lane == 0) {
                // the key stage has served both its readers (the trigonometric MMAs issued above and the compute warps,
                // whose arrival was just seen): it may be refilled as soon as those MMAs have completed
                tc_commit(b_kempty + 8 * st);
                const uint32_t mag = tmem + kUMagCol + mb * kUMagCols;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    tc_mma_bf16_ts(acc, mag + 8 * k, tc_desc_sw128(sm_bn + (k >> 2) * (NCOL * 128) + (k & 3) * 32), idesc, 1u);
                tc_commit(b_accfull + 8 * a);      // the accumulator may be read, the magnitude buffer rewritten
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

        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        for (int t = 0; t <= ntiles; ++t) {
            if (t < ntiles) {
                // magnitudes of tile t.  Their buffer is free once the MMAs that read it last have completed: those of
                // tile t - 2 with two buffers (this thread saw them complete before its last epilogue), of tile t - 1 with one.
                bool ok = mbar_wait_parked(b_kfull + 8 * (t % kUStages), (t / kUStages) & 1);
                if (kUMagBufs == 1 && t >= 1) ok = ok && mbar_wait_parked(b_accfull + 8 * ((t - 1) & 1), ((t - 1) >> 1) & 1);
                if (!__all_sync(0xffffffffu, ok)) { gave_up = 1; break; }
                tc_fence_after();
                const uint8_t *ka = gk + (t % kUStages) * kUTileBytes;
                const int mb = kUMagBufs == 2 ? (t & 1) : 0;
                const uint32_t mag = tmem + lane_base + kUMagCol + mb * kUMagCols + 16 * hs;
#pragma unroll
                for (int i = 0; i < 4; ++i) {        // 8 bands per step -> 4 "hi" cells and 4 "lo" cells
                    uint4 a, b;
                    uint32_t hi[4], lo[4];
                    if (LAYOUT == 0) {               // block hs holds bands 32 hs .. 32 hs + 31; a register = (re, im) of one band
                        a = *reinterpret_cast<const uint4 *>(ka + hs * kUBlockBytes + sw128(row, 2 * i));
                        b = *reinterpret_cast<const uint4 *>(ka + hs * kUBlockBytes + sw128(row, 2 * i + 1));
                        mag_pair<false>(a.x, a.y, hi[0], lo[0]);
                        mag_pair<false>(a.z, a.w, hi[1], lo[1]);
                        mag_pair<false>(b.x, b.y, hi[2], lo[2]);
                        mag_pair<false>(b.z, b.w, hi[3], lo[3]);
                    } else {                         // a = real parts (block 0), b = imaginary parts (block 1), two bands per register
                        a = *reinterpret_cast<const uint4 *>(ka + sw128(row, 4 * hs + i));
                        b = *reinterpret_cast<const uint4 *>(ka + kUBlockBytes + sw128(row, 4 * hs + i));
                        mag_pair<true>(a.x, b.x, hi[0], lo[0]);
                        mag_pair<true>(a.y, b.y, hi[1], lo[1]);
                        mag_pair<true>(a.z, b.z, hi[2], lo[2]);
                        mag_pair<true>(a.w, b.w, hi[3], lo[3]);
                    }
                    tc_st4(mag + 4 * i, hi[0], hi[1], hi[2], hi[3]);
                    tc_st4(mag + 32 + 4 * i, lo[0], lo[1], lo[2], lo[3]);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(b_magfull + 8 * mb);
            }
            if (t >= 1) {
                // epilogue of tile t - 1
                const int a = (t - 1) & 1;
                const bool ok = __all_sync(0xffffffffu, mbar_wait_parked(b_accfull + 8 * a, ((t - 1) >> 1) & 1));
                if (!ok) { gave_up = 1; break; }
                tc_fence_after();
                float y[HPT];
                if (g0 < G) {
                    const uint32_t taddr = tmem + lane_base + a * 32 + hs * (NCOL / 2);
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
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(b_accempty + 8 * a);     // the accumulator may be overwritten
                const int key = key_begin + (t - 1) * kUTile + row;
                if (g0 < G && key < key_end) {
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
            for (int t = 0; t < 2 * kUStages; ++t) (void)mbar_wait_parked(b_kfull + 8 * (t % kUStages), (t / kUStages) & 1);
    }
    if (warp == kUComputeWarps + 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kUTmemCols) : "memory");
    }
}

// The sleeping wait on a barrier that nothing completes: it must run out.  Leaves *device_status alone if it does (the
// spinning self-test before it has set TRI_ERR_TIMEOUT there) and overwrites it with TRI_ERR_DEVICE_CHECK if the wait
// claims success.
__global__ void k_selftest_nap(int32_t *device_status)
{
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    const bool done = mbar_wait_parked(b, 0, 1u << 8);
    if (done && threadIdx.x == 0) atomicExch(device_status, (int)TRI_ERR_DEVICE_CHECK);
}

}  // namespace tri

// Calibration statistics (Sections 3.3 and 4.1, Appendix B.5) with the query rows staged by the TMA unit.
//
// Same sums, same lane -> slot mapping and the same two-level fp32 / fp64 accumulation as k_calib_partial; what
// changes is how the rows reach the registers.  The queries are described to the TMA unit as a rank-3 tensor
// (component, head, token).  Every warp runs its own pipeline over 4 KB tiles (16 bf16 rows or 8 fp32 rows of one
// head): lane 0 issues one tiled bulk-tensor load per tile that completes on a per-(warp, stage) mbarrier, the warp
// waits (bounded), pulls the tile into registers with one shared-memory load per row at a constant offset, and
// re-arms the stage at once.  The copy engine does the strided addressing and fills rows past the last token with
// zeros, which add nothing to any sum: the arithmetic loop carries no address computation and no bounds check,
// about half the instructions per row of the version on plain loads.
//
// Needs what the TMA unit needs: a 16-byte aligned base and strides that are multiples of 16 bytes; other inputs
// take k_calib_partial.
#pragma once
#include "tri_calib.cuh"
#include "tri_score_tma.cuh"

namespace tri {

#ifndef TRI_CALIB_STAGES
#define TRI_CALIB_STAGES 2
#endif
constexpr int kCalibStages = TRI_CALIB_STAGES;
constexpr int kCalibTileBytes = 4096;
constexpr int kCalibDynSmem = kCalibWarps * kCalibStages * kCalibTileBytes;   // 65536: three blocks per SM

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];\n" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// grid (blocks, heads): a block owns the tokens [blockIdx.x * per_block, +per_block) of one head; per_block is a
// multiple of the tile height, so a tile never straddles two blocks and only the TMA unit sees the ragged end.
template <int LAYOUT, int KIND>
__global__ void __launch_bounds__(kCalibThreads, 6 / kCalibStages) k_calib_tma(const __grid_constant__ CUtensorMap tmap, const CalibParams p)
{
    constexpr int ROWB = KIND == 0 ? 256 : 512;          // bytes per row
    constexpr int ROWS = kCalibTileBytes / ROWB;         // rows per tile
    extern __shared__ __align__(1024) uint8_t stage_mem[];   // [warp][stage][4096]; reused for the block reduction
    __shared__ __align__(8) uint64_t bars[kCalibWarps][kCalibStages];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int head = blockIdx.y;
    const int64_t t_begin = (int64_t)blockIdx.x * p.per_block;
    const int64_t t_end = min(t_begin + (int64_t)p.per_block, p.T);
    const int ntiles = (int)((t_end - t_begin + ROWS - 1) / ROWS);
    const int my_n = warp < ntiles ? (ntiles - warp + kCalibWarps - 1) / kCalibWarps : 0;
    const uint32_t my_tiles = smem_u32(stage_mem) + warp * (kCalibStages * kCalibTileBytes);
    const uint32_t my_bars = smem_u32(&bars[warp][0]);

    auto issue = [&](int it) {
        const int stage = it % kCalibStages;
        const uint32_t bar = my_bars + stage * 8;
        mbar_expect_tx(bar, kCalibTileBytes);
        tma_load_3d(my_tiles + stage * kCalibTileBytes, &tmap, bar, 0, head,
                    (int)(t_begin + (int64_t)(warp + kCalibWarps * it) * ROWS));
    };
    if (lane == 0) {
        for (int st = 0; st < kCalibStages; ++st) mbar_init(my_bars + st * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        for (int it = 0; it < kCalibStages && it < my_n; ++it) issue(it);
    }
    __syncwarp();

    double acc[8];
    float part[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { acc[i] = 0.0; part[i] = 0.f; }
    int pending = 0;
    bool timed_out = false;
    for (int it = 0; it < my_n; ++it) {
        const int stage = it % kCalibStages;
        const uint32_t bar = my_bars + stage * 8, base = my_tiles + stage * kCalibTileBytes;
        if (!mbar_wait_bounded(bar, (it / kCalibStages) & 1)) { timed_out = true; break; }
        uint4 raw[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            raw[r] = make_uint4(0u, 0u, 0u, 0u);
            if (KIND == 0)
                asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(raw[r].x), "=r"(raw[r].y) : "r"(base + r * ROWB + lane * 8));
            else
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                             : "=r"(raw[r].x), "=r"(raw[r].y), "=r"(raw[r].z), "=r"(raw[r].w) : "r"(base + r * ROWB + lane * 16));
        }
        __syncwarp();
        if (lane == 0 && it + kCalibStages < my_n) {
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            issue(it + kCalibStages);
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const float4 x = widen<KIND>(raw[r]);
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
        pending += ROWS;
        if (pending >= kCalibFlush) {
#pragma unroll
            for (int i = 0; i < 8; ++i) { acc[i] += (double)part[i]; part[i] = 0.f; }
            pending = 0;
        }
    }
    if (timed_out) {
        // a copy did not land within the bound: give the copies still in flight one more bounded chance to land in
        // this block's shared memory, then poison this warp's sums so that the pass's results read NaN
        for (int st = 0; st < kCalibStages; ++st) (void)mbar_wait_bounded(my_bars + st * 8, 0);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = __longlong_as_double(0x7ff8000000000000ll);
    }
    __syncthreads();                                   // every warp is done with its stages
    double (*red)[32][8] = reinterpret_cast<double (*)[32][8]>(stage_mem);
#pragma unroll
    for (int i = 0; i < 8; ++i) red[warp][lane][i] = acc[i] + (double)part[i];
    __syncthreads();
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

}  // namespace tri

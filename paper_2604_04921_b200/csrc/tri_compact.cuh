// Eviction as an order-preserving gather (Section 4.3): dst row j <- src row kept_idx[j] for K, V and
// the slot's original position.  Rows are moved as 16-byte vectors, bit for bit.
#pragma once
#include "tri_common.cuh"

namespace tri {

constexpr int kGatherThreads = 256;
constexpr int kGatherWarps = kGatherThreads / 32;
constexpr int kGatherRowsPerWarp = 8;
constexpr int kGatherRowsPerBlock = kGatherWarps * kGatherRowsPerWarp;   // 64

struct CompactParams {
    View src, dst;
    const int32_t *kept_idx;   // [U][budget]
    const int32_t *kept_cnt;   // [U]
    int32_t *new_seq_lens;     // [S] or NULL
    int32_t S, H, budget;
    int32_t k_vec;             // 16-byte vectors per K row (16 for bf16, 32 for fp32)
    int32_t v_vec;             // 16-byte vectors per V row (16, or 0 without a value cache)
    int32_t k_esize;           // bytes per K element
    int32_t *device_status;
};

__device__ __forceinline__ uint4 ld_once(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ void st_once(void *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Out-of-place gather.  grid = (U, ceil(budget / 64)); a warp moves 8 rows at a time, lanes 0..15
// carry the K row and lanes 16..31 the V row (bf16), so every access is a full 256-byte row.
__global__ void __launch_bounds__(kGatherThreads) k_gather(const CompactParams p)
{
    const int u = blockIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int cnt = min(__ldg(p.kept_cnt + u), p.budget);
    if (blockIdx.y == 0 && threadIdx.x == 0 && p.new_seq_lens && h == 0 && l == 0) p.new_seq_lens[s] = cnt;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int j0 = blockIdx.y * kGatherRowsPerBlock + warp * kGatherRowsPerWarp;
    if (j0 >= cnt) return;
    const int32_t *idx = p.kept_idx + (int64_t)u * p.budget;
    const int per_row = p.k_vec + p.v_vec;                 // 32 for bf16 K + V

    int src_row[kGatherRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kGatherRowsPerWarp; ++r) {
        src_row[r] = (j0 + r < cnt) ? __ldg(idx + j0 + r) : -1;
        if (src_row[r] >= p.src.n_max) {        // an index outside the unit: report, do not dereference
            if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
            src_row[r] = -1;
        }
    }

    for (int c = lane; c < per_row; c += 32) {
        const bool is_k = c < p.k_vec;
        const char *sb = is_k ? p.src.k : p.src.v;
        char *db = is_k ? p.dst.k : p.dst.v;
        const int esz = is_k ? p.k_esize : 2;
        const int cb = (is_k ? c : c - p.k_vec) * 16;
        uint4 val[kGatherRowsPerWarp];
        int64_t doff[kGatherRowsPerWarp];
#pragma unroll
        for (int r = 0; r < kGatherRowsPerWarp; ++r) {
            doff[r] = -1;
            if (src_row[r] >= 0) {
                int64_t so = row_offset(p.src, l, s, h, src_row[r]);
                doff[r] = row_offset(p.dst, l, s, h, j0 + r);
                if (so < 0 || doff[r] < 0) {
                    if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                    doff[r] = -1;
                } else {
                    val[r] = ld_once(sb + so * esz + cb);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kGatherRowsPerWarp; ++r)
            if (doff[r] >= 0) st_once(db + doff[r] * esz + cb, val[r]);
    }
    if (p.dst.positions) {   // lane r moves row r's position
        int my = -1;
#pragma unroll
        for (int r = 0; r < kGatherRowsPerWarp; ++r) if (lane == r) my = src_row[r];
        if (my >= 0) {
            int pos = p.src.positions ? p.src.positions[(int64_t)u * p.src.n_max + my] : my;
            p.dst.positions[(int64_t)u * p.dst.n_max + j0 + lane] = pos;
        }
    }
}

// In-place (or aliasing) compaction: one block per unit walks the kept rows in ascending tiles.
// Every row of a tile is staged in shared memory before any row of the tile is written; since
// kept_idx[j] >= j and is increasing, a tile's destinations lie strictly below every source of the
// following tiles, so no source is overwritten before it has been read.
constexpr int kInplaceThreads = 512;
constexpr int kInplaceRows = 32;        // rows per tile: 32 x (512 B K + 256 B V) <= 24 KB

__global__ void __launch_bounds__(kInplaceThreads) k_compact_inplace(const CompactParams p)
{
    __shared__ uint4 stage[kInplaceRows * 48];
    __shared__ int32_t pos_s[kInplaceRows];
    const int u = blockIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int cnt = min(__ldg(p.kept_cnt + u), p.budget);
    if (threadIdx.x == 0 && p.new_seq_lens && h == 0 && l == 0) p.new_seq_lens[s] = cnt;
    const int32_t *idx = p.kept_idx + (int64_t)u * p.budget;
    const int per_row = p.k_vec + p.v_vec;

    for (int j0 = 0; j0 < cnt; j0 += kInplaceRows) {
        const int rows = min(kInplaceRows, cnt - j0);
        for (int i = threadIdx.x; i < rows * per_row; i += kInplaceThreads) {
            int r = i / per_row, c = i - r * per_row;
            int srow = __ldg(idx + j0 + r);
            int64_t so = (srow >= 0 && srow < p.src.n_max) ? row_offset(p.src, l, s, h, srow) : -1;
            const bool is_k = c < p.k_vec;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (so < 0) { if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK); }
            else v = is_k ? ld_once(p.src.k + so * p.k_esize + c * 16)
                          : ld_once(p.src.v + so * 2 + (c - p.k_vec) * 16);
            stage[i] = v;
        }
        if (p.dst.positions && threadIdx.x < rows) {
            int srow = min(max(__ldg(idx + j0 + threadIdx.x), 0), p.src.n_max - 1);
            pos_s[threadIdx.x] = p.src.positions ? p.src.positions[(int64_t)u * p.src.n_max + srow] : srow;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < rows * per_row; i += kInplaceThreads) {
            int r = i / per_row, c = i - r * per_row;
            int64_t dof = row_offset(p.dst, l, s, h, j0 + r);
            const bool is_k = c < p.k_vec;
            if (dof < 0) { if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK); }
            else if (is_k) *reinterpret_cast<uint4 *>(p.dst.k + dof * p.k_esize + c * 16) = stage[i];
            else *reinterpret_cast<uint4 *>(p.dst.v + dof * 2 + (c - p.k_vec) * 16) = stage[i];
        }
        if (p.dst.positions && threadIdx.x < rows)
            p.dst.positions[(int64_t)u * p.dst.n_max + j0 + threadIdx.x] = pos_s[threadIdx.x];
        __syncthreads();
    }
}

}  // namespace tri

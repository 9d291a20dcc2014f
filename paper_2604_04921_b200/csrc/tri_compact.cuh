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
    int32_t u0;                // first unit of this launch
    int32_t k_vec;             // 16-byte vectors per K row (16 for bf16, 32 for fp32, 8 for fp8)
    int32_t v_vec;             // 16-byte vectors per V row (16, 8 for fp8, or 0 without a value cache)
    int32_t k_esize;           // bytes per K element
    int32_t v_esize;           // bytes per V element
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

// The same streaming load without the read-only (.nc) path: for kernels that later overwrite the buffer they read.
__device__ __forceinline__ uint4 ld_stream(const void *p)
{
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p)
                 : "memory");
    return r;
}

__device__ __forceinline__ void st_once(void *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Gather of bf16 K and V rows (the common case), contiguous or paged on either side.
// grid = (U, ceil(budget / kFastRowsPerBlock)).  Lanes 0..15 of a warp carry a K row and lanes 16..31
// the V row of the same slot, 16 bytes each, so every access is a whole 256-byte row.  A warp keeps
// kFastRows rows in flight (all loads issued before the first store) and walks kFastIters such groups.
// Lane r < kFastRows resolves the addresses of row r of the group (index load, page-table lookups) and
// hands them to the other lanes by shuffle, so the address work is done once per row, not per lane;
// that keeps the kernel at 64 registers, four blocks per SM.
//
// AFTER_PREFIX = true is the second phase of an in-place compaction: it moves only the row tiles that
// k_compact_inplace_rows left alone (tiles whose first source lies at or beyond the kept count), whose sources
// are all outside the destination range [0, count) -- see k_compact_inplace_rows.
constexpr int kFastRows = 8;
constexpr int kFastIters = 2;
constexpr int kFastRowsPerBlock = kGatherWarps * kFastRows * kFastIters;
constexpr int kInplaceRows = 128;       // rows per tile of the in-place schedule

// ESZ = bytes per element: 2 = bf16 rows as described; 1 = e4m3 rows of 128 bytes, 8 lanes per row, so a half-warp
// carries the K and V row of one slot and a warp two slots at a time (16 rows in flight per warp).
template <bool AFTER_PREFIX, int ESZ = 2>
__global__ void __launch_bounds__(kGatherThreads, 4) k_gather_rows(const CompactParams p)
{
    constexpr int kPieces = 8 * ESZ;                 // 16-byte pieces per row
    constexpr int kSlots = 16 / kPieces;             // slots a warp moves per step: 1 or 2
    constexpr int kGroup = kFastRows * kSlots;       // rows in flight per warp
    const int u = p.u0 + blockIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int cnt = min(__ldg(p.kept_cnt + u), p.budget);
    if (!AFTER_PREFIX && blockIdx.y == 0 && threadIdx.x == 0 && p.new_seq_lens && h == 0 && l == 0)
        p.new_seq_lens[s] = cnt;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int jw = blockIdx.y * (kFastRowsPerBlock * kSlots) + warp * (kGroup * kFastIters);
    if (jw >= cnt) return;
    const int32_t *idx = p.kept_idx + (int64_t)u * p.budget;
    const bool is_v = (lane / kPieces) & 1;
    const int sub = lane / (2 * kPieces);            // which of the step's slots this lane works on
    const char *sb = (is_v ? p.src.v : p.src.k) + (lane % kPieces) * 16;
    char *db = (is_v ? p.dst.v : p.dst.k) + (lane % kPieces) * 16;
    const int n_src = p.src.n_max;

#pragma unroll 1
    for (int it = 0; it < kFastIters; ++it) {
        const int j0 = jw + it * kGroup;
        if (j0 >= cnt) break;
        if (AFTER_PREFIX && __ldg(idx + (j0 & ~(kInplaceRows * kSlots - 1))) < cnt) continue;   // the first phase moved this tile
        // lane r resolves row j0 + r; rows past the count, indices outside the unit and bad page ids are skipped
        int mine = -1;
        int64_t so = -1, dof = -1;
        if (lane < kGroup && j0 + lane < cnt) {
            mine = __ldg(idx + j0 + lane);
            if (mine >= 0 && mine < n_src) {
                so = row_offset(p.src, l, s, h, mine);
                dof = row_offset(p.dst, l, s, h, j0 + lane);
            }
            if (so < 0 || dof < 0) {
                if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                mine = -1; so = -1; dof = -1;
            }
        }
        uint4 val[kFastRows];
#pragma unroll
        for (int r = 0; r < kFastRows; ++r) {
            const int64_t o = __shfl_sync(0xffffffffu, so, r * kSlots + sub);
            if (o >= 0) val[r] = AFTER_PREFIX ? ld_stream(sb + o * ESZ) : ld_once(sb + o * ESZ);   // in place: no read-only path
        }
#pragma unroll
        for (int r = 0; r < kFastRows; ++r) {
            const int64_t o = __shfl_sync(0xffffffffu, dof, r * kSlots + sub);
            if (o >= 0) st_once(db + o * ESZ, val[r]);
        }
        if (p.dst.positions && mine >= 0)
            p.dst.positions[(int64_t)u * p.dst.n_max + j0 + lane] =
                p.src.positions ? p.src.positions[(int64_t)u * p.src.n_max + mine] : mine;
    }
}

// Out-of-place gather for the remaining cases (fp32 keys, no value cache).
// grid = (U, ceil(budget / 64)); a warp moves 8 rows at a time, 16 bytes per lane.
__global__ void __launch_bounds__(kGatherThreads) k_gather_any(const CompactParams p)
{
    const int u = p.u0 + blockIdx.x;
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
        const int esz = is_k ? p.k_esize : p.v_esize;
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
// Every row of a tile is read before any row of the tile is written; since kept_idx[j] >= j and is
// increasing, a tile's destinations lie strictly below every source of the following tiles, so no source
// is overwritten before it has been read.  Rows already in their slot (kept_idx[j] == j) are not touched.
//
// k_compact_inplace_rows (bf16 K + V): a tile is 128 rows, 8 per warp, held in registers between the loads
// and the one block barrier that separates them from the stores (lanes and address hand-off as in
// k_gather_rows).  It stops at the first tile whose first source index is >= the kept count: from there on
// every source lies outside the destination range [0, count), nothing can be overwritten before it is read,
// and k_gather_rows<true> moves those tiles with full parallelism in the next launch (its destinations,
// beyond the prefix, are never sources of the prefix, whose sources were all read here first).
constexpr int kInplaceThreads = 512;
static_assert(kInplaceRows == (kInplaceThreads / 32) * kFastRows, "a tile is 8 rows per warp");

// ESZ as in k_gather_rows: with 128-byte rows a warp holds 16 rows and a tile is 256 rows.
template <int ESZ = 2>
__global__ void __launch_bounds__(kInplaceThreads, 2) k_compact_inplace_rows(const CompactParams p)
{
    constexpr int kPieces = 8 * ESZ, kSlots = 16 / kPieces, kGroup = kFastRows * kSlots;
    const int u = p.u0 + blockIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int cnt = min(__ldg(p.kept_cnt + u), p.budget);
    if (threadIdx.x == 0 && p.new_seq_lens && h == 0 && l == 0) p.new_seq_lens[s] = cnt;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t *idx = p.kept_idx + (int64_t)u * p.budget;
    const bool is_v = (lane / kPieces) & 1;
    const int sub = lane / (2 * kPieces);
    const char *sb = (is_v ? p.src.v : p.src.k) + (lane % kPieces) * 16;
    char *db = (is_v ? p.dst.v : p.dst.k) + (lane % kPieces) * 16;
    const int n_src = p.src.n_max;

    for (int t0 = 0; t0 < cnt; t0 += kInplaceRows * kSlots) {
        if (__ldg(idx + t0) >= cnt) break;                   // the parallel pass takes over from here
        const int j0 = t0 + warp * kGroup;
        int mine = -1, pos = 0;
        int64_t so = -1, dof = -1;
        if (lane < kGroup && j0 + lane < cnt) {
            mine = __ldg(idx + j0 + lane);
            if (mine == j0 + lane) {
                mine = -1;                                   // already in its slot
            } else {
                if (mine >= 0 && mine < n_src) {
                    so = row_offset(p.src, l, s, h, mine);
                    dof = row_offset(p.dst, l, s, h, j0 + lane);
                }
                if (so < 0 || dof < 0) {
                    if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
                    mine = -1; so = -1; dof = -1;
                } else if (p.dst.positions) {
                    pos = p.src.positions ? p.src.positions[(int64_t)u * p.src.n_max + mine] : mine;
                }
            }
        }
        uint4 val[kFastRows];
#pragma unroll
        for (int r = 0; r < kFastRows; ++r) {
            const int64_t o = __shfl_sync(0xffffffffu, so, r * kSlots + sub);
            if (o >= 0) val[r] = ld_stream(sb + o * ESZ);
        }
        __syncthreads();                                     // every source of the tile has been read
#pragma unroll
        for (int r = 0; r < kFastRows; ++r) {
            const int64_t o = __shfl_sync(0xffffffffu, dof, r * kSlots + sub);
            if (o >= 0) *reinterpret_cast<uint4 *>(db + o * ESZ) = val[r];
        }
        if (p.dst.positions && mine >= 0) p.dst.positions[(int64_t)u * p.dst.n_max + j0 + lane] = pos;
    }
}

// The same schedule for the remaining cases (fp32 keys, no value cache): 32-row tiles staged in shared
// memory, the whole unit in one block.
constexpr int kInplaceAnyRows = 32;

__global__ void __launch_bounds__(kInplaceThreads) k_compact_inplace_any(const CompactParams p)
{
    __shared__ uint4 stage[kInplaceAnyRows * 48];
    __shared__ int32_t pos_s[kInplaceAnyRows];
    const int u = p.u0 + blockIdx.x;
    const int h = u % p.H, s = (u / p.H) % p.S, l = u / (p.H * p.S);
    const int cnt = min(__ldg(p.kept_cnt + u), p.budget);
    if (threadIdx.x == 0 && p.new_seq_lens && h == 0 && l == 0) p.new_seq_lens[s] = cnt;
    const int32_t *idx = p.kept_idx + (int64_t)u * p.budget;
    const int per_row = p.k_vec + p.v_vec;

    for (int j0 = 0; j0 < cnt; j0 += kInplaceAnyRows) {
        const int rows = min(kInplaceAnyRows, cnt - j0);
        // a row moves only if its index is inside the unit and both addresses resolve; anything else is reported
        // and left alone
        auto source_of = [&](int r) -> int64_t {
            const int srow = __ldg(idx + j0 + r);
            if (srow == j0 + r) return -2;                     // already in its slot
            return (srow >= 0 && srow < p.src.n_max) ? row_offset(p.src, l, s, h, srow) : -1;
        };
        for (int i = threadIdx.x; i < rows * per_row; i += kInplaceThreads) {
            const int r = i / per_row, c = i - r * per_row;
            const int64_t so = source_of(r);
            if (so == -1 && c == 0 && p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK);
            if (so < 0) continue;
            stage[i] = c < p.k_vec ? ld_stream(p.src.k + so * p.k_esize + c * 16)
                                   : ld_stream(p.src.v + so * p.v_esize + (c - p.k_vec) * 16);
        }
        if (p.dst.positions && threadIdx.x < rows) {
            const int srow = __ldg(idx + j0 + threadIdx.x);
            const bool ok = srow >= 0 && srow < p.src.n_max;
            pos_s[threadIdx.x] = !ok ? -1 : (p.src.positions ? p.src.positions[(int64_t)u * p.src.n_max + srow] : srow);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < rows * per_row; i += kInplaceThreads) {
            const int r = i / per_row, c = i - r * per_row;
            if (source_of(r) < 0) continue;
            const int64_t dof = row_offset(p.dst, l, s, h, j0 + r);
            const bool is_k = c < p.k_vec;
            if (dof < 0) { if (p.device_status) atomicExch(p.device_status, (int)TRI_ERR_DEVICE_CHECK); }
            else if (is_k) *reinterpret_cast<uint4 *>(p.dst.k + dof * p.k_esize + c * 16) = stage[i];
            else *reinterpret_cast<uint4 *>(p.dst.v + dof * p.v_esize + (c - p.k_vec) * 16) = stage[i];
        }
        if (p.dst.positions && threadIdx.x < rows && pos_s[threadIdx.x] >= 0 &&
            __ldg(idx + j0 + threadIdx.x) != j0 + (int)threadIdx.x)
            p.dst.positions[(int64_t)u * p.dst.n_max + j0 + threadIdx.x] = pos_s[threadIdx.x];
        __syncthreads();
    }
}

// new_seq_lens[s] = min(seq_lens[s], n_max, budget): the last launch of a round issued over several unit ranges (the two
// arrays may be one and the same, and every earlier kernel reads the old lengths).
__global__ void k_store_lens(const int32_t *seq_lens, int32_t *new_seq_lens, int32_t S, int32_t n_max, int32_t budget)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < S) new_seq_lens[s] = min(min(seq_lens[s], n_max), budget);
}

// With per-unit budgets the units of a sequence keep different numbers of rows: new_seq_lens[s] is the largest.
__global__ void k_store_max_lens(const int32_t *kept_cnt, int32_t *new_seq_lens, int32_t L, int32_t S, int32_t H)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    int m = 0;
    for (int l = 0; l < L; ++l)
        for (int h = 0; h < H; ++h) m = max(m, kept_cnt[((int64_t)l * S + s) * H + h]);
    new_seq_lens[s] = m;
}

// Window trigger of Section 4.3 on the device.  `decoded[s]` counts the tokens a sequence has decoded since its last
// window boundary; a call adds `step` to it.  At a boundary (count >= beta) the count starts over, and the sequence is
// due for a round if its cache exceeds the budget.  eff_lens[s] = seq_lens[s] for due sequences and 0 for the others,
// which every kernel of the round reads as "nothing cached": no key is scored, no row moves.
__global__ void k_window_begin(const int32_t *seq_lens, int32_t *decoded, int32_t *eff_lens, int32_t S, int32_t step,
                               int32_t beta, int32_t budget)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    int c = decoded[s] + step;
    const bool boundary = c >= beta;
    if (boundary) c = 0;
    decoded[s] = c;
    eff_lens[s] = (boundary && seq_lens[s] > budget) ? seq_lens[s] : 0;
}

// After the round: due sequences shrink to the budget, the others keep their length (the two arrays may be one).
__global__ void k_window_end(const int32_t *seq_lens, const int32_t *eff_lens, int32_t *new_seq_lens, int32_t S,
                             int32_t n_max, int32_t budget)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < S) new_seq_lens[s] = eff_lens[s] > 0 ? min(min(eff_lens[s], n_max), budget) : seq_lens[s];
}

}  // namespace tri

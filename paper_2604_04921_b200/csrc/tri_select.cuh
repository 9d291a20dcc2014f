// Top-B retention (Section 4.3), exact, one block per unit: 1,024 threads, or 256 for units of up to 8,192 keys
// (more blocks per SM hide the latency of the short sweeps better).
//
//   1. value histogram: final scores are z-scores, so a monotone map onto 2048 steps of 1/128 over
//      [-8, 8) spreads a unit's keys over hundreds of bins (the top bits of the fp32 image would send
//      nearly all of them to a dozen bins and serialise the shared-memory atomics).  A top-down scan
//      of the histogram gives the bin that holds the budget-th largest score.
//   2. the keys of that bin -- typically a fraction of a percent -- go to a candidate list in shared
//      memory; an 11 + 11 + 10 bit radix over the list's order-preserving uint32 images gives the exact
//      threshold key T and how many keys equal to T are kept.  If the list overflows (a unit full of
//      equal scores, say) the same radix sweeps the unit's keys instead.
//   3. emit in index order: the unit is cut into spans of at most 32 keys per thread; inside a span warp w
//      owns a contiguous run of keys, 32 at a time, so warp ballots are already in index order and one
//      block-wide scan of the warp totals per span places every kept slot.  When few keys are kept the
//      warp transposes its kept-bit matrix with ballots so that each lane places the kept keys of one row
//      of 32 (work follows the number kept, not the number scanned).
//
// FUSED = true folds the GQA normalise-then-aggregate step into sweep 1: the final score is computed from
// the raw per-head scores and the unit's (mu_g, 1/sigma_g), parked in the score buffer for the later
// sweeps (which hit L2), and the round needs no separate normalisation launch.
#pragma once
#include "tri_score.cuh"

namespace tri {

constexpr int kSelBins = 2048;
constexpr int kSelCand = 4096;                   // candidate list entries
constexpr int kSelSmallUnit = 8192;              // units up to this many keys take the 256-thread block

struct SelectParams {
    const float *scores;      // [U][n_max]   final scores: input (FUSED = false) or parked here by sweep 1
    float *scores_w;          // the same buffer, writable (FUSED = true)
    const int32_t *seq_lens;  // [S]
    int32_t *kept_idx;        // [U][budget]
    int32_t *kept_cnt;        // [U]
    int32_t S, H, n_max, budget;
    int32_t u0;               // first unit of this launch
    const int32_t *unit_budgets;   // [U] or NULL: per-unit budget, clamped to [0, budget]
    // FUSED only: raw scores and partial sums of the scoring kernel
    const float *raw;         // [U][n_max][G]
    const double2 *partials;  // [U][nchunks][G]
    int32_t G, chunk, nchunks;
};

// Monotone map of a score onto 2048 bins: steps of 1/128 over [-8, 8), everything else in the end bins.
__device__ __forceinline__ uint32_t value_bin(float x)
{
    return (uint32_t)min(max(__float2int_rd(fmaf(x, 128.f, 1024.f)), 0), kSelBins - 1);
}

// Exclusive prefix sum of `v` over the block's THREADS threads (thread order); *total gets the block sum.
// warp_sums holds 33 words.
template <int THREADS>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *warp_sums, uint32_t *total)
{
    constexpr int W = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += y;
    }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < W ? warp_sums[lane] : 0u, winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t y = __shfl_up_sync(0xffffffffu, winc, d);
            if (lane >= d) winc += y;
        }
        if (lane < W) warp_sums[lane] = winc - w;   // exclusive warp offsets
        if (lane == 31) warp_sums[32] = winc;  // block total
    }
    __syncthreads();
    uint32_t r = warp_sums[warp] + inc - v;
    *total = warp_sums[32];
    __syncthreads();                            // warp_sums may be reused right away
    return r;
}

// The bin holding the `need`-th largest entry of hist (counted from the top) -> *sel_bin, and how many
// entries are still needed from that bin -> *sel_need.  Thread t owns the 2048 / THREADS bins from
// 2047 - t * (2048 / THREADS) downwards.
template <int THREADS>
__device__ __forceinline__ void find_bin(const uint32_t *hist, uint32_t need, uint32_t *warp_sums, uint32_t *sel_bin,
                                         uint32_t *sel_need)
{
    constexpr int BPT = kSelBins / THREADS;
    const int top = kSelBins - 1 - BPT * (int)threadIdx.x;
    uint32_t c[BPT], sum = 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) { c[q] = hist[top - q]; sum += c[q]; }
    uint32_t total;
    uint32_t above = block_excl_scan<THREADS>(sum, warp_sums, &total);   // entries in strictly higher bins
#pragma unroll
    for (int q = 0; q < BPT; ++q) {
        if (above < need && need <= above + c[q]) { *sel_bin = top - q; *sel_need = need - above; }
        above += c[q];
    }
    __syncthreads();
}

template <bool FUSED, int THREADS>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS) k_select(const SelectParams p)
{
    constexpr int kSelThreads = THREADS;
    __shared__ uint32_t hist[kSelBins];
    __shared__ uint32_t cand[kSelCand];
    __shared__ uint32_t warp_sums[33];
    __shared__ uint32_t sel_bin, sel_need, ncand;
    __shared__ float mu_s[kMaxGroup], rs_s[kMaxGroup];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = p.u0 + blockIdx.x;
    const int s = (u / p.H) % p.S;
    const int n = min(__ldg(p.seq_lens + s), p.n_max);
    const float *sc = p.scores + (int64_t)u * p.n_max;
    int32_t *out = p.kept_idx + (int64_t)u * p.budget;
    const int budget = p.unit_budgets ? min(max(__ldg(p.unit_budgets + u), 0), p.budget) : p.budget;
    const int cnt = min(n, budget);
    if (tid == 0) p.kept_cnt[u] = cnt;
    if (n <= budget || budget == 0) {           // the cache does not exceed the budget: keep all (or nothing is kept)
        for (int i = tid; i < cnt; i += kSelThreads) out[i] = i;
        return;
    }

    // ---- sweep 1: value histogram (and, fused, the final scores themselves) ----
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    if (tid == 0) ncand = 0;
    if (FUSED) unit_mean_rstd(p.partials + (int64_t)u * p.nchunks * p.G, p.G, (n + p.chunk - 1) / p.chunk, n, mu_s, rs_s);
    __syncthreads();
    if (FUSED) {
        const float *rawu = p.raw + (int64_t)u * p.n_max * p.G;
        float *scw = p.scores_w + (int64_t)u * p.n_max;
        if (p.G == 4) {
#pragma unroll 8
            for (int i = tid; i < n; i += kSelThreads) {
                const float z = zmax4(*reinterpret_cast<const float4 *>(rawu + (int64_t)i * 4), mu_s, rs_s);
                scw[i] = z;
                atomicAdd(&hist[value_bin(z)], 1u);
            }
        } else if (p.G == 8) {
#pragma unroll 4
            for (int i = tid; i < n; i += kSelThreads) {
                const float z = zmax8(reinterpret_cast<const float4 *>(rawu + (int64_t)i * 8), mu_s, rs_s);
                scw[i] = z;
                atomicAdd(&hist[value_bin(z)], 1u);
            }
        } else {
            for (int i = tid; i < n; i += kSelThreads) {
                const float z = zmax(rawu + (int64_t)i * p.G, p.G, mu_s, rs_s);
                scw[i] = z;
                atomicAdd(&hist[value_bin(z)], 1u);
            }
        }
    } else {
#pragma unroll 8
        for (int i = tid; i < n; i += kSelThreads) atomicAdd(&hist[value_bin(sc[i])], 1u);
    }
    __syncthreads();                            // histogram complete; parked scores visible to the whole block
    find_bin<THREADS>(hist, (uint32_t)budget, warp_sums, &sel_bin, &sel_need);
    const uint32_t vb = sel_bin;
    uint32_t need = sel_need;                   // keys still to take from value bin vb

    // ---- sweep 2: the keys of bin vb become the candidate list ----
#pragma unroll 8
    for (int i = tid; i < n; i += kSelThreads) {
        const float x = sc[i];
        if (value_bin(x) == vb) {
            const uint32_t pos = atomicAdd(&ncand, 1u);
            if (pos < (uint32_t)kSelCand) cand[pos] = float_key(x);
        }
    }
    __syncthreads();
    const uint32_t nc = ncand;
    const bool fits = nc <= (uint32_t)kSelCand;

    // ---- the exact key of rank `need` inside bin vb, 11 + 11 + 10 bits at a time ----
    uint32_t prefix = 0, pmask = 0;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t bmask = pass == 2 ? 1023u : 2047u;
        for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        if (fits) {
            for (uint32_t i = tid; i < nc; i += kSelThreads) {
                const uint32_t k = cand[i];
                if ((k & pmask) == prefix) atomicAdd(&hist[(k >> shift) & bmask], 1u);
            }
        } else {
#pragma unroll 4
            for (int i = tid; i < n; i += kSelThreads) {
                const float x = sc[i];
                const uint32_t k = float_key(x);
                if (value_bin(x) == vb && (k & pmask) == prefix) atomicAdd(&hist[(k >> shift) & bmask], 1u);
            }
        }
        __syncthreads();
        find_bin<THREADS>(hist, need, warp_sums, &sel_bin, &sel_need);
        prefix |= sel_bin << shift;
        pmask |= bmask << shift;
        need = sel_need;
        __syncthreads();
    }
    const uint32_t T = prefix;     // key of the budget-th largest score; `need` keys equal to T are kept

    // ---- emit kept slots in ascending order; among keys equal to T the lowest slots win ----
    // J keys per thread and span (at most 32, fewer for short units so that no sweep runs empty)
    const int J = min(32, (n + kSelThreads - 1) / kSelThreads);
    const bool dense = 2 * budget > n;        // more than half of the keys are kept
    uint32_t base = 0, need_rem = need;
#pragma unroll 1
    for (int span = 0; span < n; span += kSelThreads * J) {
        const int ibase = span + warp * (32 * J) + lane;
        uint32_t m_gt = 0, m_eq = 0;                          // bit j: key ibase + 32 j is above / equal to T
#pragma unroll 8
        for (int j = 0; j < J; ++j) {                         // loads only: many in flight
            const int i = ibase + 32 * j;
            const uint32_t k = i < n ? float_key(sc[i]) : 0u;  // 0 is below every real key
            m_gt |= (uint32_t)(k > T) << j;
            m_eq |= (uint32_t)(k == T) << j;
        }
        uint32_t w_gt = __popc(m_gt), w_eq = __popc(m_eq);     // this warp's totals
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            w_gt += __shfl_xor_sync(0xffffffffu, w_gt, d);
            w_eq += __shfl_xor_sync(0xffffffffu, w_eq, d);
        }
        // a span holds at most 32,768 keys, so the two 16-bit halves never carry into each other
        uint32_t total;
        uint32_t pre = block_excl_scan<THREADS>(lane == 0 ? (w_gt | (w_eq << 16)) : 0u, warp_sums, &total);
        pre = __shfl_sync(0xffffffffu, pre, 0);
        const uint32_t gt_before = pre & 0xffffu, eq_before = pre >> 16;
        if (dense) {
            // most keys are kept: walk the J slots in order, every lane places its own key
            const uint32_t lt = (1u << lane) - 1u;
            uint32_t gb0 = gt_before, eb0 = eq_before;
            for (int j = 0; j < J; ++j) {
                const bool g = m_gt >> j & 1u, e = m_eq >> j & 1u;
                const uint32_t bg = __ballot_sync(0xffffffffu, g), be = __ballot_sync(0xffffffffu, e);
                const uint32_t gb = gb0 + __popc(bg & lt), eb = eb0 + __popc(be & lt);
                if (g) out[base + gb + min(eb, need_rem)] = ibase + 32 * j;
                else if (e && eb < need_rem) out[base + gb + eb] = ibase + 32 * j;
                gb0 += __popc(bg);
                eb0 += __popc(be);
            }
        } else {
            // Transpose the warp's 32 x J bit matrices: lane j ends up with row j (the keys ibase_w + 32 j + 0..31, one
            // bit per key), so that each lane places the kept keys of one row and work follows the number kept.
            uint32_t row_gt = 0, row_eq = 0;
#pragma unroll 8
            for (int j = 0; j < J; ++j) {
                const uint32_t bg = __ballot_sync(0xffffffffu, m_gt >> j & 1u), be = __ballot_sync(0xffffffffu, m_eq >> j & 1u);
                if (lane == j) { row_gt = bg; row_eq = be; }
            }
            const uint32_t cg = __popc(row_gt), ce = __popc(row_eq);
            uint32_t sg = cg, se = ce;                              // inclusive scans over the rows (lanes)
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t yg = __shfl_up_sync(0xffffffffu, sg, d), ye = __shfl_up_sync(0xffffffffu, se, d);
                if (lane >= d) { sg += yg; se += ye; }
            }
            const uint32_t g0 = gt_before + sg - cg, e0 = eq_before + se - ce;   // kept-above / equal keys before this row
            const int rbase = span + warp * (32 * J) + 32 * lane;                 // slot of the row's first key
            for (uint32_t r = row_gt; r; r &= r - 1) {
                const int l = __ffs(r) - 1;
                const uint32_t low = (1u << l) - 1u;
                out[base + g0 + __popc(row_gt & low) + min(e0 + __popc(row_eq & low), need_rem)] = rbase + l;
            }
            for (uint32_t r = row_eq; r; r &= r - 1) {
                const int l = __ffs(r) - 1;
                const uint32_t low = (1u << l) - 1u;
                const uint32_t eb = e0 + __popc(row_eq & low);
                if (eb < need_rem) out[base + g0 + __popc(row_gt & low) + eb] = rbase + l;
            }
        }
        const uint32_t te = min(total >> 16, need_rem);
        base += (total & 0xffffu) + te;
        need_rem -= te;
    }
}

}  // namespace tri

// Top-B retention (Section 4.3): exact radix threshold on the order-preserving uint32 image of the
// fp32 scores, then an index-ordered emit.  One thread block per unit; everything but the scores
// themselves lives in shared memory, so the pass needs no global scratch.
#pragma once
#include "tri_common.cuh"

namespace tri {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelBins = 2048;
constexpr int kEmitPerThread = 4;

struct SelectParams {
    const float *scores;      // [U][n_max]
    const int32_t *seq_lens;  // [S]
    int32_t *kept_idx;        // [U][budget]
    int32_t *kept_cnt;        // [U]
    int32_t *new_seq_lens;    // [S] or NULL
    int32_t S, H, n_max, budget;
};

// Exclusive prefix sum of `v` over the block's threads (thread order); *total gets the block sum.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t *warp_sums, uint32_t *total)
{
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
        uint32_t w = warp_sums[lane], winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t y = __shfl_up_sync(0xffffffffu, winc, d);
            if (lane >= d) winc += y;
        }
        warp_sums[lane] = winc - w;            // exclusive warp offsets
        if (lane == 31) warp_sums[32] = winc;  // block total
    }
    __syncthreads();
    uint32_t r = warp_sums[warp] + inc - v;
    *total = warp_sums[32];
    __syncthreads();                            // warp_sums may be reused right away
    return r;
}

__global__ void __launch_bounds__(kSelThreads) k_select(const SelectParams p)
{
    __shared__ uint32_t hist[kSelBins];
    __shared__ uint32_t warp_sums[33];
    __shared__ uint32_t sel_bin, sel_need;

    const int tid = threadIdx.x;
    const int u = blockIdx.x;
    const int s = (u / p.H) % p.S;
    const int n = min(__ldg(p.seq_lens + s), p.n_max);
    const float *sc = p.scores + (int64_t)u * p.n_max;
    int32_t *out = p.kept_idx + (int64_t)u * p.budget;
    const int cnt = min(n, p.budget);
    if (tid == 0) {
        p.kept_cnt[u] = cnt;
        if (p.new_seq_lens && (u % p.H) == 0 && u / (p.H * p.S) == 0) p.new_seq_lens[s] = cnt;
    }
    if (n <= p.budget) {                        // the cache does not exceed the budget: keep all
        for (int i = tid; i < n; i += kSelThreads) out[i] = i;
        return;
    }

    // ---- threshold: the budget-th largest key, 11 + 11 + 10 bits at a time ----
    uint32_t prefix = 0, pmask = 0, need = (uint32_t)p.budget;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t bmask = pass == 2 ? 1023u : 2047u;
        for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += kSelThreads) {
            uint32_t k = float_key(sc[i]);
            if ((k & pmask) == prefix) atomicAdd(&hist[(k >> shift) & bmask], 1u);
        }
        __syncthreads();
        // thread t owns bins 2t', 2t'+1 counted from the top: t' = 1023 - t
        const int hi_bin = kSelBins - 1 - 2 * tid, lo_bin = hi_bin - 1;
        const uint32_t ch = hist[hi_bin], cl = hist[lo_bin];
        uint32_t total;
        uint32_t above = block_excl_scan(ch + cl, warp_sums, &total);   // keys in strictly higher bins
        if (above < need && need <= above + ch) { sel_bin = hi_bin; sel_need = need - above; }
        else if (above + ch < need && need <= above + ch + cl) { sel_bin = lo_bin; sel_need = need - above - ch; }
        __syncthreads();
        prefix |= sel_bin << shift;
        pmask |= bmask << shift;
        need = sel_need;
        __syncthreads();
    }
    const uint32_t T = prefix;     // key of the budget-th largest score; `need` keys equal to T are kept

    // ---- emit kept slots in ascending order; among keys equal to T the lowest slots win ----
    uint32_t base = 0, need_rem = need;
    for (int start = 0; start < n; start += kSelThreads * kEmitPerThread) {
        const int i0 = start + tid * kEmitPerThread;
        uint32_t gt = 0, eq = 0, fl_gt = 0, fl_eq = 0;
#pragma unroll
        for (int j = 0; j < kEmitPerThread; ++j) {
            int i = i0 + j;
            if (i < n) {
                uint32_t k = float_key(sc[i]);
                if (k > T) { fl_gt |= 1u << j; ++gt; }
                else if (k == T) { fl_eq |= 1u << j; ++eq; }
            }
        }
        uint32_t total;
        uint32_t pre = block_excl_scan(gt | (eq << 16), warp_sums, &total);
        uint32_t gt_before = pre & 0xffffu, eq_before = pre >> 16;
#pragma unroll
        for (int j = 0; j < kEmitPerThread; ++j) {
            if (fl_gt >> j & 1u) {
                out[base + gt_before + min(eq_before, need_rem)] = i0 + j;
                ++gt_before;
            } else if (fl_eq >> j & 1u) {
                if (eq_before < need_rem) out[base + gt_before + eq_before] = i0 + j;
                ++eq_before;
            }
        }
        uint32_t tg = total & 0xffffu, te = min(total >> 16, need_rem);
        base += tg + te;
        need_rem -= te;
    }
}

}  // namespace tri

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
// Long units that keep at most an eighth of their keys (fused round only) skip all that: a sample gives a safe lower
// bound of the threshold, one ordered sweep over the raw scores collects the few keys above it, and steps 2-3 run on
// that list; the general path stays as the fallback when the check of the list fails (see select_sampled).
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
constexpr int kSelLongUnit = 65536;              // units from this many keys on may take the one-sweep path (measured:
                                                 // at 32,768 keys its fixed phases cost what the saved sweeps gain)

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

// The score whose order-preserving image (float_key) is k.
__device__ __forceinline__ float key_score(uint32_t k)
{
    return __uint_as_float((k >> 31) ? (k ^ 0x80000000u) : ~k);
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

// The exact key of rank `need` (counted from the top) among the keys `each` visits, 11 + 11 + 10 bits at a time.
// `each(visit)` must call visit(key) for every key, spread over the block's threads.  Returns the key and leaves in
// `need` how many keys equal to it belong to the top.
template <int THREADS, class Each>
__device__ __forceinline__ uint32_t radix_kth(Each each, uint32_t &need, uint32_t *hist, uint32_t *warp_sums,
                                              uint32_t *sel_bin, uint32_t *sel_need)
{
    uint32_t prefix = 0, pmask = 0;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t bmask = pass == 2 ? 1023u : 2047u;
        for (int i = threadIdx.x; i < kSelBins; i += THREADS) hist[i] = 0;
        __syncthreads();
        each([&](uint32_t k) {
            // lanes that hit the same bin count as one atomic: scores of one unit share their leading bits, and
            // same-address shared-memory atomics would serialise
            if ((k & pmask) == prefix) {
                const uint32_t bin = (k >> shift) & bmask;
                const uint32_t peers = __match_any_sync(__activemask(), bin);
                if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
            }
        });
        __syncthreads();
        find_bin<THREADS>(hist, need, warp_sums, sel_bin, sel_need);
        prefix |= *sel_bin << shift;
        pmask |= bmask << shift;
        need = *sel_need;
        __syncthreads();
    }
    return prefix;
}

// Ordered emit: of the entries i in [0, n) with key_at(i) > T, and the first `need` entries with key_at(i) == T,
// writes val_at(i) to out in ascending order of i; positions from `cap` on are dropped.
// Returns how many entries qualified.  The range is cut into spans of at most 32 entries per thread; inside a span
// warp w owns a contiguous run, 32 entries at a time, so warp ballots are already in order and one block-wide scan
// of the warp totals per span places everything.  With dense = false the warp transposes its bit matrix with ballots
// so that each lane places the qualifying entries of one row of 32 (work follows the number kept, not the number
// scanned).
template <int THREADS, class KeyAt, class ValAt>
__device__ __forceinline__ uint32_t emit_ordered(int n, KeyAt key_at, uint32_t T, uint32_t need, bool dense, int32_t *out,
                                                 ValAt val_at, uint32_t cap, uint32_t *warp_sums)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int J = min(32, (n + THREADS - 1) / THREADS);   // fewer per thread for short ranges, so that no sweep runs empty
    uint32_t base = 0, need_rem = need;
    auto put = [&](uint32_t pos, int i) {
        if (pos < cap) out[pos] = val_at(i);
    };
#pragma unroll 1
    for (int span = 0; span < n; span += THREADS * J) {
        const int ibase = span + warp * (32 * J) + lane;
        uint32_t m_gt = 0, m_eq = 0;                          // bit j: entry ibase + 32 j is above / equal to T
#pragma unroll 8
        for (int j = 0; j < J; ++j) {                         // loads only: many in flight
            const int i = ibase + 32 * j;
            const uint32_t k = i < n ? key_at(i) : 0u;         // 0 is below every real key
            m_gt |= (uint32_t)(k > T) << j;
            m_eq |= (uint32_t)(k == T) << j;
        }
        uint32_t w_gt = __popc(m_gt), w_eq = __popc(m_eq);     // this warp's totals
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            w_gt += __shfl_xor_sync(0xffffffffu, w_gt, d);
            w_eq += __shfl_xor_sync(0xffffffffu, w_eq, d);
        }
        // a span holds at most 32,768 entries, so the two 16-bit halves never carry into each other
        uint32_t total;
        uint32_t pre = block_excl_scan<THREADS>(lane == 0 ? (w_gt | (w_eq << 16)) : 0u, warp_sums, &total);
        pre = __shfl_sync(0xffffffffu, pre, 0);
        const uint32_t gt_before = pre & 0xffffu, eq_before = pre >> 16;
        if (dense) {
            // most entries qualify: walk the J slots in order, every lane places its own entry
            const uint32_t lt = (1u << lane) - 1u;
            uint32_t gb0 = gt_before, eb0 = eq_before;
            for (int j = 0; j < J; ++j) {
                const bool g = m_gt >> j & 1u, e = m_eq >> j & 1u;
                const uint32_t bg = __ballot_sync(0xffffffffu, g), be = __ballot_sync(0xffffffffu, e);
                const uint32_t gb = gb0 + __popc(bg & lt), eb = eb0 + __popc(be & lt);
                if (g) put(base + gb + min(eb, need_rem), ibase + 32 * j);
                else if (e && eb < need_rem) put(base + gb + eb, ibase + 32 * j);
                gb0 += __popc(bg);
                eb0 += __popc(be);
            }
        } else {
            // Transpose the warp's 32 x J bit matrices: lane j ends up with row j (the entries ibase_w + 32 j + 0..31,
            // one bit each), so that each lane places the qualifying entries of one row.
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
            const uint32_t g0 = gt_before + sg - cg, e0 = eq_before + se - ce;   // qualifying entries before this row
            const int rbase = span + warp * (32 * J) + 32 * lane;                 // index of the row's first entry
            for (uint32_t r = row_gt; r; r &= r - 1) {
                const int l = __ffs(r) - 1;
                const uint32_t low = (1u << l) - 1u;
                put(base + g0 + __popc(row_gt & low) + min(e0 + __popc(row_eq & low), need_rem), rbase + l);
            }
            for (uint32_t r = row_eq; r; r &= r - 1) {
                const int l = __ffs(r) - 1;
                const uint32_t low = (1u << l) - 1u;
                const uint32_t eb = e0 + __popc(row_eq & low);
                if (eb < need_rem) put(base + g0 + __popc(row_gt & low) + eb, rbase + l);
            }
        }
        const uint32_t te = min(total >> 16, need_rem);
        base += (total & 0xffffu) + te;
        need_rem -= te;
    }
    return base;
}

// Long units that keep a small share of their keys, fused round only: one sweep over the raw scores instead of
// three over the final ones, which are never written out.
//   1. sample: kSelCand keys in 512 jittered runs of 8 neighbours (whole 128-byte lines; single keys would cost a
//      DRAM access each).  The sample's k-th largest final score T_lo, k = expected rank of the budget-th largest plus
//      four standard deviations of the sampling error (taken for fully correlated runs), lies below the true
//      threshold unless the sample misleads.
//   2. sweep: the unit is cut into tiles of 128 keys dealt round-robin to the warps, so that every warp sees the
//      whole range of positions (scores depend on the distance to the query; a contiguous share per warp would
//      give the warp that owns the newest keys several times the average).  A warp appends the keys at or above
//      T_lo, slot and score image, to its own segment of a list kept in the unit's score buffer; no block-wide
//      synchronisation while the sweep runs.
//   3. the exact selection on the list, a small multiple of the budget long: the value histogram of the list (filled
//      during the sweep) gives the bin of the budget-th largest, a radix over that bin's few entries its exact image T;
//      then every entry above T (equal to T) sets its slot's bit in one of two bitmaps over the unit, and the kept
//      slots are read off the bitmaps in ascending order, the lowest slots first among those equal to T.
// Whether the sample was good enough is checked, not assumed: if fewer than `budget` keys came through, or a
// segment overflowed, false is returned and the general path runs, so the result is the exact top-B either way.
// GS = group size known at compile time (0: any).
template <int THREADS, int GS>
__device__ __forceinline__ bool select_sampled(const SelectParams &p, const float *rawu, float *scw, int n, int budget,
                                               int32_t *out, const float *mu_s, const float *rs_s, uint32_t *hist,
                                               uint32_t *cand, uint32_t *warp_sums, uint32_t *sel_bin, uint32_t *sel_need,
                                               uint32_t *seg_at, uint32_t *n_sub)
{
    constexpr int W = THREADS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, G = p.G;
    auto key_of = [&](int i) -> uint32_t {       // order-preserving image of the final score of key i
        if (GS == 4) return float_key(zmax4(*reinterpret_cast<const float4 *>(rawu + (int64_t)i * 4), mu_s, rs_s));
        if (GS == 8) return float_key(zmax8(reinterpret_cast<const float4 *>(rawu + (int64_t)i * 8), mu_s, rs_s));
        return float_key(zmax(rawu + (int64_t)i * G, G, mu_s, rs_s));
    };
    // ---- 1. sample ----
    const float share = (float)budget / (float)n;
    // neighbours' scores are correlated (their rotations differ little in the slow bands); in the worst case a run
    // counts as one draw, which multiplies the standard deviation of the sampled count by sqrt(8)
    uint32_t need_lo = (uint32_t)ceilf(kSelCand * share + 4.f * sqrtf(8.f * kSelCand * share * (1.f - share)) + 2.f);
    const uint32_t run_stride = (uint32_t)n / (kSelCand / 8);             // >= 16: n >= 2 kSelCand
    for (uint32_t j = tid; j < (uint32_t)kSelCand; j += THREADS) {
        const uint32_t q = j >> 3;
        const uint32_t first = (q * run_stride + __umulhi(q * 2654435761u, run_stride - 7)) & ~7u;
        cand[j] = key_of((int)(first + (j & 7)));
    }
    __syncthreads();
    const uint32_t T_lo = radix_kth<THREADS>(
        [&](auto visit) {
            for (uint32_t j = tid; j < (uint32_t)kSelCand; j += THREADS) visit(cand[j]);
        },
        need_lo, hist, warp_sums, sel_bin, sel_need);
    if (T_lo == 0) return false;

    // ---- 2. sweep ----  the unit's score buffer: two bitmaps over the slots, then per-warp segments of slots and keys
    const uint32_t bm_words = ((uint32_t)p.n_max + 31) / 32, seg_cap = ((uint32_t)p.n_max - 2 * bm_words) / (2 * W);
    uint32_t *bm_gt = reinterpret_cast<uint32_t *>(scw), *bm_eq = bm_gt + bm_words;
    int32_t *seg_idx = reinterpret_cast<int32_t *>(scw) + 2 * bm_words;
    uint32_t *seg_key = reinterpret_cast<uint32_t *>(scw) + 2 * bm_words + W * seg_cap;
    const uint32_t lt = (1u << lane) - 1u, my_seg = warp * seg_cap;
    uint32_t mine = 0;                                   // entries this warp has appended (warp-uniform)
    for (int i = tid; i < kSelBins; i += THREADS) hist[i] = 0;
    if (tid == 0) *n_sub = 0;
    __syncthreads();
#pragma unroll 1
    for (int r = warp * 128; r < n; r += W * 128) {
        uint32_t k[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int i = r + 32 * x + lane;
            k[x] = i < n ? key_of(i) : 0u;
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const bool take = k[x] >= T_lo;
            const uint32_t b = __ballot_sync(0xffffffffu, take);
            const uint32_t pos = mine + __popc(b & lt);
            if (take) {
                atomicAdd(&hist[value_bin(key_score(k[x]))], 1u);     // value histogram of the list, for step 3
                if (pos < seg_cap) { seg_idx[my_seg + pos] = r + 32 * x + lane; seg_key[my_seg + pos] = k[x]; }
            }
            mine += __popc(b);
        }
    }
    if (lane == 0) warp_sums[warp] = mine;
    const uint32_t n_words = ((uint32_t)n + 31) / 32;
    for (uint32_t j = tid; j < n_words; j += THREADS) { bm_gt[j] = 0u; bm_eq[j] = 0u; }
    __syncthreads();                                     // segments, histogram and cleared bitmaps visible to the block
    uint32_t c = 0;
    bool fits = true;
    for (int w = 0; w < W; ++w) {                        // seg_at[0 .. W] <- where each segment starts in the list
        const uint32_t cw = warp_sums[w];
        if (tid == 0) seg_at[w] = c;
        c += cw;
        fits = fits && cw <= seg_cap;
    }
    if (tid == 0) seg_at[W] = c;
    __syncthreads();                                     // warp_sums is reused below
    if (!fits || c < (uint32_t)budget) return false;

    // ---- 3. the exact selection on the list ----
    auto locate = [&](uint32_t i) -> uint32_t {          // list position -> position in the segment arrays
        uint32_t w = 0;
#pragma unroll
        for (int step = W / 2; step > 0; step >>= 1)
            if (seg_at[w + step] <= i) w += step;
        return w * seg_cap + (i - seg_at[w]);
    };
    // value bin of the budget-th largest; its entries (a few dozen) go to shared memory for the radix.  The list is
    // read 8 entries per thread at a time, loads first: other blocks are streaming, and every dependent trip to
    // global memory costs microseconds
    find_bin<THREADS>(hist, (uint32_t)budget, warp_sums, sel_bin, sel_need);
    const uint32_t vb = *sel_bin;
    uint32_t need = *sel_need;
    __syncthreads();
#pragma unroll 1
    for (uint32_t j0 = 0; j0 < c; j0 += 8 * THREADS) {
        uint32_t k[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const uint32_t j = j0 + x * THREADS + tid;
            k[x] = j < c ? seg_key[locate(j)] : 0u;
        }
#pragma unroll
        for (int x = 0; x < 8; ++x)
            if (k[x] != 0u && value_bin(key_score(k[x])) == vb) {
                const uint32_t pos = atomicAdd(n_sub, 1u);
                if (pos < (uint32_t)kSelCand) cand[pos] = k[x];
            }
    }
    __syncthreads();
    const uint32_t nc = *n_sub;
    if (nc > (uint32_t)kSelCand) return false;           // a value bin full of (nearly) equal scores: general path
    const uint32_t T = radix_kth<THREADS>(
        [&](auto visit) {
            for (uint32_t j = tid; j < nc; j += THREADS) visit(cand[j]);
        },
        need, hist, warp_sums, sel_bin, sel_need);
#pragma unroll 1
    for (uint32_t j0 = 0; j0 < c; j0 += 8 * THREADS) {
        uint32_t k[8];
        int32_t slot[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const uint32_t j = j0 + x * THREADS + tid;
            const uint32_t at = j < c ? locate(j) : 0u;
            k[x] = j < c ? seg_key[at] : 0u;
            slot[x] = j < c ? seg_idx[at] : 0;
        }
#pragma unroll
        for (int x = 0; x < 8; ++x)
            if (k[x] >= T) atomicOr((k[x] > T ? bm_gt : bm_eq) + ((uint32_t)slot[x] >> 5), 1u << (slot[x] & 31));
    }
    __syncthreads();
    // thread t reads off the words [t * wpt, (t + 1) * wpt): counts, two block-wide scans, then its slots in order
    const uint32_t wpt = (n_words + THREADS - 1) / THREADS;
    const uint32_t w0 = min((uint32_t)tid * wpt, n_words), w1 = min(w0 + wpt, n_words);
    uint32_t my_gt = 0, my_eq = 0;
    for (uint32_t j = w0; j < w1; ++j) { my_gt += __popc(bm_gt[j]); my_eq += __popc(bm_eq[j]); }
    uint32_t total;
    uint32_t gb = block_excl_scan<THREADS>(my_gt, warp_sums, &total);
    uint32_t eb = block_excl_scan<THREADS>(my_eq, warp_sums, &total);
    if (my_gt + my_eq)
        for (uint32_t j = w0; j < w1; ++j) {
            const uint32_t g = bm_gt[j], e = bm_eq[j];
            for (uint32_t m = g | e; m; m &= m - 1) {
                const int l = __ffs(m) - 1;
                const int slot = (int)(j * 32 + l);
                if (g >> l & 1u) { out[gb + min(eb, need)] = slot; ++gb; }
                else { if (eb < need) out[gb + eb] = slot; ++eb; }
            }
        }
    return true;
}

template <bool FUSED, int THREADS>
__global__ void __launch_bounds__(THREADS, 2048 / THREADS) k_select(const SelectParams p)
{
    constexpr int kSelThreads = THREADS;
    __shared__ uint32_t hist[kSelBins];
    __shared__ uint32_t cand[kSelCand];
    __shared__ uint32_t warp_sums[33];
    __shared__ uint32_t sel_bin, sel_need, ncand;
    __shared__ uint32_t seg_at[33];
    __shared__ float mu_s[kMaxGroup], rs_s[kMaxGroup];

    const int tid = threadIdx.x;
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
    const float *rawu = FUSED ? p.raw + (int64_t)u * p.n_max * p.G : nullptr;
    float *scw = FUSED ? p.scores_w + (int64_t)u * p.n_max : nullptr;
    if (FUSED) {
        unit_mean_rstd(p.partials + (int64_t)u * p.nchunks * p.G, p.G, (n + p.chunk - 1) / p.chunk, n, mu_s, rs_s);
        __syncthreads();
    }

    // ---- long units that keep a small share: one sweep instead of three (select_sampled) ----
    if constexpr (FUSED && THREADS == 1024) if (n >= kSelLongUnit && 8 * (int64_t)budget <= (int64_t)n) {
        bool done;
        if (p.G == 4) done = select_sampled<THREADS, 4>(p, rawu, scw, n, budget, out, mu_s, rs_s, hist, cand, warp_sums, &sel_bin, &sel_need, seg_at, &ncand);
        else if (p.G == 8) done = select_sampled<THREADS, 8>(p, rawu, scw, n, budget, out, mu_s, rs_s, hist, cand, warp_sums, &sel_bin, &sel_need, seg_at, &ncand);
        else done = select_sampled<THREADS, 0>(p, rawu, scw, n, budget, out, mu_s, rs_s, hist, cand, warp_sums, &sel_bin, &sel_need, seg_at, &ncand);
        if (done) return;
    }

    // ---- sweep 1: value histogram (and, fused, the final scores themselves) ----
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    if (tid == 0) ncand = 0;
    __syncthreads();
    if (FUSED) {
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

    // ---- the exact key of rank `need` inside bin vb ----
    uint32_t T;                    // key of the budget-th largest score; `need` keys equal to T are kept
    if (nc <= (uint32_t)kSelCand)
        T = radix_kth<THREADS>(
            [&](auto visit) {
                for (uint32_t i = tid; i < nc; i += kSelThreads) visit(cand[i]);
            },
            need, hist, warp_sums, &sel_bin, &sel_need);
    else
        T = radix_kth<THREADS>(
            [&](auto visit) {
#pragma unroll 4
                for (int i = tid; i < n; i += kSelThreads) {
                    const float x = sc[i];
                    if (value_bin(x) == vb) visit(float_key(x));
                }
            },
            need, hist, warp_sums, &sel_bin, &sel_need);

    // ---- emit kept slots in ascending order; among keys equal to T the lowest slots win ----
    emit_ordered<THREADS>(n, [&](int i) { return float_key(sc[i]); }, T, need, 2 * budget > n, out, [](int i) { return i; },
                          (uint32_t)budget, warp_sums);
}

}  // namespace tri

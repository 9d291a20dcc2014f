// Shared device-side definitions of the TriAttention compression library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "tri_attention.h"

namespace tri {

constexpr int kHeadDim = 128;
constexpr int kBands = 64;
constexpr int kTileKeys = 16;          // keys per warp tile of the scoring kernel (one MMA M block)
constexpr int kScoreThreads = 256;     // 8 warps
constexpr int kScoreWarps = kScoreThreads / 32;
constexpr int kMaxGroup = 16;

// Device-side copy of a tri_cache_view (same meaning field by field).
struct View {
    char *k;
    char *v;
    int32_t k_kind, paged;
    int64_t stride_layer, stride_seq, stride_head, stride_tok;
    const int32_t *page_table;
    int32_t max_pages_per_seq, page_size, n_pages;
    int32_t page_shift;        // log2(page_size) when it is a power of two, else -1 (host-derived)
    int64_t stride_page, stride_slot;
    const int32_t *seq_lens;
    int32_t *positions;
    int32_t n_max;
};

// Element offset of row n of unit (l, s, h), or -1 if the page id is out of range.
__device__ __forceinline__ int64_t row_offset(const View &w, int l, int s, int h, int n)
{
    if (!w.paged)
        return (int64_t)l * w.stride_layer + (int64_t)s * w.stride_seq + (int64_t)h * w.stride_head +
               (int64_t)n * w.stride_tok;
    const int pg = w.page_shift >= 0 ? n >> w.page_shift : n / w.page_size;
    int page = __ldg(w.page_table + (int64_t)s * w.max_pages_per_seq + pg);
    if (w.n_pages > 0 && (page < 0 || page >= w.n_pages)) return -1;
    return (int64_t)l * w.stride_layer + (int64_t)page * w.stride_page + (int64_t)h * w.stride_head +
           (int64_t)(n - pg * w.page_size) * w.stride_slot;
}

// Order-preserving image of an fp32 in uint32: a > b  <=>  key(a) > key(b) (for non-NaN values); -0.0 and
// +0.0 are equal scores and get the same image.  Never 0 for a non-NaN input.
__device__ __forceinline__ uint32_t float_key(float x)
{
    uint32_t b = __float_as_uint(x + 0.0f);          // -0.0 + 0.0 = +0.0
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}

}  // namespace tri

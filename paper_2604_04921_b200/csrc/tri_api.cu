// Host side of the C ABI declared in include/tri_attention.h: argument checks, workspace carving and
// kernel launches.  Nothing here synchronises the device or allocates after tri_create.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "tri_calib.cuh"
#include "tri_calib_tma.cuh"
#include "tri_compact.cuh"
#include "tri_score.cuh"
#include "tri_score_pre.cuh"
#include "tri_score_tma.cuh"
#include "tri_score_umma.cuh"
#include "tri_select.cuh"

using namespace tri;

constexpr int kHostSlabs = 8;     // layer ranges tri_compress_host is pipelined over
constexpr int kMaxRanges = 16;    // unit ranges one tri_compress may be issued over
constexpr int kKinds = 5;         // kernel kinds timed while profiling: fold, score, normalise, select, compact
constexpr int kMaxProf = 2 + 5 * kMaxRanges;   // launches of one round

struct ProfRec { cudaEvent_t b, e; int kind; };

struct tri_ctx {
    tri_model_desc desc;
    int device;
    double *omega_d;     // [64]
    double2 *dbar_d;     // [64]  (1/|D|) sum_delta e^{i omega_f delta}
    float *qc_d;         // [L][H*G][128]
    float *mw_d;         // [L][H*G][64]   weight of |k_f| in the norm term
    float2 *rot_lo_d, *rot_hi_d;   // phasor tables of the bf16 pre-RoPE path (see k_score_bf16_pre)
    // tri_profile_begin .. tri_profile_end: an event pair around every launch of tri_compress
    bool profiling;
    ProfRec prof[kMaxProf];
    int prof_used;
    // tri_compress_host: device-to-host copies of one layer range run on `back` while the caller's stream
    // already brings in and compresses the next range
    cudaStream_t back;
    cudaEvent_t slab_done[kHostSlabs], back_done;
    bool have_back;
    // tri_compress over unit ranges: selection and compaction of range i run on `side` (highest priority)
    // while the caller's stream already scores range i + 1
    cudaStream_t side;
    cudaEvent_t scored[kMaxRanges], side_done;
    bool have_side;
    int pipeline;        // 0: number of ranges chosen per call, 1: single stream, n: n ranges
    int score_kernel;    // bf16 keys: 0 = tcgen05 kernel (128-key tiles), 1 = mma.sync kernel (16-key warp tiles)
};

// While profiling: an event before and after a launch, on the stream it goes to.  Returns the record's slot.
static int prof_open(tri_ctx *c, int kind, cudaStream_t st)
{
    if (!c->profiling || c->prof_used >= kMaxProf) return -1;
    const int i = c->prof_used++;
    c->prof[i].kind = kind;
    cudaEventRecord(c->prof[i].b, st);
    return i;
}
static void prof_close(tri_ctx *c, int i, cudaStream_t st)
{
    if (i >= 0) cudaEventRecord(c->prof[i].e, st);
}

// Named range on the calling host thread for timeline tools (a no-op when no tool is attached).
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

static thread_local char g_err[256] = "";

static tri_status cuda_fail(cudaError_t e, const char *what)
{
    snprintf(g_err, sizeof g_err, "%s: %s", what, cudaGetErrorString(e));
    return TRI_ERR_CUDA;
}
#define TRI_CUDA(call)                                            \
    do {                                                          \
        cudaError_t e_ = (call);                                  \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);       \
    } while (0)

extern "C" const char *tri_last_cuda_error(void) { return g_err; }

namespace {
cudaError_t prepare_device();   // per-device kernel attributes, defined with the launch helpers below
}

// ----------------------------------------------------------------------------------------------
// context
// ----------------------------------------------------------------------------------------------
extern "C" tri_status tri_create(const tri_model_desc *desc, const float *q_center, const float *q_mean_norm,
                                 tri_ctx **out)
{
    if (!desc || !q_center || !q_mean_norm || !out) return TRI_ERR_INVALID_ARG;
    *out = nullptr;
    if (desc->n_layers <= 0 || desc->n_kv_heads <= 0 || desc->group_size <= 0 || !(desc->rope_theta > 0.0))
        return TRI_ERR_INVALID_ARG;
    if (desc->n_offsets <= 0 || desc->n_offsets > 64 || !desc->offsets) return TRI_ERR_INVALID_ARG;
    for (int i = 0; i < desc->n_offsets; ++i)
        if (desc->offsets[i] < 0) return TRI_ERR_INVALID_ARG;
    if (desc->pair_layout < 0 || desc->pair_layout > 1 || desc->norm_variant < 0 || desc->norm_variant > 2)
        return TRI_ERR_INVALID_ARG;
    if (desc->head_dim != kHeadDim || desc->group_size > kMaxGroup) return TRI_ERR_UNSUPPORTED;

    tri_ctx *c = new (std::nothrow) tri_ctx();
    if (!c) return TRI_ERR_INVALID_ARG;
    c->desc = *desc;
    c->desc.offsets = nullptr;
    c->omega_d = nullptr; c->dbar_d = nullptr; c->qc_d = nullptr; c->mw_d = nullptr; c->rot_lo_d = nullptr; c->rot_hi_d = nullptr;
    c->profiling = false;
    c->prof_used = 0;
    c->have_back = false;
    c->have_side = false;
    c->pipeline = 1;
    // Measured on B200: at G <= 4 the mma.sync kernel already streams at the copy rate and draws less power; from
    // G = 5 on its tensor and issue load grows with G while the tcgen05 kernel's does not (5.8 against 5.5 TB/s at G = 8).
    c->score_kernel = desc->group_size > 4 ? 0 : 1;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "cudaGetDevice"); }

    // omega_f = theta^(-2f/d) (Section 2.1) and the offset-averaged phasor of Section 4.2, in double
    double omega[kBands];
    double2 dbar[kBands];
    for (int f = 0; f < kBands; ++f) {
        omega[f] = std::exp(-(2.0 * f / kHeadDim) * std::log(desc->rope_theta));
        double re = 0.0, im = 0.0;
        for (int i = 0; i < desc->n_offsets; ++i) {
            double a = omega[f] * (double)desc->offsets[i];
            re += std::cos(a);
            im += std::sin(a);
        }
        dbar[f] = make_double2(re / desc->n_offsets, im / desc->n_offsets);
    }
    const size_t nq = (size_t)desc->n_layers * desc->n_kv_heads * desc->group_size;
    std::vector<float> mw(nq * kBands);
    for (size_t i = 0; i < nq; ++i)
        for (int f = 0; f < kBands; ++f) {
            int ir = desc->pair_layout == 0 ? 2 * f : f, ii = desc->pair_layout == 0 ? 2 * f + 1 : f + kBands;
            double cr = q_center[i * kHeadDim + ir], ci = q_center[i * kHeadDim + ii];
            double en = q_mean_norm[i * kBands + f];
            double w = desc->norm_variant == 0 ? en - std::sqrt(cr * cr + ci * ci)
                     : desc->norm_variant == 1 ? en : 0.0;
            mw[i * kBands + f] = (float)w;
        }
    // phasors of query-to-key distances for pre-RoPE bf16 keys: Dbar_f e^{i omega_f b} and e^{i omega_f 512 a}, band-major
    std::vector<float2> rot_lo((size_t)kBands * kRotLo), rot_hi((size_t)kBands * kRotHi);
    for (int f = 0; f < kBands; ++f) {
        for (int b = 0; b < kRotLo; ++b) {
            const double cs = std::cos(omega[f] * b), sn = std::sin(omega[f] * b);
            rot_lo[(size_t)f * kRotLo + b] = make_float2((float)(cs * dbar[f].x - sn * dbar[f].y), (float)(cs * dbar[f].y + sn * dbar[f].x));
        }
        for (int a = 0; a < kRotHi; ++a) {
            const double ang = omega[f] * (double)kRotLo * a;
            rot_hi[(size_t)f * kRotHi + a] = make_float2((float)std::cos(ang), (float)std::sin(ang));
        }
    }
    tri_status st = TRI_OK;
    do {
        if ((e = prepare_device()) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->omega_d, sizeof omega)) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->dbar_d, sizeof dbar)) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->qc_d, nq * kHeadDim * sizeof(float))) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->mw_d, nq * kBands * sizeof(float))) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->omega_d, omega, sizeof omega, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->dbar_d, dbar, sizeof dbar, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->qc_d, q_center, nq * kHeadDim * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->mw_d, mw.data(), nq * kBands * sizeof(float), cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->rot_lo_d, rot_lo.size() * sizeof(float2))) != cudaSuccess) break;
        if ((e = cudaMalloc(&c->rot_hi_d, rot_hi.size() * sizeof(float2))) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->rot_lo_d, rot_lo.data(), rot_lo.size() * sizeof(float2), cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(c->rot_hi_d, rot_hi.data(), rot_hi.size() * sizeof(float2), cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaStreamCreateWithFlags(&c->back, cudaStreamNonBlocking)) != cudaSuccess) break;
        int made = 0;
        for (; made <= kHostSlabs; ++made)
            if ((e = cudaEventCreateWithFlags(made < kHostSlabs ? &c->slab_done[made] : &c->back_done,
                                              cudaEventDisableTiming)) != cudaSuccess)
                break;
        if (e != cudaSuccess) {
            for (int i = 0; i < made; ++i) cudaEventDestroy(i < kHostSlabs ? c->slab_done[i] : c->back_done);
            cudaStreamDestroy(c->back);
            break;
        }
        c->have_back = true;
        // the side stream of the pipelined round; without it (creation failed) rounds run on one stream
        int least = 0, greatest = 0;
        if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) { cudaGetLastError(); break; }
        if (cudaStreamCreateWithPriority(&c->side, cudaStreamNonBlocking, greatest) != cudaSuccess) { cudaGetLastError(); break; }
        int ok = 0;
        for (; ok <= kMaxRanges; ++ok)
            if (cudaEventCreateWithFlags(ok < kMaxRanges ? &c->scored[ok] : &c->side_done, cudaEventDisableTiming) != cudaSuccess)
                break;
        if (ok <= kMaxRanges) {
            cudaGetLastError();
            for (int i = 0; i < ok; ++i) cudaEventDestroy(c->scored[i]);
            cudaStreamDestroy(c->side);
            break;
        }
        c->have_side = true;
    } while (0);
    if (e != cudaSuccess) {
        st = cuda_fail(e, "tri_create");
        tri_destroy(c);
        return st;
    }
    *out = c;
    return TRI_OK;
}

extern "C" tri_status tri_destroy(tri_ctx *c)
{
    if (!c) return TRI_OK;
    if (c->profiling) tri_profile_end(c);
    if (c->have_side) {
        for (int i = 0; i < kMaxRanges; ++i) cudaEventDestroy(c->scored[i]);
        cudaEventDestroy(c->side_done);
        cudaStreamDestroy(c->side);
    }
    if (c->have_back) {
        for (int i = 0; i < kHostSlabs; ++i) cudaEventDestroy(c->slab_done[i]);
        cudaEventDestroy(c->back_done);
        cudaStreamDestroy(c->back);
    }
    cudaFree(c->omega_d);
    cudaFree(c->dbar_d);
    cudaFree(c->qc_d);
    cudaFree(c->mw_d);
    cudaFree(c->rot_lo_d);
    cudaFree(c->rot_hi_d);
    delete c;
    return TRI_OK;
}

// ----------------------------------------------------------------------------------------------
// workspace
// ----------------------------------------------------------------------------------------------
namespace {

struct Plan {
    int32_t U, chunk, nchunks;
    size_t off_E, off_bt, off_bn, off_raw, off_part, off_scores, off_idx, off_cnt, off_eff, total;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Keys per scoring block, evened out over the unit: about 96 warp tiles of 16 keys (1,536 keys) for the mma.sync
// kernel, about 32 tiles of 128 keys (4,096 keys) for the tcgen05 kernel.
void pick_chunk(int32_t n_max, int score_kernel, int32_t *chunk, int32_t *nchunks)
{
    const int32_t tile = score_kernel == 0 ? kUTile : kTileKeys, want = score_kernel == 0 ? 32 : 96;
    int32_t tiles = (n_max + tile - 1) / tile;
    int32_t nch = (tiles + want / 2) / want;
    if (nch < 1) nch = 1;
    int32_t per = (tiles + nch - 1) / nch;
    *chunk = per * tile;
    *nchunks = (tiles + per - 1) / per;
}

// A range of the context's layers; views handed down with it start at its first layer.
struct Layers { int32_t first, count; };

Plan make_plan(const tri_ctx *c, int32_t S, int32_t n_max, int32_t budget, int32_t n_layers = 0)
{
    Plan p;
    const int G = c->desc.group_size;
    p.U = (n_layers > 0 ? n_layers : c->desc.n_layers) * S * c->desc.n_kv_heads;
    pick_chunk(n_max, c->score_kernel, &p.chunk, &p.nchunks);
    size_t o = 0;
    p.off_E = o;      o += align256((size_t)S * kBands * sizeof(double2));
    // tcgen05 kernel: folded B operands per unit (trig) and per (layer, KV head) (norm), 256 bytes per accumulator column
    const size_t ncol = c->score_kernel == 0 ? (G <= 8 ? 16 : 32) : 0;
    p.off_bt = o;     o += align256((size_t)p.U * ncol * 256);
    p.off_bn = o;     o += align256((size_t)(p.U / S) * ncol * 256);
    p.off_raw = o;    o += align256((size_t)p.U * n_max * G * sizeof(float));
    p.off_part = o;   o += align256((size_t)p.U * p.nchunks * G * sizeof(double2));
    p.off_scores = o; o += align256((size_t)p.U * n_max * sizeof(float));
    p.off_idx = o;    o += align256((size_t)p.U * (size_t)(budget > 0 ? budget : 0) * sizeof(int32_t));
    p.off_cnt = o;    o += align256((size_t)p.U * sizeof(int32_t));
    p.off_eff = o;    o += align256((size_t)S * sizeof(int32_t));      // effective lengths of the windowed round
    p.total = o;
    return p;
}

View to_view(const tri_cache_view *v)
{
    View w;
    w.k = (char *)v->k; w.v = (char *)v->v;
    w.k_kind = v->k_kind; w.paged = v->paged;
    w.stride_layer = v->stride_layer; w.stride_seq = v->stride_seq;
    w.stride_head = v->stride_head; w.stride_tok = v->stride_tok;
    w.page_table = v->page_table; w.max_pages_per_seq = v->max_pages_per_seq;
    w.page_size = v->page_size; w.n_pages = v->n_pages;
    w.page_shift = -1;
    if (v->page_size > 0 && (v->page_size & (v->page_size - 1)) == 0)
        for (int sh = 0; sh < 31; ++sh)
            if ((1 << sh) == v->page_size) w.page_shift = sh;
    w.stride_page = v->stride_page; w.stride_slot = v->stride_slot;
    w.seq_lens = v->seq_lens; w.positions = v->positions; w.n_max = v->n_max;
    return w;
}

// Bytes per key element / per value element of a view's format (fp8 caches hold V in fp8 too).
int k_esize_of(int32_t k_kind) { return k_kind == 1 ? 4 : (k_kind == 3 ? 1 : 2); }
int v_esize_of(int32_t k_kind) { return k_kind == 3 ? 1 : 2; }

tri_status check_view(const tri_cache_view *v, bool need_lens)
{
    if (!v || !v->k) return TRI_ERR_INVALID_ARG;
    if (v->k_kind < 0 || v->k_kind > 3 || v->n_max <= 0) return TRI_ERR_INVALID_ARG;
    if (need_lens && !v->seq_lens) return TRI_ERR_INVALID_ARG;
    if (((uintptr_t)v->k & 15) || ((uintptr_t)v->v & 15)) return TRI_ERR_INVALID_ARG;
    const int q = v->k_kind == 3 ? 16 : 8;            // strides in elements; every row starts on a 16-byte boundary
    if (v->stride_layer % q || v->stride_head % q) return TRI_ERR_INVALID_ARG;
    if (v->paged) {
        if (!v->page_table || v->max_pages_per_seq <= 0 || v->page_size <= 0) return TRI_ERR_INVALID_ARG;
        if (v->page_size % kTileKeys) return TRI_ERR_UNSUPPORTED;
        if (v->stride_page % q || v->stride_slot % q || v->stride_slot < kHeadDim) return TRI_ERR_INVALID_ARG;
        if ((int64_t)v->max_pages_per_seq * v->page_size < v->n_max) return TRI_ERR_INVALID_ARG;
    } else {
        if (v->stride_seq % q || v->stride_tok % q || v->stride_tok < kHeadDim) return TRI_ERR_INVALID_ARG;
    }
    return TRI_OK;
}

tri_status check_launch(const char *what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, what);
    return TRI_OK;
}

// The key cache as a rank-5 bf16 tensor for the TMA unit: (dim, row, KV head, sequence | page, layer),
// box = 64 dims x 16 rows, 128-byte swizzle.  Host-side encode only; nothing is allocated.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

tri_status encode_fn(EncodeTiledFn *out)
{
    static EncodeTiledFn fn = nullptr;
    static std::mutex fn_mu;
    std::lock_guard<std::mutex> lock(fn_mu);
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q);
        if (e != cudaSuccess || !ptr) return cuda_fail(e == cudaSuccess ? cudaErrorUnknown : e, "cuTensorMapEncodeTiled lookup");
        fn = (EncodeTiledFn)ptr;
    }
    *out = fn;
    return TRI_OK;
}

tri_status encode_key_map(const tri_ctx *c, const tri_cache_view *v, int32_t S, int32_t n_layers, CUtensorMap *out)
{
    EncodeTiledFn fn;
    tri_status fs = encode_fn(&fn);
    if (fs != TRI_OK) return fs;
    const bool key8 = v->k_kind == 3;               // e4m3 rows: 128 one-byte elements, one box per 16-row tile
    auto bytes = [key8](int64_t elems) { return (cuuint64_t)(elems > 0 ? elems : 16) * (key8 ? 1 : 2); };
    cuuint64_t dims[5], strides[4];
    dims[0] = kHeadDim;
    dims[2] = (cuuint64_t)c->desc.n_kv_heads;
    dims[4] = (cuuint64_t)n_layers;
    if (v->paged) {
        dims[1] = (cuuint64_t)v->page_size;
        dims[3] = v->n_pages > 0 ? (cuuint64_t)v->n_pages : (cuuint64_t)0x7fffffff;
        strides[0] = bytes(v->stride_slot);
        strides[2] = bytes(v->stride_page);
    } else {
        dims[1] = (cuuint64_t)v->n_max;
        dims[3] = (cuuint64_t)S;
        strides[0] = bytes(v->stride_tok);
        strides[2] = bytes(v->stride_seq);
    }
    strides[1] = bytes(v->stride_head);
    strides[3] = bytes(v->stride_layer);
    cuuint32_t box[5] = {(cuuint32_t)(key8 ? kHeadDim : kHeadDim / 2), kTileKeys, 1, 1, 1}, estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(out, key8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, v->k, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_err, sizeof g_err, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return TRI_ERR_CUDA;
    }
    return TRI_OK;
}

// Opt-in shared-memory size of the scoring kernel.  The attribute belongs to (function, device); tri_create sets it
// on the context's device, so contexts on several GPUs need no process-wide bookkeeping.
template <int NT, int LAYOUT>
cudaError_t allow_score_smem()
{
    return cudaFuncSetAttribute(k_score_tma<NT, LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScoreDynSmem);
}

template <int NCOL, int LAYOUT>
cudaError_t allow_umma_smem()
{
    return cudaFuncSetAttribute(k_score_umma<NCOL, LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, umma_smem_bytes(NCOL));
}

cudaError_t prepare_device()
{
    cudaError_t e;
    if ((e = allow_score_smem<1, 0>()) != cudaSuccess) return e;
    if ((e = allow_score_smem<2, 0>()) != cudaSuccess) return e;
    if ((e = allow_score_smem<4, 0>()) != cudaSuccess) return e;
    if ((e = allow_score_smem<1, 1>()) != cudaSuccess) return e;
    if ((e = allow_score_smem<2, 1>()) != cudaSuccess) return e;
    if ((e = allow_score_smem<4, 1>()) != cudaSuccess) return e;
    if ((e = allow_umma_smem<16, 0>()) != cudaSuccess) return e;
    if ((e = allow_umma_smem<32, 0>()) != cudaSuccess) return e;
    if ((e = allow_umma_smem<16, 1>()) != cudaSuccess) return e;
    return allow_umma_smem<32, 1>();
}

// Every entry point that launches kernels runs on the device the context was created on.
tri_status check_device(const tri_ctx *c)
{
    int dev = -1;
    TRI_CUDA(cudaGetDevice(&dev));
    if (dev != c->device) {
        snprintf(g_err, sizeof g_err, "context belongs to device %d but device %d is current", c->device, dev);
        return TRI_ERR_INVALID_ARG;
    }
    return TRI_OK;
}

template <int NT, int LAYOUT>
tri_status launch_score_tma_one(dim3 grid, cudaStream_t st, const CUtensorMap &map, const ScoreParams &sp)
{
    k_score_tma<NT, LAYOUT><<<grid, kScoreThreads, kScoreDynSmem, st>>>(map, sp);
    return TRI_OK;
}

template <int LAYOUT>
void launch_score_fp8(int NT, dim3 grid, cudaStream_t st, const CUtensorMap &map, const ScoreParams &sp)
{
    if (NT == 1) k_score_tma<1, LAYOUT, true><<<grid, kScoreThreads, kScoreDynSmem / 2, st>>>(map, sp);
    else if (NT == 2) k_score_tma<2, LAYOUT, true><<<grid, kScoreThreads, kScoreDynSmem / 2, st>>>(map, sp);
    else k_score_tma<4, LAYOUT, true><<<grid, kScoreThreads, kScoreDynSmem / 2, st>>>(map, sp);
}

template <int LAYOUT>
tri_status launch_score_tma(int NT, dim3 grid, cudaStream_t st, const CUtensorMap &map, const ScoreParams &sp)
{
    if (NT == 1) return launch_score_tma_one<1, LAYOUT>(grid, st, map, sp);
    if (NT == 2) return launch_score_tma_one<2, LAYOUT>(grid, st, map, sp);
    return launch_score_tma_one<4, LAYOUT>(grid, st, map, sp);
}

template <int LAYOUT>
void launch_score_umma(int G, dim3 grid, cudaStream_t st, const CUtensorMap &map, const ScoreParams &sp)
{
    if (G <= 8) k_score_umma<16, LAYOUT><<<grid, kUThreads, umma_smem_bytes(16), st>>>(map, sp);
    else k_score_umma<32, LAYOUT><<<grid, kUThreads, umma_smem_bytes(32), st>>>(map, sp);
}

// A contiguous range of units (u = (layer * S + seq) * H + head) one launch covers.
struct Units { int32_t first, count; };

template <int LAYOUT>
void launch_fold_operands(int G, int U, cudaStream_t st, const OperandParams &op)
{
    if (G <= 8) k_fold_operands<16, LAYOUT><<<U, 256, 0, st>>>(op);
    else k_fold_operands<32, LAYOUT><<<U, 512, 0, st>>>(op);
}

// Fold of everything the scoring kernels need that does not depend on the keys: the phasors of every sequence and,
// for the tcgen05 kernel on bf16 keys, the B operands of its two contractions.
tri_status run_fold(tri_ctx *c, int32_t S, const int64_t *cur_pos, char *ws, const Plan &pl, cudaStream_t st,
                    bool bf16_keys = true, Layers ly = Layers{0, 0})
{
    const int pr = prof_open(c, 0, st);
    k_fold_phasors<<<S, kBands, 0, st>>>(c->omega_d, c->dbar_d, cur_pos, (double2 *)(ws + pl.off_E));
    if (c->score_kernel == 0 && bf16_keys) {
        const size_t head0 = (size_t)ly.first * c->desc.n_kv_heads * c->desc.group_size;
        OperandParams op;
        op.E = (const double2 *)(ws + pl.off_E); op.qc = c->qc_d + head0 * kHeadDim; op.mw = c->mw_d + head0 * kBands;
        op.bt = (uint8_t *)(ws + pl.off_bt); op.bn = (uint8_t *)(ws + pl.off_bn);
        op.S = S; op.H = c->desc.n_kv_heads; op.G = c->desc.group_size;
        if (c->desc.pair_layout == 0) launch_fold_operands<0>(op.G, pl.U, st, op);
        else launch_fold_operands<1>(op.G, pl.U, st, op);
    }
    prof_close(c, pr, st);
    return check_launch("k_fold");
}

// raw scores -> z-score/max (2 launches) of the units `un`; without the last one when `scores` is NULL: the fused
// round leaves the normalisation to its selection kernel.  The phasors must have been folded (run_fold).
tri_status run_score(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos, float *scores,
                     float *raw_out, char *ws, const Plan &pl, int32_t *device_status, cudaStream_t st,
                     Units un, Layers ly = Layers{0, 0}, int32_t skip_upto = 0, const int32_t *unit_budgets = nullptr)
{
    if (ly.count == 0) ly.count = c->desc.n_layers;
    const size_t head0 = (size_t)ly.first * c->desc.n_kv_heads * c->desc.group_size;   // first query head of the range
    const int G = c->desc.group_size;
    double2 *E = (double2 *)(ws + pl.off_E);
    float *raw = raw_out ? raw_out : (float *)(ws + pl.off_raw);
    double2 *part = (double2 *)(ws + pl.off_part);
    tri_status r;

    ScoreParams sp;
    sp.src = to_view(src);
    sp.S = S; sp.H = c->desc.n_kv_heads; sp.G = G; sp.u0 = un.first; sp.skip_upto = skip_upto; sp.unit_budgets = unit_budgets;
    sp.chunk = pl.chunk; sp.nchunks = pl.nchunks;
    sp.E = E; sp.qc = c->qc_d + head0 * kHeadDim; sp.mw = c->mw_d + head0 * kBands;
    sp.bt = (const uint8_t *)(ws + pl.off_bt); sp.bn = (const uint8_t *)(ws + pl.off_bn);
    sp.raw = raw; sp.partials = part; sp.device_status = device_status;
    dim3 grid((unsigned)((size_t)un.count * pl.nchunks));
    int pr = prof_open(c, 1, st);
    if (src->k_kind == 3) {
        // e4m3 keys: the mma.sync kernel on f16 operands, whatever the setting for bf16 keys is
        const int NT = G <= 4 ? 1 : (G <= 8 ? 2 : 4);
        CUtensorMap map;
        if ((r = encode_key_map(c, src, S, ly.count, &map)) != TRI_OK) return r;
        if (c->desc.pair_layout == 0) launch_score_fp8<0>(NT, grid, st, map, sp);
        else launch_score_fp8<1>(NT, grid, st, map, sp);
    } else if (src->k_kind == 0) {
        int NT = G <= 4 ? 1 : (G <= 8 ? 2 : 4);
        CUtensorMap map;
        if ((r = encode_key_map(c, src, S, ly.count, &map)) != TRI_OK) return r;
        if (c->score_kernel == 0) {
            if (c->desc.pair_layout == 0) launch_score_umma<0>(G, grid, st, map, sp);
            else launch_score_umma<1>(G, grid, st, map, sp);
        } else {
            r = c->desc.pair_layout == 0 ? launch_score_tma<0>(NT, grid, st, map, sp)
                                         : launch_score_tma<1>(NT, grid, st, map, sp);
            if (r != TRI_OK) return r;
        }
    } else if (src->k_kind == 2) {
        const int gp = G <= 4 ? 4 : (G <= 8 ? 8 : 16);
        if (c->desc.pair_layout == 0) {
            if (gp == 4) k_score_bf16_pre<0, 4><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
            else if (gp == 8) k_score_bf16_pre<0, 8><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
            else k_score_bf16_pre<0, 16><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
        } else {
            if (gp == 4) k_score_bf16_pre<1, 4><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
            else if (gp == 8) k_score_bf16_pre<1, 8><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
            else k_score_bf16_pre<1, 16><<<grid, kScoreThreads, 0, st>>>(sp, c->rot_lo_d, c->rot_hi_d, cur_pos);
        }
    } else {
        if (c->desc.pair_layout == 0)
            k_score_f32_pre<0><<<grid, kScoreThreads, 0, st>>>(sp, c->omega_d, c->dbar_d, cur_pos);
        else
            k_score_f32_pre<1><<<grid, kScoreThreads, 0, st>>>(sp, c->omega_d, c->dbar_d, cur_pos);
    }
    prof_close(c, pr, st);
    if ((r = check_launch("k_score")) != TRI_OK) return r;
    if (!scores) return TRI_OK;

    NormParams np;
    np.raw = raw; np.partials = part; np.seq_lens = src->seq_lens; np.scores = scores;
    np.S = S; np.H = c->desc.n_kv_heads; np.G = G; np.n_max = src->n_max;
    np.chunk = pl.chunk; np.nchunks = pl.nchunks; np.u0 = un.first;
    pr = prof_open(c, 2, st);
    k_normalize<<<grid, 256, 0, st>>>(np);
    prof_close(c, pr, st);
    return check_launch("k_normalize");
}

// Top-B selection of the units `un`.  pl == NULL: from the final scores in `scores` (tri_select).  pl != NULL: the
// fused round, straight from the raw scores and partial sums in the workspace `ws`; final scores are parked in its
// score area.
tri_status run_select(tri_ctx *c, const float *scores, const int32_t *seq_lens, int32_t S, int32_t n_max,
                      int32_t budget, int32_t *kept_idx, int32_t *kept_cnt,
                      Units un, const Plan *pl, char *ws, cudaStream_t st, const int32_t *unit_budgets = nullptr)
{
    SelectParams p;
    p.unit_budgets = unit_budgets;
    p.scores = scores; p.scores_w = nullptr; p.seq_lens = seq_lens; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
    p.S = S; p.H = c->desc.n_kv_heads; p.n_max = n_max; p.budget = budget; p.u0 = un.first;
    p.raw = nullptr; p.partials = nullptr; p.G = c->desc.group_size; p.chunk = 0; p.nchunks = 0;
    const int U = un.count;
    const int pr = prof_open(c, 3, st);
    if (pl) {
        p.scores_w = (float *)(ws + pl->off_scores);
        p.scores = p.scores_w;
        p.raw = (const float *)(ws + pl->off_raw);
        p.partials = (const double2 *)(ws + pl->off_part);
        p.chunk = pl->chunk; p.nchunks = pl->nchunks;
        if (n_max <= kSelSmallUnit) k_select<true, 256><<<U, 256, 0, st>>>(p);
        else k_select<true, 1024><<<U, 1024, 0, st>>>(p);
    } else {
        if (n_max <= kSelSmallUnit) k_select<false, 256><<<U, 256, 0, st>>>(p);
        else k_select<false, 1024><<<U, 1024, 0, st>>>(p);
    }
    prof_close(c, pr, st);
    return check_launch("k_select");
}

bool aliases(const tri_cache_view *a, const tri_cache_view *b)
{
    return a->k == b->k || (a->v && a->v == b->v) || (a->positions && a->positions == b->positions);
}

// Whether the round compacts bf16 K + V in place: then the gather is two launches (tiled prefix, parallel pass).
bool two_pass_compaction(const tri_cache_view *src, const tri_cache_view *dst)
{
    return aliases(src, dst) && src->k_kind != 1 && src->v && dst->v;
}

tri_status run_compact(tri_ctx *c, const tri_cache_view *src, const int32_t *kept_idx, const int32_t *kept_cnt,
                       int32_t S, int32_t budget, const tri_cache_view *dst, int32_t *new_seq_lens,
                       int32_t *device_status, Units un, cudaStream_t st)
{
    CompactParams p;
    p.src = to_view(src); p.dst = to_view(dst);
    p.kept_idx = kept_idx; p.kept_cnt = kept_cnt; p.new_seq_lens = new_seq_lens;
    p.S = S; p.H = c->desc.n_kv_heads; p.budget = budget; p.u0 = un.first;
    p.k_esize = k_esize_of(src->k_kind);
    p.v_esize = v_esize_of(src->k_kind);
    p.k_vec = kHeadDim * p.k_esize / 16;
    p.v_vec = (src->v && dst->v) ? kHeadDim * p.v_esize / 16 : 0;
    p.device_status = device_status;
    const bool rows16 = (src->k_kind == 0 || src->k_kind == 2) && p.v_vec != 0;     // bf16 K and V: the row-gather kernel applies
    const int U = un.count;
    dim3 grid(U, (budget + kFastRowsPerBlock - 1) / kFastRowsPerBlock);
    const int pr = prof_open(c, 4, st);
    if (aliases(src, dst)) {
        // in place: the prefix whose sources lie inside the destination range goes tile by tile in one block
        // per unit; everything behind it is a hazard-free gather
        if (rows16) {
            k_compact_inplace_rows<2><<<U, kInplaceThreads, 0, st>>>(p);
            k_gather_rows<true><<<grid, kGatherThreads, 0, st>>>(p);
        } else if (src->k_kind == 3 && p.v_vec != 0) {
            dim3 grid8(U, (budget + 2 * kFastRowsPerBlock - 1) / (2 * kFastRowsPerBlock));
            k_compact_inplace_rows<1><<<U, kInplaceThreads, 0, st>>>(p);
            k_gather_rows<true, 1><<<grid8, kGatherThreads, 0, st>>>(p);
        } else {
            k_compact_inplace_any<<<U, kInplaceThreads, 0, st>>>(p);
        }
    } else if (rows16) {
        k_gather_rows<false><<<grid, kGatherThreads, 0, st>>>(p);
    } else if (src->k_kind == 3 && p.v_vec != 0) {
        dim3 grid8(U, (budget + 2 * kFastRowsPerBlock - 1) / (2 * kFastRowsPerBlock));      // 128-byte rows: two slots per warp step
        k_gather_rows<false, 1><<<grid8, kGatherThreads, 0, st>>>(p);
    } else {
        dim3 grid_any(U, (budget + kGatherRowsPerBlock - 1) / kGatherRowsPerBlock);
        k_gather_any<<<grid_any, kGatherThreads, 0, st>>>(p);
    }
    prof_close(c, pr, st);
    return check_launch("k_compact");
}

// Number of unit ranges a round over U units is issued in.  One range = everything on the caller's stream (the
// default).  With several, selection and compaction of a range run on the context's side stream under the scoring of
// the next.  0 asks for an automatic count: about one range per 32 units, at most 8.
int pick_ranges(const tri_ctx *c, int32_t U)
{
    if (!c->have_side) return 1;
    int m = c->pipeline > 0 ? c->pipeline : U / 32;
    if (c->pipeline == 0 && m > 8) m = 8;
    if (m > kMaxRanges) m = kMaxRanges;
    if (m > U) m = U;
    return m < 1 ? 1 : m;
}

tri_status check_common(const tri_ctx *c, int32_t S, int32_t n_max, int32_t budget)
{
    if (!c || S <= 0 || n_max <= 0 || budget <= 0) return TRI_ERR_INVALID_ARG;
    int64_t U = (int64_t)c->desc.n_layers * S * c->desc.n_kv_heads;
    if (U > (1 << 24) || (budget + kGatherRowsPerBlock - 1) / kGatherRowsPerBlock > 65535) return TRI_ERR_UNSUPPORTED;
    return TRI_OK;
}

}  // namespace

extern "C" size_t tri_workspace_bytes(const tri_ctx *c, int32_t S, int32_t n_max, int32_t budget)
{
    if (!c || S <= 0 || n_max <= 0) return 0;
    return make_plan(c, S, n_max, budget).total;
}

// ----------------------------------------------------------------------------------------------
// entry points
// ----------------------------------------------------------------------------------------------
extern "C" tri_status tri_score(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                float *scores, float *raw, void *ws, size_t ws_bytes, void *stream)
{
    tri_status r;
    if (!c || !src || !cur_pos || !scores || !ws) return TRI_ERR_INVALID_ARG;
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_view(src, true)) != TRI_OK) return r;
    if ((r = check_common(c, S, src->n_max, 1)) != TRI_OK) return r;
    if ((uintptr_t)ws & 255) return TRI_ERR_INVALID_ARG;
    Plan pl = make_plan(c, S, src->n_max, 0);
    if (ws_bytes < pl.total) return TRI_ERR_WORKSPACE;
    if ((r = run_fold(c, S, cur_pos, (char *)ws, pl, (cudaStream_t)stream, src->k_kind == 0)) != TRI_OK) return r;
    return run_score(c, src, S, cur_pos, scores, raw, (char *)ws, pl, nullptr, (cudaStream_t)stream, Units{0, pl.U});
}

static tri_status select_impl(tri_ctx *c, const float *scores, const int32_t *seq_lens, int32_t S, int32_t n_max,
                              int32_t budget, const int32_t *unit_budgets, int32_t *kept_idx, int32_t *kept_cnt, void *stream)
{
    tri_status r;
    if (!c || !scores || !seq_lens || !kept_idx || !kept_cnt) return TRI_ERR_INVALID_ARG;
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_common(c, S, n_max, budget)) != TRI_OK) return r;
    int32_t U = c->desc.n_layers * S * c->desc.n_kv_heads;
    return run_select(c, scores, seq_lens, S, n_max, budget, kept_idx, kept_cnt, Units{0, U}, nullptr, nullptr,
                      (cudaStream_t)stream, unit_budgets);
}

extern "C" tri_status tri_select(tri_ctx *c, const float *scores, const int32_t *seq_lens, int32_t S,
                                 int32_t n_max, int32_t budget, int32_t *kept_idx, int32_t *kept_cnt,
                                 void *ws, size_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;   // the selection keeps its histograms and candidates in shared memory
    return select_impl(c, scores, seq_lens, S, n_max, budget, nullptr, kept_idx, kept_cnt, stream);
}

extern "C" tri_status tri_select_budgets(tri_ctx *c, const float *scores, const int32_t *seq_lens, int32_t S,
                                         int32_t n_max, int32_t budget, const int32_t *unit_budgets, int32_t *kept_idx,
                                         int32_t *kept_cnt, void *stream)
{
    if (!unit_budgets) return TRI_ERR_INVALID_ARG;
    return select_impl(c, scores, seq_lens, S, n_max, budget, unit_budgets, kept_idx, kept_cnt, stream);
}

extern "C" tri_status tri_compact(tri_ctx *c, const tri_cache_view *src, const int32_t *kept_idx,
                                  const int32_t *kept_cnt, int32_t S, int32_t budget, const tri_cache_view *dst,
                                  int32_t *new_seq_lens, void *stream)
{
    tri_status r;
    if (!c || !kept_idx || !kept_cnt) return TRI_ERR_INVALID_ARG;
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_view(src, false)) != TRI_OK) return r;
    if ((r = check_view(dst, false)) != TRI_OK) return r;
    if ((r = check_common(c, S, src->n_max, budget)) != TRI_OK) return r;
    if (dst->n_max < budget && dst->n_max < src->n_max) return TRI_ERR_INVALID_ARG;
    if (src->k_kind != dst->k_kind) return TRI_ERR_INVALID_ARG;
    int32_t U = c->desc.n_layers * S * c->desc.n_kv_heads;
    return run_compact(c, src, kept_idx, kept_cnt, S, budget, dst, new_seq_lens, nullptr, Units{0, U}, (cudaStream_t)stream);
}

// The fused round over a range of layers; the views start at the range's first layer.  `ranges` > 1 issues it
// over that many unit ranges, selection and compaction of each on the side stream.
static tri_status compress_layers(tri_ctx *c, Layers ly, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                  int32_t budget, const tri_cache_view *dst, int32_t *kept_idx, int32_t *kept_cnt,
                                  int32_t *new_seq_lens, int32_t *device_status, void *ws, size_t ws_bytes,
                                  cudaStream_t st, int ranges, const int32_t *unit_budgets = nullptr)
{
    tri_status r;
    NvtxRange whole("tri_compress");
    Plan pl = make_plan(c, S, src->n_max, budget, ly.count);
    if (ws_bytes < pl.total) return TRI_ERR_WORKSPACE;
    char *w = (char *)ws;
    int32_t *idx = kept_idx ? kept_idx : (int32_t *)(w + pl.off_idx);
    int32_t *cnt = kept_cnt ? kept_cnt : (int32_t *)(w + pl.off_cnt);
    c->prof_used = 0;
    if ((r = run_fold(c, S, cur_pos, w, pl, st, src->k_kind == 0, ly)) != TRI_OK) return r;
    if (ranges <= 1) {
        const Units all{0, pl.U};
        {
            NvtxRange part("tri_compress: score");
            // sequences that do not exceed the budget are kept whole: their keys are not even read
            if ((r = run_score(c, src, S, cur_pos, nullptr, nullptr, w, pl, device_status, st, all, ly, budget, unit_budgets)) != TRI_OK) return r;
        }
        {
            NvtxRange part("tri_compress: normalise + select");
            if ((r = run_select(c, nullptr, src->seq_lens, S, src->n_max, budget, idx, cnt, all, &pl, w, st, unit_budgets)) != TRI_OK)
                return r;
        }
        // new_seq_lens may be the very array the scoring and selection kernels read the lengths from, so only the
        // last launch of the round (the gather, which reads kept counts, never lengths) stores it
        NvtxRange part("tri_compress: compact");
        if (!unit_budgets || !new_seq_lens) return run_compact(c, src, idx, cnt, S, budget, dst, new_seq_lens, device_status, all, st);
        // per-unit budgets: the units of a sequence keep different numbers of rows; the sequence's entry is the largest
        if ((r = run_compact(c, src, idx, cnt, S, budget, dst, nullptr, device_status, all, st)) != TRI_OK) return r;
        k_store_max_lens<<<(S + 255) / 256, 256, 0, st>>>(cnt, new_seq_lens, ly.count, S, c->desc.n_kv_heads);
        return check_launch("k_store_max_lens");
    }
    // Pipelined: the caller's stream scores range after range; behind each range an event lets the side stream
    // select and compact it while the next range is being scored.  The caller's stream waits for the side stream
    // at the end, so the round is complete for whatever the caller enqueues next (and for a graph capture the
    // side stream has joined again).
    for (int i = 0; i < ranges; ++i) {
        const int32_t a = (int32_t)((int64_t)pl.U * i / ranges), b = (int32_t)((int64_t)pl.U * (i + 1) / ranges);
        const Units un{a, b - a};
        if (un.count == 0) continue;
        if ((r = run_score(c, src, S, cur_pos, nullptr, nullptr, w, pl, device_status, st, un, ly, budget, unit_budgets)) != TRI_OK) return r;
        TRI_CUDA(cudaEventRecord(c->scored[i], st));
        TRI_CUDA(cudaStreamWaitEvent(c->side, c->scored[i], 0));
        if ((r = run_select(c, nullptr, src->seq_lens, S, src->n_max, budget, idx, cnt, un, &pl, w, c->side, unit_budgets)) != TRI_OK) return r;
        if ((r = run_compact(c, src, idx, cnt, S, budget, dst, nullptr, device_status, un, c->side)) != TRI_OK) return r;
    }
    TRI_CUDA(cudaEventRecord(c->side_done, c->side));
    TRI_CUDA(cudaStreamWaitEvent(st, c->side_done, 0));
    if (new_seq_lens) {
        // after every kernel that reads the lengths (new_seq_lens may be that very array)
        if (unit_budgets) k_store_max_lens<<<(S + 255) / 256, 256, 0, st>>>(cnt, new_seq_lens, ly.count, S, c->desc.n_kv_heads);
        else k_store_lens<<<(S + 255) / 256, 256, 0, st>>>(src->seq_lens, new_seq_lens, S, src->n_max, budget);
        return check_launch("k_store_lens");
    }
    return TRI_OK;
}

static tri_status compress_impl(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos, int32_t budget,
                                const int32_t *unit_budgets, const tri_cache_view *dst, int32_t *kept_idx, int32_t *kept_cnt,
                                int32_t *new_seq_lens, int32_t *device_status, void *ws, size_t ws_bytes, void *stream)
{
    tri_status r;
    if (!c || !cur_pos || !ws) return TRI_ERR_INVALID_ARG;
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_view(src, true)) != TRI_OK) return r;
    if ((r = check_view(dst, false)) != TRI_OK) return r;
    if ((r = check_common(c, S, src->n_max, budget)) != TRI_OK) return r;
    if (dst->n_max < budget && dst->n_max < src->n_max) return TRI_ERR_INVALID_ARG;
    if (src->k_kind != dst->k_kind) return TRI_ERR_INVALID_ARG;
    if ((uintptr_t)ws & 255) return TRI_ERR_INVALID_ARG;
    const int32_t U = c->desc.n_layers * S * c->desc.n_kv_heads;
    return compress_layers(c, Layers{0, c->desc.n_layers}, src, S, cur_pos, budget, dst, kept_idx, kept_cnt, new_seq_lens,
                           device_status, ws, ws_bytes, (cudaStream_t)stream, pick_ranges(c, U), unit_budgets);
}

extern "C" tri_status tri_compress(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                   int32_t budget, const tri_cache_view *dst, int32_t *kept_idx,
                                   int32_t *kept_cnt, int32_t *new_seq_lens, int32_t *device_status,
                                   void *ws, size_t ws_bytes, void *stream)
{
    return compress_impl(c, src, S, cur_pos, budget, nullptr, dst, kept_idx, kept_cnt, new_seq_lens, device_status, ws, ws_bytes,
                         stream);
}

extern "C" tri_status tri_compress_budgets(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                           int32_t budget, const int32_t *unit_budgets, const tri_cache_view *dst,
                                           int32_t *kept_idx, int32_t *kept_cnt, int32_t *new_seq_lens,
                                           int32_t *device_status, void *ws, size_t ws_bytes, void *stream)
{
    if (!unit_budgets) return TRI_ERR_INVALID_ARG;
    return compress_impl(c, src, S, cur_pos, budget, unit_budgets, dst, kept_idx, kept_cnt, new_seq_lens, device_status, ws,
                         ws_bytes, stream);
}

extern "C" tri_status tri_compress_windowed(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                            int32_t budget, int32_t *decoded, int32_t step, int32_t beta,
                                            const tri_cache_view *dst, int32_t *kept_idx, int32_t *kept_cnt,
                                            int32_t *new_seq_lens, int32_t *device_status, void *ws, size_t ws_bytes,
                                            void *stream)
{
    if (!c || !src || !decoded || step < 0 || beta <= 0 || !ws || ((uintptr_t)ws & 255) || S <= 0 || !src->seq_lens)
        return TRI_ERR_INVALID_ARG;
    Plan pl = make_plan(c, S, src->n_max > 0 ? src->n_max : 1, budget);
    if (ws_bytes < pl.total) return TRI_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t *eff = (int32_t *)((char *)ws + pl.off_eff);
    tri_cache_view due = *src;
    due.seq_lens = eff;
    // argument checks of the round itself, before the counters are touched
    tri_status r;
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_view(src, true)) != TRI_OK) return r;
    if ((r = check_view(dst, false)) != TRI_OK) return r;
    if ((r = check_common(c, S, src->n_max, budget)) != TRI_OK) return r;
    if (dst->n_max < budget && dst->n_max < src->n_max) return TRI_ERR_INVALID_ARG;
    if (src->k_kind != dst->k_kind) return TRI_ERR_INVALID_ARG;
    k_window_begin<<<(S + 255) / 256, 256, 0, st>>>(src->seq_lens, decoded, eff, S, step, beta, budget);
    if ((r = check_launch("k_window_begin")) != TRI_OK) return r;
    if ((r = compress_impl(c, &due, S, cur_pos, budget, nullptr, dst, kept_idx, kept_cnt, nullptr, device_status, ws, ws_bytes,
                           stream)) != TRI_OK)
        return r;
    if (new_seq_lens) {
        k_window_end<<<(S + 255) / 256, 256, 0, st>>>(src->seq_lens, eff, new_seq_lens, S, src->n_max, budget);
        return check_launch("k_window_end");
    }
    return TRI_OK;
}

extern "C" tri_status tri_set_pipeline(tri_ctx *c, int32_t ranges)
{
    if (!c || ranges < 0 || ranges > kMaxRanges) return TRI_ERR_INVALID_ARG;
    c->pipeline = ranges;
    return TRI_OK;
}

extern "C" tri_status tri_set_score_kernel(tri_ctx *c, int32_t which)
{
    if (!c || which < 0 || which > 1) return TRI_ERR_INVALID_ARG;
    c->score_kernel = which;
    return TRI_OK;
}

extern "C" int32_t tri_compress_launches(const tri_ctx *c, const tri_cache_view *src, int32_t S, const tri_cache_view *dst)
{
    if (!c || !src || !dst || S <= 0) return 0;
    // the phasor fold, then per unit range: score, select (which also normalises), gather; an in-place round of
    // bf16 K + V splits the gather into the tiled prefix pass and the parallel pass behind it
    const int m = pick_ranges(c, c->desc.n_layers * S * c->desc.n_kv_heads);
    return 1 + m * (3 + (two_pass_compaction(src, dst) ? 1 : 0));
}

extern "C" tri_status tri_compress_host(tri_ctx *c, const tri_cache_view *src_host, const tri_cache_view *src_dev,
                                        int32_t S, const int64_t *cur_pos_host, int64_t *cur_pos_dev, int32_t budget,
                                        const tri_cache_view *dst_host, const tri_cache_view *dst_dev,
                                        int32_t *kept_cnt_host, int32_t *kept_cnt_dev,
                                        void *ws, size_t ws_bytes, void *stream)
{
    if (!c || !src_host || !src_dev || !dst_host || !dst_dev || !cur_pos_host || !cur_pos_dev || !kept_cnt_dev)
        return TRI_ERR_INVALID_ARG;
    if (src_host->paged || src_dev->paged || dst_host->paged || dst_dev->paged) return TRI_ERR_UNSUPPORTED;
    if (src_host->stride_layer != src_dev->stride_layer || dst_host->stride_layer != dst_dev->stride_layer ||
        src_host->n_max != src_dev->n_max || dst_host->n_max != dst_dev->n_max)
        return TRI_ERR_INVALID_ARG;
    if (!src_host->seq_lens || !src_dev->seq_lens || !src_host->k || !dst_host->k) return TRI_ERR_INVALID_ARG;
    tri_status r;
    NvtxRange whole("tri_compress_host");
    if ((r = check_device(c)) != TRI_OK) return r;
    if ((r = check_view(src_dev, true)) != TRI_OK) return r;
    if ((r = check_view(dst_dev, false)) != TRI_OK) return r;
    if ((r = check_common(c, S, src_dev->n_max, budget)) != TRI_OK) return r;
    if (dst_dev->n_max < budget && dst_dev->n_max < src_dev->n_max) return TRI_ERR_INVALID_ARG;
    if (src_dev->k_kind != dst_dev->k_kind || !ws || ((uintptr_t)ws & 255)) return TRI_ERR_INVALID_ARG;
    if (src_dev->k_kind == 3) return TRI_ERR_UNSUPPORTED;       // host-resident fp8 caches: not built
    cudaStream_t st = (cudaStream_t)stream;
    const int L = c->desc.n_layers, H = c->desc.n_kv_heads;
    const size_t kes = src_host->k_kind == 1 ? 4 : 2;
    // Keys are streamed in full by the scoring kernel, so they are copied.  Values and positions are only read
    // for the kept rows: when the host arrays are device-accessible (pinned, mapped), the gather reads those
    // rows straight from host memory and the bulk copies are skipped.
    auto device_alias = [](const void *host_ptr) -> void * {
        cudaPointerAttributes a;
        if (!host_ptr || cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
    };
    // (in place only pays when most rows are dropped: row-sized reads across the link are slower than a bulk copy)
    const bool sparse = 2 * (int64_t)budget <= src_dev->n_max;
    void *v_alias = (sparse && src_host->v && src_dev->v) ? device_alias(src_host->v) : nullptr;
    void *pos_alias = (sparse && src_host->positions && src_dev->positions) ? device_alias(src_host->positions) : nullptr;
    // Layer ranges: range i is copied in and compressed on the caller's stream; its results go back to the host
    // on the context's copy stream while range i + 1 is already coming in (the link is full duplex).
    const int M = c->have_back ? (L < kHostSlabs ? L : kHostSlabs) : 1;
    // the workspace must hold the largest range; checked before the first copy is enqueued
    const int widest = (L + M - 1) / M;
    if (ws_bytes < make_plan(c, S, src_dev->n_max, budget, widest).total) return TRI_ERR_WORKSPACE;
    TRI_CUDA(cudaMemcpyAsync((void *)src_dev->seq_lens, src_host->seq_lens, S * sizeof(int32_t),
                             cudaMemcpyHostToDevice, st));
    TRI_CUDA(cudaMemcpyAsync(cur_pos_dev, cur_pos_host, S * sizeof(int64_t), cudaMemcpyHostToDevice, st));
    cudaStream_t back = M > 1 ? c->back : st;
    const size_t upl = (size_t)S * H;                                  // units per layer
    for (int i = 0; i < M; ++i) {
        const int l0 = (int)((int64_t)L * i / M), nl = (int)((int64_t)L * (i + 1) / M) - l0;
        const size_t so = (size_t)l0 * src_host->stride_layer, sn = (size_t)nl * src_host->stride_layer;
        const size_t dof = (size_t)l0 * dst_host->stride_layer, dn = (size_t)nl * dst_host->stride_layer;
        const size_t u0 = (size_t)l0 * upl, un = (size_t)nl * upl;
        tri_cache_view sv = *src_dev, dv = *dst_dev;
        sv.k = (char *)src_dev->k + so * kes;
        TRI_CUDA(cudaMemcpyAsync(sv.k, (const char *)src_host->k + so * kes, sn * kes, cudaMemcpyHostToDevice, st));
        if (src_host->v && src_dev->v) {
            if (v_alias) {
                sv.v = (char *)v_alias + so * 2;
            } else {
                sv.v = (char *)src_dev->v + so * 2;
                TRI_CUDA(cudaMemcpyAsync(sv.v, (const char *)src_host->v + so * 2, sn * 2, cudaMemcpyHostToDevice, st));
            }
        }
        if (src_host->positions && src_dev->positions) {
            const size_t po = u0 * src_host->n_max, pn = un * src_host->n_max;
            if (pos_alias) {
                sv.positions = (int32_t *)pos_alias + po;
            } else {
                sv.positions = src_dev->positions + po;
                TRI_CUDA(cudaMemcpyAsync(sv.positions, src_host->positions + po, pn * sizeof(int32_t),
                                         cudaMemcpyHostToDevice, st));
            }
        }
        dv.k = (char *)dst_dev->k + dof * kes;
        if (dst_dev->v) dv.v = (char *)dst_dev->v + dof * 2;
        if (dst_dev->positions) dv.positions = dst_dev->positions + u0 * dst_dev->n_max;
        if ((r = compress_layers(c, Layers{l0, nl}, &sv, S, cur_pos_dev, budget, &dv, nullptr, kept_cnt_dev + u0, nullptr,
                                 nullptr, ws, ws_bytes, st, 1)) != TRI_OK)
            return r;
        if (M > 1) {
            TRI_CUDA(cudaEventRecord(c->slab_done[i], st));
            TRI_CUDA(cudaStreamWaitEvent(back, c->slab_done[i], 0));
        }
        TRI_CUDA(cudaMemcpyAsync((char *)dst_host->k + dof * kes, dv.k, dn * kes, cudaMemcpyDeviceToHost, back));
        if (dst_host->v && dst_dev->v)
            TRI_CUDA(cudaMemcpyAsync((char *)dst_host->v + dof * 2, dv.v, dn * 2, cudaMemcpyDeviceToHost, back));
        if (dst_host->positions && dst_dev->positions)
            TRI_CUDA(cudaMemcpyAsync(dst_host->positions + u0 * dst_host->n_max, dv.positions,
                                     un * dst_host->n_max * sizeof(int32_t), cudaMemcpyDeviceToHost, back));
        if (kept_cnt_host)
            TRI_CUDA(cudaMemcpyAsync(kept_cnt_host + u0, kept_cnt_dev + u0, un * sizeof(int32_t), cudaMemcpyDeviceToHost, back));
    }
    if (M > 1) {
        TRI_CUDA(cudaEventRecord(c->back_done, back));
        TRI_CUDA(cudaStreamWaitEvent(st, c->back_done, 0));
    }
    return TRI_OK;
}

extern "C" tri_status tri_selftest_bounded_wait(int32_t *device_status, void *stream)
{
    if (!device_status) return TRI_ERR_INVALID_ARG;
    k_selftest_wait<<<1, 32, 0, (cudaStream_t)stream>>>(device_status);      // the spinning wait of the mma.sync kernel
    k_selftest_nap<<<1, 32, 0, (cudaStream_t)stream>>>(device_status);       // the sleeping wait of the tcgen05 kernel
    return check_launch("k_selftest_wait");
}

// ----------------------------------------------------------------------------------------------
// per-kernel timing of tri_compress (measurement aid)
// ----------------------------------------------------------------------------------------------
extern "C" tri_status tri_profile_begin(tri_ctx *c)
{
    if (!c) return TRI_ERR_INVALID_ARG;
    if (c->profiling) return TRI_OK;
    for (int i = 0; i < kMaxProf; ++i) {
        cudaError_t e = cudaEventCreate(&c->prof[i].b);
        if (e == cudaSuccess && (e = cudaEventCreate(&c->prof[i].e)) != cudaSuccess) cudaEventDestroy(c->prof[i].b);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) { cudaEventDestroy(c->prof[j].b); cudaEventDestroy(c->prof[j].e); }
            return cuda_fail(e, "cudaEventCreate");
        }
    }
    c->prof_used = 0;
    c->profiling = true;
    return TRI_OK;
}

extern "C" tri_status tri_profile_read(tri_ctx *c, float *ms)
{
    if (!c || !ms || !c->profiling) return TRI_ERR_INVALID_ARG;
    for (int k = 0; k < kKinds; ++k) ms[k] = 0.f;
    for (int i = 0; i < c->prof_used; ++i) {
        float t = 0.f;
        TRI_CUDA(cudaEventSynchronize(c->prof[i].e));
        TRI_CUDA(cudaEventElapsedTime(&t, c->prof[i].b, c->prof[i].e));
        ms[c->prof[i].kind] += t;
    }
    return TRI_OK;
}

extern "C" tri_status tri_profile_end(tri_ctx *c)
{
    if (!c) return TRI_ERR_INVALID_ARG;
    if (c->profiling)
        for (int i = 0; i < kMaxProf; ++i) { cudaEventDestroy(c->prof[i].b); cudaEventDestroy(c->prof[i].e); }
    c->profiling = false;
    c->prof_used = 0;
    return TRI_OK;
}

// ----------------------------------------------------------------------------------------------
// tri_score_static: scoring with the workspace in a device global instead of a caller's buffer
// ----------------------------------------------------------------------------------------------
// One copy per device that loads this module, held until the process exits.  In host code the name
// below is only a handle for cudaGetSymbolAddress: it is not a device address and must never be
// passed to a kernel as one.
static __device__ __align__(256) unsigned char g_score_scratch[TRI_SCORE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static void *g_score_scratch_addr[kMaxDevices];   // device address of g_score_scratch, per device, once looked up
static std::mutex g_score_scratch_mu;

// Device address of the scratch array on the current device; the first call per device asks the runtime.
static tri_status score_scratch_address(int dev, void **out)
{
    std::lock_guard<std::mutex> lock(g_score_scratch_mu);
    if (!g_score_scratch_addr[dev]) {
        void *p = nullptr;
        TRI_CUDA(cudaGetSymbolAddress(&p, g_score_scratch));
        if (!p) return cuda_fail(cudaErrorInvalidSymbol, "cudaGetSymbolAddress(g_score_scratch)");
        g_score_scratch_addr[dev] = p;
    }
    *out = g_score_scratch_addr[dev];
    return TRI_OK;
}

extern "C" size_t tri_score_static_bytes(const tri_ctx *c, int32_t S, int32_t n_max)
{
    if (!c || S <= 0 || n_max <= 0) return 0;
    return make_plan(c, S, n_max, 0).off_scores;    // phasors (+ folded operands) + raw scores + partial sums
}

extern "C" tri_status tri_score_static(tri_ctx *c, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                       float *scores, float *raw, void *stream)
{
    tri_status r;
    if (!c || !src || !cur_pos || !scores) return TRI_ERR_INVALID_ARG;
    if ((r = check_view(src, true)) != TRI_OK) return r;
    if ((r = check_common(c, S, src->n_max, 1)) != TRI_OK) return r;
    Plan pl = make_plan(c, S, src->n_max, 0);
    const size_t need = pl.off_scores;           // phasors + raw scores + partial sums; scores go to the caller
    if (need > (size_t)TRI_SCORE_STATIC_SCRATCH_BYTES) {
        snprintf(g_err, sizeof g_err, "tri_score_static: this shape needs %zu bytes of scratch, the built-in array holds %zu",
                 need, (size_t)TRI_SCORE_STATIC_SCRATCH_BYTES);
        return TRI_ERR_WORKSPACE;
    }
    int dev = -1;
    TRI_CUDA(cudaGetDevice(&dev));
    if (dev != c->device || dev < 0 || dev >= kMaxDevices) return TRI_ERR_INVALID_ARG;
    void *ws = nullptr;
    if ((r = score_scratch_address(dev, &ws)) != TRI_OK) return r;
    if ((r = run_fold(c, S, cur_pos, (char *)ws, pl, (cudaStream_t)stream, src->k_kind == 0)) != TRI_OK) return r;
    return run_score(c, src, S, cur_pos, scores, raw, (char *)ws, pl, nullptr, (cudaStream_t)stream, Units{0, pl.U});
}

// ----------------------------------------------------------------------------------------------
// calibration statistics
// ----------------------------------------------------------------------------------------------
namespace {

// Blocks per head and tokens per block: enough blocks to fill the GPU several times over, at least 256
// tokens each, at most 1,024 blocks per head.
void calib_shape(int32_t n_heads, int64_t T, int32_t *nblocks, int32_t *per_block)
{
    int64_t want = (148 * 16 + n_heads - 1) / n_heads;
    int64_t most = (T + 255) / 256;
    int64_t nb = want < most ? want : most;
    if (nb > 1024) nb = 1024;
    if (nb < 1) nb = 1;
    int64_t per = ((T + nb - 1) / nb + 15) / 16 * 16;      // whole 16-token tiles
    *per_block = (int32_t)per;
    *nblocks = (int32_t)((T + per - 1) / per);
}

// The queries as a rank-3 tensor (component, head, token) for the TMA unit, box = one 4 KB tile of one head.
// false when the layout does not meet the unit's alignment rules (the caller then takes the plain-load kernel).
bool calib_tma_ok(const void *q, int32_t q_kind, int64_t T, int32_t n_heads, int64_t stride_tok, int64_t stride_head)
{
    const int64_t es = q_kind == 0 ? 2 : 4;
    if (((uintptr_t)q & 15) || (stride_tok * es) % 16 || stride_tok <= 0 || T >= (int64_t)1 << 31) return false;
    if (n_heads > 1 && ((stride_head * es) % 16 || stride_head <= 0)) return false;
    return stride_tok * es < ((int64_t)1 << 40) && stride_head * es < ((int64_t)1 << 40);
}

tri_status encode_calib_map(const void *q, int32_t q_kind, int64_t T, int32_t n_heads, int64_t stride_tok,
                            int64_t stride_head, CUtensorMap *out)
{
    EncodeTiledFn fn;
    tri_status fs = encode_fn(&fn);
    if (fs != TRI_OK) return fs;
    const cuuint64_t es = q_kind == 0 ? 2 : 4;
    cuuint64_t dims[3] = {kHeadDim, (cuuint64_t)n_heads, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)(n_heads > 1 ? stride_head : kHeadDim) * es, (cuuint64_t)stride_tok * es};
    cuuint32_t box[3] = {kHeadDim, 1, (cuuint32_t)(kCalibTileBytes / (kHeadDim * es))}, estr[3] = {1, 1, 1};
    CUresult r = fn(out, q_kind == 0 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                    const_cast<void *>(q), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_err, sizeof g_err, "cuTensorMapEncodeTiled (calibration) failed with CUresult %d", (int)r);
        return TRI_ERR_CUDA;
    }
    return TRI_OK;
}

template <int LAYOUT, int KIND>
tri_status launch_calib_tma(dim3 grid, cudaStream_t st, const CUtensorMap &map, const CalibParams &p)
{
    // the attribute belongs to (function, device): set it on the current device before every launch (cheap, no sync)
    TRI_CUDA(cudaFuncSetAttribute(k_calib_tma<LAYOUT, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, kCalibDynSmem));
    k_calib_tma<LAYOUT, KIND><<<grid, kCalibThreads, kCalibDynSmem, st>>>(map, p);
    return TRI_OK;
}

}  // namespace

extern "C" size_t tri_calib_state_bytes(int32_t n_heads)
{
    return n_heads > 0 ? ((size_t)n_heads * kCalibSums + 1) * sizeof(double) : 0;
}

extern "C" size_t tri_calib_workspace_bytes(int32_t n_heads, int64_t T)
{
    if (n_heads <= 0 || T <= 0) return 0;
    int32_t nb, per;
    calib_shape(n_heads, T, &nb, &per);
    return (size_t)n_heads * nb * kCalibSums * sizeof(double);
}

extern "C" tri_status tri_calib_reset(void *state, int32_t n_heads, void *stream)
{
    if (!state || n_heads <= 0 || ((uintptr_t)state & 7)) return TRI_ERR_INVALID_ARG;
    TRI_CUDA(cudaMemsetAsync(state, 0, tri_calib_state_bytes(n_heads), (cudaStream_t)stream));
    return TRI_OK;
}

extern "C" tri_status tri_calib_accumulate(const void *q, int32_t q_kind, int64_t T, int32_t n_heads, int64_t stride_tok,
                                           int64_t stride_head, int32_t pair_layout, void *state, void *ws,
                                           size_t ws_bytes, void *stream)
{
    if (!q || !state || !ws || T <= 0 || n_heads <= 0 || n_heads > 65535) return TRI_ERR_INVALID_ARG;
    if (q_kind < 0 || q_kind > 1 || pair_layout < 0 || pair_layout > 1) return TRI_ERR_INVALID_ARG;
    if (stride_tok % 4 || stride_head % 4 || stride_head < kHeadDim || ((uintptr_t)q & (q_kind == 0 ? 7 : 15)))
        return TRI_ERR_INVALID_ARG;
    if (((uintptr_t)state & 7) || ((uintptr_t)ws & 7)) return TRI_ERR_INVALID_ARG;
    if (ws_bytes < tri_calib_workspace_bytes(n_heads, T)) return TRI_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    CalibParams p;
    p.q = q; p.T = T; p.stride_tok = stride_tok; p.stride_head = stride_head;
    int32_t nb;
    calib_shape(n_heads, T, &nb, &p.per_block);
    p.partials = (double *)ws;
    dim3 grid(nb, n_heads);
    if (calib_tma_ok(q, q_kind, T, n_heads, stride_tok, stride_head)) {
        CUtensorMap map;
        tri_status ms = encode_calib_map(q, q_kind, T, n_heads, stride_tok, stride_head, &map);
        if (ms != TRI_OK) return ms;
        if (pair_layout == 0 && q_kind == 0) ms = launch_calib_tma<0, 0>(grid, st, map, p);
        else if (pair_layout == 0) ms = launch_calib_tma<0, 1>(grid, st, map, p);
        else if (q_kind == 0) ms = launch_calib_tma<1, 0>(grid, st, map, p);
        else ms = launch_calib_tma<1, 1>(grid, st, map, p);
        if (ms != TRI_OK) return ms;
    } else if (pair_layout == 0 && q_kind == 0) k_calib_partial<0, 0><<<grid, kCalibThreads, 0, st>>>(p);
    else if (pair_layout == 0) k_calib_partial<0, 1><<<grid, kCalibThreads, 0, st>>>(p);
    else if (q_kind == 0) k_calib_partial<1, 0><<<grid, kCalibThreads, 0, st>>>(p);
    else k_calib_partial<1, 1><<<grid, kCalibThreads, 0, st>>>(p);
    tri_status r = check_launch("k_calib_partial");
    if (r != TRI_OK) return r;
    k_calib_merge<<<n_heads, kCalibSums, 0, st>>>(p.partials, nb, T, (double *)state, n_heads);
    return check_launch("k_calib_merge");
}

extern "C" tri_status tri_calib_finalize(const void *state, int32_t n_heads, int32_t pair_layout, float *q_center,
                                         float *q_mean_norm, float *mrl, void *stream)
{
    if (!state || !q_center || !q_mean_norm || n_heads <= 0 || pair_layout < 0 || pair_layout > 1)
        return TRI_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (pair_layout == 0) k_calib_finish<0><<<n_heads, kBands, 0, st>>>((const double *)state, n_heads, q_center, q_mean_norm, mrl);
    else k_calib_finish<1><<<n_heads, kBands, 0, st>>>((const double *)state, n_heads, q_center, q_mean_norm, mrl);
    return check_launch("k_calib_finish");
}
